"""The entry point that allocates nothing (vq_gemm_small_batch_host_static).

Some users of this library run where device allocation is off limits: inside a server whose GPU
memory belongs to its own arena, in a latency-critical loop that must not enter the driver's
allocator, or as a plug-in that receives device pointers but no allocator.  For them the library
keeps the device staging copies of X and Y in a fixed 2 MiB array of its own.  This file checks,
through the C-ABI, that the variant returns what the workspace-based entry point returns, twice in
a row (the second call meets the first call's left-overs in the shared array), and that problems
beyond the fixed size are refused before anything is launched.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test."""
import ctypes
import gc

import numpy as np
import pytest

import vq_synth
from oracle import vq_oracle as orc
from tests.helpers import TOL, DeviceLayer, draw, oracle_fmt

import paper_2402_15319_b200 as vq


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2402_15319_b200 import build as vq_build
    vq_build.build()
    vq.load()


def test_oversized_problem_is_refused_on_the_host():
    # 16 x (65536 + 65536) x 2 bytes = 4 MiB > 2 MiB: refused by size alone, no pointer is touched
    fmt = vq.VQFormat(65536, 65536, 2, 4, 1, 2048, vq.VQ_CB_INT8_SCALED)
    fake = ctypes.c_void_p(0x10000)
    c = fmt.c()
    code = vq.load().vq_gemm_small_batch_host_static(ctypes.byref(c), fake, fake, fake, fake, fake, 16, None)
    assert code == 5
    assert vq.vq_static_scratch_bytes() == 2 << 20
    assert vq.load().vq_gemm_small_batch_host_static(ctypes.byref(c), fake, fake, fake, None, fake, 1, None) == 1
    assert vq.load().vq_gemm_small_batch_host_static(ctypes.byref(c), fake, fake, fake, fake, fake, 17, None) == 6


@pytest.mark.gpu
@pytest.mark.parametrize("spec", [
    vq_synth.LayerSpec("na_blockcb", N=256, K=1024, d=2, b=6, Br=128, Bc=128, int8=False),
    vq_synth.LayerSpec("na_rowcb", N=208, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("na_generic", N=37, K=312, d=1, b=5, Br=1, Bc=156, int8=False),
], ids=lambda s: s.name)
def test_static_scratch_variant_matches_workspace_variant_twice(spec):
    import torch
    L = draw(spec, 31)
    dev = DeviceLayer(spec, L)
    f = oracle_fmt(spec)
    for call, batch in enumerate((5, 3)):      # two calls in a row, the second smaller than the first
        X = vq_synth.make_x(spec, 40 + call, batch)
        hX = torch.from_numpy(X).pin_memory()
        # existing entry point: caller-allocated workspace
        hY_ref = torch.zeros((batch, spec.N), dtype=torch.float16).pin_memory()
        ws = torch.zeros(vq.vq_workspace_bytes_host(dev.fmt, batch), dtype=torch.uint8, device="cuda")
        vq.vq_gemm_small_batch_host(dev.fmt, dev.idx, dev.cb, dev.scale, hX, hY_ref, batch, ws)
        torch.cuda.synchronize()
        # new entry point: no workspace argument at all
        hY = torch.full((batch, spec.N), float("nan"), dtype=torch.float16).pin_memory()
        vq.vq_gemm_small_batch_host_static(dev.fmt, dev.idx, dev.cb, dev.scale, hX, hY, batch)
        torch.cuda.synchronize()
        got, want = hY.numpy().astype(np.float64), hY_ref.numpy().astype(np.float64)
        assert np.isfinite(got).all()
        Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X, threads=4)
        assert (np.abs(got - want) <= TOL * A).all(), f"{spec.name} call {call}: differs from the workspace variant"
        assert (np.abs(got - Y) <= TOL * A).all(), f"{spec.name} call {call}: differs from the oracle"
        # a further call allocates nothing: neither the driver's free memory nor torch's pool moves
        # (garbage of earlier tests is collected first, so that nothing but this call can move the numbers)
        gc.collect()
        torch.cuda.synchronize()
        free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        vq.vq_gemm_small_batch_host_static(dev.fmt, dev.idx, dev.cb, dev.scale, hX, hY, batch)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free0 and torch.cuda.memory_allocated() <= alloc0
