"""Shared test plumbing: draw a synthetic layer, describe it to the oracle and to the library."""
from __future__ import annotations

import numpy as np

import vq_synth
from oracle import vq_oracle as orc

TOL = 1e-3  # |y_gpu - y_ref| <= TOL * sum_k |W_nk x_k| per output element


def oracle_fmt(spec: vq_synth.LayerSpec) -> orc.Fmt:
    return orc.Fmt(spec.N, spec.K, spec.d, spec.b, spec.Br, spec.Bc, spec.int8)


def lib_fmt(spec: vq_synth.LayerSpec):
    import paper_2402_15319_b200 as vq
    return vq.VQFormat(spec.N, spec.K, spec.d, spec.b, spec.Br, spec.Bc,
                       vq.VQ_CB_INT4_G128 if int(spec.int8) == 2 else vq.VQ_CB_INT8_SCALED if spec.int8 else vq.VQ_CB_FP16)


def draw(spec: vq_synth.LayerSpec, seed: int, layer_id: int = 0) -> vq_synth.Layer:
    return vq_synth.make_layer(spec, oracle_fmt(spec).stride, seed, layer_id)


CANARY = 0xA5          # byte pattern of the guard bands
GUARD = 256            # bytes on either side of every output buffer


def guarded(shape, dtype, device, fill=float("nan")):
    """An output tensor with GUARD bytes of a known pattern on both sides: (view, raw buffer)."""
    import torch
    n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
    raw = torch.full((GUARD + n + GUARD,), CANARY, dtype=torch.uint8, device=device)
    view = raw[GUARD:GUARD + n].view(dtype).view(*shape)
    if fill is not None:
        view.fill_(fill)
    return view, raw


def assert_guards_intact(raw, what=""):
    """Nothing wrote before the start or past the end of the buffer."""
    import torch
    lo, hi = raw[:GUARD], raw[-GUARD:]
    assert bool((lo == CANARY).all()) and bool((hi == CANARY).all()), f"{what}: write outside the output buffer"


class DeviceLayer:
    """Device copies of one layer + workspace, made with torch (memory plumbing only).  Outputs are
    allocated with guard bands that are checked after every call."""

    def __init__(self, spec, layer, max_batch=16, device="cuda:0"):
        import torch
        import paper_2402_15319_b200 as vq
        self.spec, self.fmt = spec, lib_fmt(spec)
        self.idx = torch.from_numpy(layer.idx).to(device)
        self.cb = torch.from_numpy(layer.cb).to(device)
        self.scale = None if layer.scale is None else torch.from_numpy(layer.scale).to(device)
        # ticket counters at the start of the workspace must be zero on first use (the kernels leave them zero)
        self.ws = torch.zeros(vq.vq_workspace_bytes(self.fmt, max_batch), dtype=torch.uint8, device=device)
        self.device = device

    def gemm(self, X: np.ndarray, impl=None):
        import torch
        import paper_2402_15319_b200 as vq
        X = np.ascontiguousarray(np.atleast_2d(X))
        batch = X.shape[0]
        dX = torch.from_numpy(X).to(self.device)
        dY, raw = guarded((batch, self.spec.N), torch.float16, self.device)
        if impl is None:
            vq.vq_gemm_small_batch(self.fmt, self.idx, self.cb, self.scale, dX, dY, batch, self.ws)
        elif impl == "gemv":
            assert batch == 1
            vq.vq_gemv(self.fmt, self.idx, self.cb, self.scale, dX, dY, self.ws)
        else:
            vq.vq_gemm_small_batch_impl(self.fmt, self.idx, self.cb, self.scale, dX, dY, batch, self.ws, impl)
        torch.cuda.synchronize()
        assert_guards_intact(raw, f"{self.spec.name} gemm batch {batch} impl {impl}")
        return dY.cpu().numpy()

    def decode(self):
        import torch
        import paper_2402_15319_b200 as vq
        dW, raw = guarded((self.spec.N, self.spec.K), torch.float16, self.device)
        vq.vq_decode_weights(self.fmt, self.idx, self.cb, self.scale, dW)
        torch.cuda.synchronize()
        assert_guards_intact(raw, f"{self.spec.name} decode")
        return dW.cpu().numpy()


def assert_outputs_close(Y_gpu: np.ndarray, Y_ref: np.ndarray, A_ref: np.ndarray, what=""):
    """The acceptance bound: per element |y_gpu - y_ref| <= 1e-3 * sum_k |W x|."""
    assert Y_gpu.shape == Y_ref.shape, (Y_gpu.shape, Y_ref.shape)
    assert np.isfinite(Y_gpu.astype(np.float64)).all(), f"{what}: non-finite output"
    err = np.abs(Y_gpu.astype(np.float64) - Y_ref)
    bound = TOL * A_ref
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} outputs beyond tolerance; worst at {i}: "
                             f"gpu={Y_gpu[i]} ref={Y_ref[i]} err={err[i]:.3e} bound={bound[i]:.3e}")
    return float((err / np.maximum(bound, 1e-300)).max())
