"""GPU parity: the CUDA library, called through the C-ABI, against the CPU oracle on the same
seeded inputs.  Unpack/decode must be bit-exact; GEMV/GEMM outputs must satisfy
|y_gpu - y_ref| <= 1e-3 * sum_k |W_nk x_k| per element."""
import numpy as np
import pytest

import vq_synth
from oracle import vq_oracle as orc
from tests.helpers import DeviceLayer, assert_guards_intact, assert_outputs_close, draw, guarded, lib_fmt, oracle_fmt

pytestmark = pytest.mark.gpu

import paper_2402_15319_b200 as vq  # noqa: E402

IMPLS = [vq.VQ_IMPL_GENERIC, vq.VQ_IMPL_AUTO]
THREADS = orc.hardware_threads() or 8


def _check_layer(spec, seed, batches, impls=IMPLS, decode=True, rows=None, layer_id=0):
    f = oracle_fmt(spec)
    L = draw(spec, seed, layer_id)
    dev = DeviceLayer(spec, L)
    if decode:
        _, W16 = orc.decode(f, L.idx, L.cb, L.scale, exact=False)
        W_gpu = dev.decode().view(np.uint16)
        assert np.array_equal(W_gpu, W16), f"{spec.name}: decode not bit-exact"
    worst = 0.0
    for batch in batches:
        X = vq_synth.make_x(spec, seed + 17, batch, layer_id)
        Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X, rows=rows, threads=8)
        for impl in impls:
            Yg = dev.gemm(X, impl)
            if rows is not None:
                Yg = Yg[:, rows]
            worst = max(worst, assert_outputs_close(Yg, Y, A, f"{spec.name} batch={batch} impl={impl}"))
    return worst


# ---- every (d, b, codebook type) on small ragged shapes --------------------------------------
@pytest.mark.parametrize("int8", [False, True])
@pytest.mark.parametrize("b", range(1, 9))
@pytest.mark.parametrize("d", [1, 2, 4])
def test_all_formats_small(d, b, int8):
    # K/d = 104 indices: not a multiple of 8*anything nice, 13 groups of 8; 37 rows: ragged vs 8/16-row tiles
    spec = vq_synth.LayerSpec(f"small_d{d}b{b}", N=37, K=104 * d, d=d, b=b, Br=1, Bc=52 * d, int8=int8)
    _check_layer(spec, seed=10 * b + d, batches=(1, 3))
    # tall blocks, several block rows, K/d = 9 -> a ragged last group of indices
    spec = vq_synth.LayerSpec(f"tall_d{d}b{b}", N=48, K=9 * d, d=d, b=b, Br=16, Bc=3 * d, int8=int8)
    _check_layer(spec, seed=20 * b + d, batches=(2,))


@pytest.mark.parametrize("batch", range(1, 17))
def test_every_batch(batch):
    spec = vq_synth.LayerSpec("b", N=200, K=512, d=2, b=6, Br=8, Bc=128, int8=False)
    _check_layer(spec, seed=batch, batches=(batch,), decode=False)
    spec = vq_synth.LayerSpec("b8", N=96, K=1024, d=2, b=4, Br=1, Bc=512, int8=True)
    _check_layer(spec, seed=batch + 50, batches=(batch,), decode=False)


def test_degenerate_shapes():
    _check_layer(vq_synth.LayerSpec("one", N=1, K=4, d=4, b=8, Br=1, Bc=4, int8=False), 1, (1, 16))
    _check_layer(vq_synth.LayerSpec("one_idx", N=3, K=1, d=1, b=1, Br=3, Bc=1, int8=True), 2, (1,))
    _check_layer(vq_synth.LayerSpec("wide", N=2, K=16384, d=2, b=5, Br=2, Bc=8192, int8=False), 3, (1, 2))
    _check_layer(vq_synth.LayerSpec("tall", N=5000, K=8, d=2, b=3, Br=1000, Bc=8, int8=True), 4, (1,))


# ---- tile-aligned shapes of the benchmark format families, several tiles + row tails ----------
FAMILY = [
    vq_synth.LayerSpec("fam1", N=272, K=2048, d=2, b=4, Br=1, Bc=1024, int8=False),
    vq_synth.LayerSpec("fam2", N=144, K=4096, d=1, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("fam3", N=384, K=1024, d=2, b=6, Br=128, Bc=128, int8=False),
    vq_synth.LayerSpec("fam3w", N=128, K=11008, d=2, b=6, Br=128, Bc=128, int8=False),
    vq_synth.LayerSpec("fam4", N=512, K=1024, d=4, b=8, Br=256, Bc=512, int8=False, cb_sigma=0.015),
    vq_synth.LayerSpec("fam5", N=208, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True),
]

# further format points of the paper served by the tall-block kernel: int8 codebooks (Sec. 3.2:
# 8-bit codebook entries with a scale per group), 5-bit indices (2.5 bits per dimension), 256-column groups
TALL_BLOCK_EXTRA = [
    vq_synth.LayerSpec("tb_d2b6_i8", N=384, K=1024, d=2, b=6, Br=128, Bc=128, int8=True),
    vq_synth.LayerSpec("tb_d2b6_i8_256", N=256, K=2816, d=2, b=6, Br=256, Bc=256, int8=True),
    vq_synth.LayerSpec("tb_d2b5", N=256, K=1280, d=2, b=5, Br=128, Bc=256, int8=False),
    vq_synth.LayerSpec("tb_d2b5_i8", N=128, K=5632, d=2, b=5, Br=128, Bc=128, int8=True),
    vq_synth.LayerSpec("tb_d4b8_i8", N=512, K=1536, d=4, b=8, Br=256, Bc=512, int8=True),
    # groups of 8192 weights with at most 256 columns (Sec. 4.1): 32 x 256 blocks, one pair of tables per warp
    vq_synth.LayerSpec("wb_d2b6_i8_32x256", N=256, K=2304, d=2, b=6, Br=32, Bc=256, int8=True),
    vq_synth.LayerSpec("wb_d2b6_64x128", N=384, K=1024, d=2, b=6, Br=64, Bc=128, int8=False),
    vq_synth.LayerSpec("wb_d2b5_i8_32x256", N=128, K=4352, d=2, b=5, Br=32, Bc=256, int8=True),
    vq_synth.LayerSpec("wb_d2b5_32x128", N=256, K=768, d=2, b=5, Br=32, Bc=128, int8=False),
    # 4-bit indices with a few rows per block (4 x 256 groups, Sec. 4.1): the row kernel, every lane
    # taking its own rows' block
    vq_synth.LayerSpec("rb_d2b4_4x256_i8", N=212, K=2048, d=2, b=4, Br=4, Bc=256, int8=True),
    vq_synth.LayerSpec("rb_d2b4_4x256", N=64, K=4096, d=2, b=4, Br=4, Bc=256, int8=False),
    vq_synth.LayerSpec("rb_d1b4_4x256_i8", N=132, K=1024, d=1, b=4, Br=4, Bc=256, int8=True),
    vq_synth.LayerSpec("rb_d2b4_128x512", N=256, K=1024, d=2, b=4, Br=128, Bc=512, int8=False),
]


@pytest.mark.parametrize("spec", FAMILY, ids=lambda s: s.name)
def test_benchmark_families_medium(spec):
    _check_layer(spec, seed=77, batches=(1, 2, 4, 8, 16))


# ---- the persistent kernel, forced (AUTO only picks it for large layers and groups) ------------
STREAM_CASES = [
    # per-row 2-D 4-bit (fp16 / int8), 1-D int8, few rows per block; row counts with tails, several slabs
    vq_synth.LayerSpec("st_d2b4", N=272, K=2048, d=2, b=4, Br=1, Bc=1024, int8=False),
    vq_synth.LayerSpec("st_d2b4_i8", N=208, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("st_d2b4_i8_long", N=1000, K=28672, d=2, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("st_d1b4_i8", N=144, K=4096, d=1, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("st_d2b4_4x512", N=212, K=2048, d=2, b=4, Br=4, Bc=512, int8=True),
    vq_synth.LayerSpec("st_d2b4_many", N=5000, K=1024, d=2, b=4, Br=1, Bc=512, int8=False),
    # shared codebooks, 6-bit: 128 x 128 blocks (fp16, int8), 256 x 256, 64 x 128, 32 x 256
    vq_synth.LayerSpec("st_d2b6", N=384, K=1024, d=2, b=6, Br=128, Bc=128, int8=False),
    vq_synth.LayerSpec("st_d2b6_wide", N=128, K=11008, d=2, b=6, Br=128, Bc=128, int8=False),
    vq_synth.LayerSpec("st_d2b6_i8", N=512, K=2816, d=2, b=6, Br=256, Bc=256, int8=True),
    vq_synth.LayerSpec("st_d2b6_64", N=384, K=1024, d=2, b=6, Br=64, Bc=128, int8=False),
    vq_synth.LayerSpec("st_d2b6_32_i8", N=256, K=2304, d=2, b=6, Br=32, Bc=256, int8=True),
    vq_synth.LayerSpec("st_d2b6_many", N=4096, K=512, d=2, b=6, Br=128, Bc=128, int8=False),
]


@pytest.mark.parametrize("spec", STREAM_CASES, ids=lambda s: s.name)
def test_persistent_kernel_forced(spec):
    """Every policy of the persistent kernel against the oracle at every batch class; the same
    workspace serves all batches in turn (its ticket counters must come back to zero each time)."""
    _check_layer(spec, seed=55, batches=(1, 2, 5, 8, 9, 16), impls=[vq.VQ_IMPL_STREAM], decode=False)


def test_persistent_kernel_repeats_bitwise():
    """Slabs shared between CTAs are summed in CTA order whatever order the tickets are drawn in."""
    spec = vq_synth.LayerSpec("st_rep", N=4096, K=8192, d=2, b=4, Br=1, Bc=2048, int8=True)
    dev = DeviceLayer(spec, draw(spec, 9))
    for batch in (1, 16):
        X = vq_synth.make_x(spec, 10, batch)
        first = dev.gemm(X, vq.VQ_IMPL_STREAM).view(np.uint16)
        for _ in range(30):
            assert np.array_equal(dev.gemm(X, vq.VQ_IMPL_STREAM).view(np.uint16), first)


def test_gemv_entry_point_against_oracle():
    """vq_gemv (one token) with device pointers, on a cluster-kernel format and a large per-row one."""
    for spec in (vq_synth.LayerSpec("gv_blk", N=384, K=1024, d=2, b=6, Br=128, Bc=128, int8=False),
                 vq_synth.LayerSpec("gv_row", N=8192, K=2048, d=2, b=4, Br=1, Bc=1024, int8=True),
                 vq_synth.LayerSpec("gv_gen", N=37, K=312, d=1, b=5, Br=1, Bc=156, int8=False)):
        f = oracle_fmt(spec)
        L = draw(spec, 12)
        dev = DeviceLayer(spec, L)
        X = vq_synth.make_x(spec, 13, 1)
        Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X, threads=8)
        assert_outputs_close(dev.gemm(X, "gemv"), Y, A, f"{spec.name} vq_gemv")


GROUPS = [
    # (format template, member rows, K): members of different heights, one with a row tail
    (vq_synth.LayerSpec("g_row", N=0, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True), [2048, 264, 256]),
    (vq_synth.LayerSpec("g_row16", N=0, K=2048, d=2, b=4, Br=1, Bc=1024, int8=False), [300, 1000]),
    (vq_synth.LayerSpec("g_blk", N=0, K=1024, d=2, b=6, Br=128, Bc=128, int8=False), [512, 128, 128, 256]),
    (vq_synth.LayerSpec("g_blk32", N=0, K=1024, d=2, b=6, Br=32, Bc=256, int8=True), [256, 128, 384]),
    (vq_synth.LayerSpec("g_d4b8", N=0, K=1024, d=4, b=8, Br=256, Bc=512, int8=False), [256, 512]),
    (vq_synth.LayerSpec("g_i4cb", N=0, K=1024, d=2, b=6, Br=32, Bc=128, int8=2), [256, 128]),
    (vq_synth.LayerSpec("g_generic", N=0, K=312, d=1, b=5, Br=1, Bc=156, int8=False), [37, 5]),
    # the pair-table kernel over several layers in one launch: ragged member heights (row tails inside the group)
    (vq_synth.LayerSpec("g_pt_d2b5", N=0, K=1280, d=2, b=5, Br=4, Bc=256, int8=True), [212, 64, 36, 100]),
    (vq_synth.LayerSpec("g_pt_d1b2", N=0, K=1024, d=1, b=2, Br=1, Bc=256, int8=True), [33, 200]),
    (vq_synth.LayerSpec("g_pt_d2b8", N=0, K=768, d=2, b=8, Br=256, Bc=256, int8=False), [256, 512]),
    (vq_synth.LayerSpec("g_pt_d4b8", N=0, K=1024, d=4, b=8, Br=128, Bc=256, int8=True), [128, 384]),
    (vq_synth.LayerSpec("g_pt_i4cb", N=0, K=1280, d=2, b=5, Br=4, Bc=256, int8=2), [100, 36, 64]),
]


@pytest.mark.parametrize("tmpl,rows", GROUPS, ids=lambda v: v.name if hasattr(v, "name") else None)
def test_grouped_call_matches_oracle_per_member(tmpl, rows):
    import torch
    for batch in (1, 4, 16):
        specs = [vq_synth.LayerSpec(f"{tmpl.name}.{i}", N=n, K=tmpl.K, d=tmpl.d, b=tmpl.b, Br=tmpl.Br, Bc=tmpl.Bc, int8=tmpl.int8)
                 for i, n in enumerate(rows)]
        layers = [draw(sp, 21, i) for i, sp in enumerate(specs)]
        X = vq_synth.make_x(specs[0], 22, batch)
        total = vq_synth.LayerSpec("sum", N=sum(rows), K=tmpl.K, d=tmpl.d, b=tmpl.b, Br=tmpl.Br, Bc=tmpl.Bc, int8=tmpl.int8)
        fmt = lib_fmt(total)
        ws = torch.zeros(vq.vq_workspace_bytes(fmt, batch), dtype=torch.uint8, device="cuda")
        dX = torch.from_numpy(X).cuda()
        members, outs = [], []
        for sp, L in zip(specs, layers):
            Y, raw = guarded((batch, sp.N), torch.float16, "cuda")
            outs.append((Y, raw))
            members.append((torch.from_numpy(L.idx).cuda(), torch.from_numpy(L.cb).cuda(),
                            None if L.scale is None else torch.from_numpy(L.scale).cuda(), Y, sp.N))
        for _ in range(2):   # twice on the same workspace
            vq.vq_gemm_small_batch_grouped(fmt, members, dX, batch, ws)
        torch.cuda.synchronize()
        for sp, L, (Y, raw) in zip(specs, layers, outs):
            assert_guards_intact(raw, sp.name)
            Yr, A = orc.gemm(oracle_fmt(sp), L.idx, L.cb, L.scale, X, threads=8)
            assert_outputs_close(Y.cpu().numpy(), Yr, A, f"{sp.name} batch {batch}")


@pytest.mark.parametrize("spec", TALL_BLOCK_EXTRA, ids=lambda s: s.name)
def test_tall_block_kernel_extra_formats(spec):
    # tuned kernel only (no fallback), every batch size class, against the oracle
    _check_layer(spec, seed=91, batches=(1, 3, 8, 16), impls=[vq.VQ_IMPL_TUNED, vq.VQ_IMPL_GENERIC], decode=True)


# the rows of the paper's table of VQ configurations (App. on VQ configurations) that no other tuned family
# takes, and formats around them: small codebook blocks, 5-bit and 8-bit 2-D indices, 1-D indices looked up
# two at a time; ragged row counts, K parts that do not divide among the warps, block columns of 64..256
PAIR_TABLE_CASES = [
    vq_synth.LayerSpec("pt_d1b2_1x256_i8", N=200, K=1024, d=1, b=2, Br=1, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d1b2_1x128_i8", N=48, K=1152, d=1, b=2, Br=1, Bc=128, int8=True),
    vq_synth.LayerSpec("pt_d2b5_4x256_i8", N=212, K=2048, d=2, b=5, Br=4, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d2b5_2x256_i8", N=130, K=1280, d=2, b=5, Br=2, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d2b5_1x256", N=77, K=768, d=2, b=5, Br=1, Bc=256, int8=False),
    vq_synth.LayerSpec("pt_d1b3_32x256_i8", N=96, K=2304, d=1, b=3, Br=32, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d2b8_256x256_i8", N=512, K=1024, d=2, b=8, Br=256, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d2b7_16x64", N=64, K=4480, d=2, b=7, Br=16, Bc=64, int8=False),
    vq_synth.LayerSpec("pt_d2b3_8x128_i8", N=72, K=640, d=2, b=3, Br=8, Bc=128, int8=True),
    vq_synth.LayerSpec("pt_d2b6_4x256", N=100, K=11008, d=2, b=6, Br=4, Bc=256, int8=False),
    vq_synth.LayerSpec("pt_d1b4_8x64", N=40, K=704, d=1, b=4, Br=8, Bc=64, int8=False),
    vq_synth.LayerSpec("pt_d2b1_1x64_i8", N=33, K=320, d=2, b=1, Br=1, Bc=64, int8=True),
    vq_synth.LayerSpec("pt_d1b1_2x192", N=34, K=1344, d=1, b=1, Br=2, Bc=192, int8=False),
    vq_synth.LayerSpec("pt_d2b2_48x64_i8", N=96, K=64, d=2, b=2, Br=48, Bc=64, int8=True),
    # 4-D, 8-bit indices with blocks of fewer than 256 rows (128 x 256: the 2.25-bit 4-D row of the paper's
    # table): one byte looks up four weights
    vq_synth.LayerSpec("pt_d4b8_128x256_i8", N=256, K=1024, d=4, b=8, Br=128, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_d4b8_16x64", N=48, K=704, d=4, b=8, Br=16, Bc=64, int8=False, cb_sigma=0.015),
    vq_synth.LayerSpec("pt_d4b8_8x128_i8", N=40, K=640, d=4, b=8, Br=8, Bc=128, int8=True),
    # degenerate shapes: one row, one step, one block spanning K, the largest table set a warp may hold
    vq_synth.LayerSpec("pt_one_row_one_step", N=1, K=64, d=2, b=5, Br=1, Bc=64, int8=True),
    vq_synth.LayerSpec("pt_17_rows", N=17, K=128, d=1, b=3, Br=1, Bc=64, int8=False),
    vq_synth.LayerSpec("pt_block_spans_k", N=5, K=4096, d=2, b=6, Br=1, Bc=4096, int8=True),
]


@pytest.mark.parametrize("spec", PAIR_TABLE_CASES, ids=lambda s: s.name)
def test_pair_table_kernel_formats(spec):
    # tuned kernel only (no fallback), every batch size class, against the oracle
    _check_layer(spec, seed=113, batches=(1, 3, 8, 9, 16), impls=[vq.VQ_IMPL_TUNED, vq.VQ_IMPL_AUTO], decode=False)


@pytest.mark.parametrize("spec", [
    vq_synth.LayerSpec("pt_full_d2b5_4x256_i8", N=4096, K=4096, d=2, b=5, Br=4, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_full_d1b2_1x256_i8", N=14336, K=4096, d=1, b=2, Br=1, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_full_d2b8_256x256_i8", N=4096, K=14336, d=2, b=8, Br=256, Bc=256, int8=True),
    vq_synth.LayerSpec("pt_full_d4b8_128x256_i8", N=14336, K=4096, d=4, b=8, Br=128, Bc=256, int8=True),
], ids=lambda s: s.name)
def test_pair_table_kernel_layer_sizes(spec):
    """Llama-3-8B-sized layers in the paper's small-block configurations: sampled output rows against the
    oracle in the launch shapes that full-size layers get (fewer warps per CTA as the row count grows)."""
    rows = _sample_rows(spec.N, spec.Br, n=128, seed=5)
    _check_layer(spec, seed=7, batches=(1, 8, 16), impls=[vq.VQ_IMPL_TUNED], decode=False, rows=rows)


@pytest.mark.parametrize("cfg", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "llama3_8b", "llama3_8b_int4cb", "llama3_8b_d2b5_4x256"])
def test_tuned_kernels_cover_every_benchmark_format(cfg):
    """VQ_IMPL_TUNED never falls back: it must run (not VQ_ERR_UNSUPPORTED) on every layer shape of
    the five configurations, at every batch of the configuration (row count cut to two tiles)."""
    conf = vq_synth.CONFIGS[cfg]
    seen = set()
    for spec in conf["layers"]:
        if spec.K in seen:
            continue
        seen.add(spec.K)
        small = vq_synth.LayerSpec(spec.name + ".cut", N=2 * max(spec.Br, 128), K=spec.K, d=spec.d, b=spec.b, Br=spec.Br,
                                   Bc=spec.Bc, int8=spec.int8, cb_sigma=spec.cb_sigma)
        _check_layer(small, seed=conf["seed"], batches=conf["batches"], impls=[vq.VQ_IMPL_TUNED], decode=False)


def _sweep_specs():
    """Seeded draw of valid formats inside and around what the tuned kernels cover: block shapes,
    index widths, codebook types, row counts with tails, column counts with short last chunks."""
    rng = np.random.default_rng(20240229)
    specs = []
    for i in range(28):
        fam = i % 4
        if fam == 0:      # tall blocks, 2-D, 5/6 bits (shared or warp-private tables)
            Br = int(rng.choice([32, 64, 128, 256])); Bc = int(rng.choice([128, 256, 512]))
            N = Br * int(rng.integers(1, 4)) if Br >= 128 else 128 * int(rng.integers(1, 3))
            K = Bc * int(rng.integers(1, 12)); K += (-K) % 256
            K = K if K % Bc == 0 else Bc * (K // Bc + 1)
            specs.append(vq_synth.LayerSpec(f"sw{i}", N, K, 2, int(rng.choice([5, 6])), Br, Bc, bool(rng.integers(2))))
        elif fam == 1:    # 4-D 8-bit, 256-row blocks
            Bc = int(rng.choice([256, 512, 1024]))
            specs.append(vq_synth.LayerSpec(f"sw{i}", 256 * int(rng.integers(1, 3)), Bc * int(rng.integers(1, 7)), 4, 8, 256, Bc,
                                            bool(rng.integers(2)), cb_sigma=0.015))
        elif fam == 2:    # 4-bit, few rows per block (row kernel)
            d = int(rng.choice([1, 2])); Br = int(rng.choice([1, 2, 4, 8])); Bc = int(rng.choice([256, 512, 1024, 2048]))
            int8 = True if d == 1 else bool(rng.integers(2))
            specs.append(vq_synth.LayerSpec(f"sw{i}", Br * int(rng.integers(3, 60)), Bc * int(rng.integers(1, 5)), d, 4, Br, Bc, int8))
        else:             # anything valid: generic kernels (and the tuned decode / E-step where they apply)
            d = int(rng.choice([1, 2, 4])); b = int(rng.integers(1, 9)); Br = int(rng.choice([1, 3, 16, 32]))
            Bc = d * 8 * int(rng.choice([1, 4, 16, 32]))
            specs.append(vq_synth.LayerSpec(f"sw{i}", Br * int(rng.integers(1, 9)), Bc * int(rng.integers(1, 6)), d, b, Br, Bc,
                                            bool(rng.integers(2))))
    return specs


@pytest.mark.parametrize("spec", _sweep_specs(), ids=lambda s: f"{s.name}_{s.N}x{s.K}_d{s.d}b{s.b}_{s.Br}x{s.Bc}_{'i8' if s.int8 else 'f16'}")
def test_randomized_format_sweep(spec):
    batch = 1 + (spec.N + spec.K) % 16
    _check_layer(spec, seed=spec.N + spec.K, batches=(1, batch))
    # E-step on the same format where the kernel covers it: byte-exact stream
    import torch
    f = oracle_fmt(spec)
    tables = (32 // spec.Br if spec.Br < 32 else 1) * max(1, 256 * spec.d // spec.Bc) * (1 << spec.b) * spec.d * 4   # bytes per tile
    if ((spec.K // spec.d) % 8 == 0 and spec.Bc % (8 * spec.d) == 0 and (spec.Bc & (spec.Bc - 1)) == 0
            and (32 % spec.Br == 0 or spec.Br % 32 == 0) and tables <= 96 * 1024):
        L = draw(spec, spec.N + spec.K)
        W = (0.05 * vq_synth.normal(spec.N, 40, spec.N * spec.K)).astype(np.float16).reshape(spec.N, spec.K)
        dev = DeviceLayer(spec, L)
        d_idx = torch.zeros((spec.N, f.stride), dtype=torch.uint8, device="cuda")
        vq.vq_assign_indices(dev.fmt, torch.from_numpy(W).cuda(), dev.cb, dev.scale, None, d_idx)
        torch.cuda.synchronize()
        assert np.array_equal(d_idx.cpu().numpy(), orc.pack(f, orc.assign(f, W, L.cb, L.scale)))


@pytest.mark.parametrize("spec,batch", [
    (vq_synth.LayerSpec("rep_tall", N=1024, K=4096, d=2, b=6, Br=128, Bc=128, int8=False), 3),
    (vq_synth.LayerSpec("rep_row", N=2048, K=8192, d=2, b=4, Br=1, Bc=2048, int8=True), 16),
    (vq_synth.LayerSpec("rep_d4", N=512, K=5120, d=4, b=8, Br=256, Bc=512, int8=False), 8),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_repeated_calls_are_bitwise_identical(spec, batch):
    """The K-part reduction adds in a fixed order whatever order the partial sums arrive in: sixty
    launches on the same inputs give the same bits (cluster split, remote stores, streamed activations)."""
    L = draw(spec, 7)
    dev = DeviceLayer(spec, L)
    X = vq_synth.make_x(spec, 8, batch)
    first = dev.gemm(X, vq.VQ_IMPL_TUNED).view(np.uint16)
    for _ in range(60):
        assert np.array_equal(dev.gemm(X, vq.VQ_IMPL_TUNED).view(np.uint16), first)


def test_no_wait_ran_out_inside_a_kernel():
    # bounded waits on asynchronous copies never expired in anything this process has run so far
    import torch
    torch.cuda.synchronize()
    assert vq.vq_device_wait_failures() == 0


# ---- properties that hold at any size ---------------------------------------------------------
def test_unit_vectors_return_decoded_columns():
    spec = vq_synth.LayerSpec("unit", N=256, K=256, d=2, b=6, Br=128, Bc=128, int8=False)
    L = draw(spec, 5)
    dev = DeviceLayer(spec, L)
    W = dev.decode()
    for k0 in (0, 1, 127, 128, 255):
        X = np.zeros((1, spec.K), np.float16)
        X[0, k0] = 1.0
        for impl in IMPLS:
            assert np.array_equal(dev.gemm(X, impl)[0].view(np.uint16), W[:, k0].view(np.uint16))


def test_int8_unit_scale_integer_inputs_exact_and_deterministic():
    spec = vq_synth.LayerSpec("int", N=64, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True)
    L = draw(spec, 6)
    L.scale[:] = 1.0
    rng = np.random.default_rng(0)
    X = rng.integers(-2, 3, size=(2, spec.K)).astype(np.float16)
    Y, _ = orc.gemm(oracle_fmt(spec), L.idx, L.cb, L.scale, X)
    assert np.abs(Y).max() < 60000  # partial sums are integers < 2^24: exact in fp32, finite in fp16
    dev = DeviceLayer(spec, L)
    for impl in IMPLS:
        Yg = dev.gemm(X, impl)
        assert np.array_equal(Yg.astype(np.float64), Y.astype(np.float16).astype(np.float64))
        assert np.array_equal(dev.gemm(X, impl).view(np.uint16), Yg.view(np.uint16))  # run-to-run identical


def test_zero_codebook_gives_exact_zero():
    spec = vq_synth.LayerSpec("zero", N=64, K=2048, d=2, b=4, Br=1, Bc=1024, int8=False)
    L = draw(spec, 8)
    L.cb[:] = 0
    dev = DeviceLayer(spec, L)
    X = vq_synth.make_x(spec, 1, 4)
    for impl in IMPLS:
        assert not dev.gemm(X, impl).any()


# ---- the five benchmark configurations at full size -------------------------------------------
def _sample_rows(N, Br, n=192, seed=0):
    rng = np.random.default_rng(seed)
    rows = set(rng.integers(0, N, size=n).tolist()) | {0, 1, N - 1, N - 2, min(N - 1, Br), max(0, N - Br - 1)}
    return np.array(sorted(rows), np.int32)


def _decode_slab_check(spec, L, dev_W, block_row):
    """Bit-exact decode of one block-row (Br rows) of a full-size layer."""
    r0 = block_row * spec.Br
    bpr = spec.K // spec.Bc
    sub = orc.Fmt(spec.Br, spec.K, spec.d, spec.b, spec.Br, spec.Bc, spec.int8)
    cb = L.cb[block_row * bpr:(block_row + 1) * bpr]
    sc = None if L.scale is None else L.scale[block_row * bpr:(block_row + 1) * bpr]
    _, W16 = orc.decode(sub, L.idx[r0:r0 + spec.Br], cb, sc, exact=False)
    assert np.array_equal(dev_W[r0:r0 + spec.Br].view(np.uint16), W16), f"{spec.name}: decode rows {r0}.."


@pytest.mark.parametrize("cfg", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "llama3_8b", "llama3_8b_int4cb", "llama3_8b_d2b5_4x256"])
def test_benchmark_configs_full_size(cfg):
    conf = vq_synth.CONFIGS[cfg]
    seen = set()
    for layer_id, spec in enumerate(conf["layers"]):
        if (spec.N, spec.K) in seen:       # q/k/v/o share a shape: one of each shape is enough
            continue
        seen.add((spec.N, spec.K))
        f = oracle_fmt(spec)
        L = draw(spec, conf["seed"], layer_id)
        dev = DeviceLayer(spec, L)
        # every element of the decoded layer
        W = dev.decode()
        _, W16 = orc.decode(f, L.idx, L.cb, L.scale, exact=False)
        assert np.array_equal(W.view(np.uint16), W16), f"{spec.name}: decode not bit-exact"
        del W, W16
        rows = _sample_rows(spec.N, spec.Br, seed=layer_id)
        for batch in conf["batches"]:
            X = vq_synth.make_x(spec, conf["seed"], batch, layer_id)
            if batch == conf["batches"][0]:
                # every output row of the layer at the configuration's first batch size
                Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X, threads=THREADS)
                assert_outputs_close(dev.gemm(X), Y, A, f"{spec.name} batch={batch} all rows")
                Yg2 = dev.gemm(X, vq.VQ_IMPL_GENERIC)
                assert_outputs_close(Yg2[:, rows], Y[:, rows], A[:, rows], f"{spec.name} generic")
            else:
                Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X, rows=rows, threads=THREADS)
                Yg = dev.gemm(X)
                assert np.isfinite(Yg.astype(np.float64)).all()
                assert_outputs_close(Yg[:, rows], Y, A, f"{spec.name} batch={batch}")


@pytest.mark.parametrize("cfg,names", [("cfg5", ("q", "k", "v")), ("cfg5", ("gate", "up")),
                                       ("cfg3", ("q", "k", "v")), ("cfg3", ("gate", "up")),
                                       ("llama3_8b_d2b5_4x256", ("q", "k", "v")), ("llama3_8b_d2b5_4x256", ("gate", "up"))],
                         ids=lambda v: v if isinstance(v, str) else "+".join(v))
def test_benchmark_groups_full_size(cfg, names):
    """The grouped calls bench.py times, at full size and in its launch configuration (one launch per
    group): every output row of every member at the configuration's first batch, sampled rows at the
    others; twice on one workspace."""
    import torch
    conf = vq_synth.CONFIGS[cfg]
    ids = [i for i, sp in enumerate(conf["layers"]) if sp.name.split(".")[-1] in names]
    specs = [conf["layers"][i] for i in ids]
    assert len(specs) == len(names)
    layers = [draw(sp, conf["seed"], i) for sp, i in zip(specs, ids)]
    t = specs[0]
    total = vq_synth.LayerSpec("sum", N=sum(sp.N for sp in specs), K=t.K, d=t.d, b=t.b, Br=t.Br, Bc=t.Bc, int8=t.int8)
    fmt = lib_fmt(total)
    dev = [(torch.from_numpy(L.idx).cuda(), torch.from_numpy(L.cb).cuda(), None if L.scale is None else torch.from_numpy(L.scale).cuda())
           for L in layers]
    batches = conf["batches"] if cfg != "cfg5" else (1, 4, 8, 16)
    for batch in batches:
        assert vq.vq_grouped_kernel_launches(fmt, len(specs), batch) == 1
        X = vq_synth.make_x(specs[0], conf["seed"], batch, ids[0])
        dX = torch.from_numpy(X).cuda()
        ws = torch.zeros(vq.vq_workspace_bytes(fmt, batch), dtype=torch.uint8, device="cuda")
        outs = [guarded((batch, sp.N), torch.float16, "cuda") for sp in specs]
        members = [(d[0], d[1], d[2], o[0], sp.N) for d, o, sp in zip(dev, outs, specs)]
        for _ in range(2):
            vq.vq_gemm_small_batch_grouped(fmt, members, dX, batch, ws)
        torch.cuda.synchronize()
        assert vq.vq_device_wait_failures() == 0
        for sp, L, (Y, raw), lid in zip(specs, layers, outs, ids):
            assert_guards_intact(raw, sp.name)
            Yg = Y.cpu().numpy()
            assert np.isfinite(Yg.astype(np.float64)).all()
            if batch == batches[0]:
                Yr, A = orc.gemm(oracle_fmt(sp), L.idx, L.cb, L.scale, X, threads=THREADS)
                assert_outputs_close(Yg, Yr, A, f"{sp.name} grouped batch={batch} all rows")
            else:
                rows = _sample_rows(sp.N, sp.Br, seed=lid)
                Yr, A = orc.gemm(oracle_fmt(sp), L.idx, L.cb, L.scale, X, rows=rows, threads=THREADS)
                assert_outputs_close(Yg[:, rows], Yr, A, f"{sp.name} grouped batch={batch}")


# ---- INT4 g128 yard-stick ---------------------------------------------------------------------
@pytest.mark.parametrize("N,K", [(100, 256), (64, 4096), (37, 11008 - 11008 % 128)])
def test_int4g128(N, K):
    import torch
    q, s = vq_synth.make_int4g128(N, K, seed=3)
    spec = vq_synth.LayerSpec("i4", N, K, 1, 4, 1, 128, True)
    for batch in (1, 5, 16):
        X = vq_synth.make_x(spec, 9, batch)
        Y, A = orc.int4g128_gemm(q, s, X, threads=4)
        dq, ds, dX = (torch.from_numpy(a).cuda() for a in (q, s, X))
        dY = torch.full((batch, N), float("nan"), dtype=torch.float16, device="cuda")
        ws = torch.zeros(vq.vq_int4g128_workspace_bytes(N, batch), dtype=torch.uint8, device="cuda")
        vq.vq_int4g128_gemm_small_batch(N, K, dq, ds, dX, dY, batch, ws)
        torch.cuda.synchronize()
        assert_outputs_close(dY.cpu().numpy(), Y, A, f"int4 {N}x{K} b{batch}")


@pytest.mark.parametrize("N,K", [(37, 256), (300, 1408)])
def test_unpack_uniform_bit_exact(N, K):
    """App. B yard-sticks: fp16 copy, int8 with a row scale, int4 g128; every output bit against the oracle."""
    import torch
    q4, s4 = vq_synth.make_int4g128(N, K, seed=11)
    rng_bytes = vq_synth.random_bytes(12, 1, N * K).reshape(N, K)
    q8 = rng_bytes.view(np.int8)
    s8 = (0.001 + 0.003 * vq_synth.uniform01(12, 2, N)).astype(np.float16)
    w16 = vq_synth.normal(12, 3, N * K).astype(np.float16).reshape(N, K)
    cases = [(vq.VQ_UNPACK_FP16, "fp16", w16, None), (vq.VQ_UNPACK_INT8_ROW, "int8row", q8, s8),
             (vq.VQ_UNPACK_INT4_G128, "int4g128", q4, s4)]
    for kind, name, src, scale in cases:
        want = orc.unpack_uniform(name, src, scale)
        d_src = torch.from_numpy(np.ascontiguousarray(src)).cuda()
        d_scale = None if scale is None else torch.from_numpy(np.ascontiguousarray(scale)).cuda()
        d_W = torch.full((N, K), float("nan"), dtype=torch.float16, device="cuda")
        vq.vq_unpack_uniform(kind, N, K, d_src, d_scale, d_W)
        torch.cuda.synchronize()
        assert np.array_equal(d_W.cpu().numpy().view(np.uint16), want.view(np.uint16)), name
    with pytest.raises(vq.VQError):
        vq.vq_unpack_uniform(7, N, K, d_src, d_scale, d_W)           # unknown kind
    with pytest.raises(vq.VQError):
        vq.vq_unpack_uniform(vq.VQ_UNPACK_INT4_G128, N, K + 64, d_src, d_scale, d_W)   # K % 128


ASSIGN_CASES = [
    vq_synth.LayerSpec("as_d2b6", N=200, K=1024, d=2, b=6, Br=8, Bc=128, int8=False),
    vq_synth.LayerSpec("as_d2b6_i8_32x256", N=96, K=2304, d=2, b=6, Br=32, Bc=256, int8=True),
    vq_synth.LayerSpec("as_d1b3_1x256", N=37, K=768, d=1, b=3, Br=1, Bc=256, int8=False),
    vq_synth.LayerSpec("as_d4b8", N=256, K=1024, d=4, b=8, Br=256, Bc=512, int8=False, cb_sigma=0.015),
    vq_synth.LayerSpec("as_d2b4_i8_rows", N=130, K=4096, d=2, b=4, Br=1, Bc=2048, int8=True),
    vq_synth.LayerSpec("as_d2b5", N=64, K=1280, d=2, b=5, Br=64, Bc=256, int8=False),
]


@pytest.mark.parametrize("weighted", [False, True])
@pytest.mark.parametrize("spec", ASSIGN_CASES, ids=lambda s: s.name)
def test_assign_indices_bit_exact(spec, weighted):
    """E-step (Eq. 5): the packed index stream the library writes equals pack(assign) of the oracle,
    byte for byte (padding included), and re-decoding it gives the oracle's quantized matrix."""
    import torch
    f = oracle_fmt(spec)
    L = draw(spec, 31)
    sigma = 0.02 if not spec.int8 else 0.1
    W = (sigma * vq_synth.normal(31, 40, spec.N * spec.K)).astype(np.float16).reshape(spec.N, spec.K)
    h = (0.25 + 2.0 * vq_synth.uniform01(31, 41, spec.K)).astype(np.float32) if weighted else None
    want = orc.pack(f, orc.assign(f, W, L.cb, L.scale, h))
    dev = DeviceLayer(spec, L)
    d_W = torch.from_numpy(W).cuda()
    d_h = None if h is None else torch.from_numpy(h).cuda()
    d_idx, raw_idx = guarded((spec.N, f.stride), torch.uint8, "cuda", fill=None)
    d_idx.fill_(0x5A)
    for _ in range(2):
        vq.vq_assign_indices(dev.fmt, d_W, dev.cb, dev.scale, d_h, d_idx)
    torch.cuda.synchronize()
    assert_guards_intact(raw_idx, f"{spec.name} assign")
    got = d_idx.cpu().numpy()
    assert np.array_equal(got, want), f"{spec.name}: {np.count_nonzero(got != want)} bytes differ"
    # the stream feeds the decode path: quantize -> decode is the oracle's Q(W); SQNR is finite and positive
    dev.idx = d_idx
    Q = dev.decode()
    _, Q16 = orc.decode(f, want, L.cb, L.scale, exact=False)
    assert np.array_equal(Q.view(np.uint16), Q16)
    assert orc.sqnr_db(W, Q) > 0.0


def test_assign_indices_rejects_what_it_does_not_cover():
    import torch
    spec = vq_synth.LayerSpec("as_bad", N=8, K=24, d=2, b=3, Br=1, Bc=12, int8=False)   # 12 indices per row
    L = draw(spec, 1)
    dev = DeviceLayer(spec, L)
    d_W = torch.zeros((8, 24), dtype=torch.float16, device="cuda")
    with pytest.raises(vq.VQError):
        vq.vq_assign_indices(dev.fmt, d_W, dev.cb, dev.scale, None, dev.idx)


INT4_CODEBOOK_CASES = [
    # (layer, whether a tuned kernel takes it: the pair-table kernel does when blocks have 1/2/4/8 or a multiple
    # of 16 rows and block columns are multiples of 64)
    (vq_synth.LayerSpec("i4cb_d2b3", N=64, K=1024, d=2, b=3, Br=32, Bc=256, int8=2), True),
    (vq_synth.LayerSpec("i4cb_d2b6", N=37, K=256, d=2, b=6, Br=37, Bc=128, int8=2), False),
    (vq_synth.LayerSpec("i4cb_d1b4", N=20, K=384, d=1, b=4, Br=4, Bc=96, int8=2), False),
    (vq_synth.LayerSpec("i4cb_d4b8", N=16, K=1280, d=4, b=8, Br=16, Bc=640, int8=2), True),
    (vq_synth.LayerSpec("i4cb_d4b8_tile", N=96, K=2560, d=4, b=8, Br=32, Bc=512, int8=2), True),   # tile decode kernel
    (vq_synth.LayerSpec("i4cb_d1b4_tile", N=40, K=512, d=1, b=4, Br=8, Bc=128, int8=2), True),
    (vq_synth.LayerSpec("i4cb_d2b5_4x256", N=212, K=1280, d=2, b=5, Br=4, Bc=256, int8=2), True),
    (vq_synth.LayerSpec("i4cb_d1b2_1x128", N=50, K=1152, d=1, b=2, Br=1, Bc=128, int8=2), True),
    (vq_synth.LayerSpec("i4cb_d1b1_2x64", N=34, K=384, d=1, b=1, Br=2, Bc=64, int8=2), True),
]


@pytest.mark.parametrize("spec,tuned", INT4_CODEBOOK_CASES, ids=lambda v: v.name if hasattr(v, "name") else None)
def test_int4_codebooks_with_group_scales(spec, tuned):
    """INT4 codebooks decoded with a scale per row and group of 128 columns (Sec. 4.2): bit-exact
    decode, mat-vec within the tolerance through the format-generic kernel and through whatever the
    library picks; VQ_IMPL_TUNED runs the pair-table kernel (entries in the tables as exact fp16 integers,
    every looked-up pair multiplied by its row-group scale) on the shapes it takes and refuses the others."""
    _check_layer(spec, seed=55, batches=(1, 5, 16), impls=[vq.VQ_IMPL_GENERIC, vq.VQ_IMPL_AUTO])
    if tuned:
        _check_layer(spec, seed=56, batches=(1, 8, 9), impls=[vq.VQ_IMPL_TUNED], decode=False)
        return
    L = draw(spec, 55)
    dev = DeviceLayer(spec, L)
    with pytest.raises(vq.VQError) as err:
        dev.gemm(vq_synth.make_x(spec, 1, 1), vq.VQ_IMPL_TUNED)
    assert err.value.code == 7


INT4_CODEBOOK_TUNED = [
    # 2-D, 3 bits per dimension, blocks of 4096 weights: the setting of the paper's INT4-codebook table (Sec. 4.2)
    vq_synth.LayerSpec("i4cb_tb_d2b6_32x128", N=256, K=1024, d=2, b=6, Br=32, Bc=128, int8=2),
    vq_synth.LayerSpec("i4cb_tb_d2b6_128x128", N=384, K=2816, d=2, b=6, Br=128, Bc=128, int8=2),
    vq_synth.LayerSpec("i4cb_tb_d2b5_64x256", N=128, K=1280, d=2, b=5, Br=64, Bc=256, int8=2),
    vq_synth.LayerSpec("i4cb_tb_d2b5_256x128", N=256, K=768, d=2, b=5, Br=256, Bc=128, int8=2),
]


@pytest.mark.parametrize("spec", INT4_CODEBOOK_TUNED, ids=lambda s: s.name)
def test_int4_codebooks_in_the_tall_block_kernel(spec):
    """The tuned shared-codebook kernels with INT4 codebooks (Sec. 4.2): entries enter the look-up tables
    as exact fp16 integers, every looked-up pair is multiplied by the fp16 scale of its row and group of
    128 columns; no fallback (VQ_IMPL_TUNED), every batch class, against the oracle."""
    _check_layer(spec, seed=77, batches=(1, 3, 8, 16), impls=[vq.VQ_IMPL_TUNED, vq.VQ_IMPL_AUTO, vq.VQ_IMPL_GENERIC], decode=True)


# ---- block-wise normalisation applied at decode ---------------------------------------------------------
NORM_CASES = [
    # (layer, columns per sub-row): the paper's sub-row sizes 16 / 32 / 64 and others, every codebook type,
    # every d, ragged index groups, an odd number of sub-rows per row (a half-used last code byte)
    (vq_synth.LayerSpec("nm_d2b6_i8", N=96, K=768, d=2, b=6, Br=32, Bc=256, int8=True), 32),
    (vq_synth.LayerSpec("nm_d2b5_4x256_i8", N=52, K=1280, d=2, b=5, Br=4, Bc=256, int8=True), 64),
    (vq_synth.LayerSpec("nm_d1b3_f16", N=37, K=208, d=1, b=3, Br=1, Bc=16, int8=False), 16),
    (vq_synth.LayerSpec("nm_d4b8_f16", N=64, K=1536, d=4, b=8, Br=16, Bc=512, int8=False, cb_sigma=0.015), 16),
    (vq_synth.LayerSpec("nm_d2b4_row_i8", N=40, K=2048, d=2, b=4, Br=1, Bc=2048, int8=True), 2048),
    (vq_synth.LayerSpec("nm_d2b3_i4cb", N=64, K=1024, d=2, b=3, Br=32, Bc=256, int8=2), 32),
    (vq_synth.LayerSpec("nm_d2b7_odd", N=9, K=36, d=2, b=7, Br=3, Bc=12, int8=False), 4),
]


@pytest.mark.parametrize("spec,nbc", NORM_CASES, ids=lambda v: v.name if hasattr(v, "name") else None)
def test_normalized_decode_and_gemm(spec, nbc):
    """vq_decode_weights_normalized bit-exact and vq_gemm_small_batch_normalized within the tolerance, against
    the oracle's decoded value times the scale selected by the sub-row's 4-bit code."""
    import torch
    f = oracle_fmt(spec)
    L = draw(spec, 71)
    codes, lut = vq_synth.make_norm(spec, nbc, 72)
    dev = DeviceLayer(spec, L)
    row_bytes, codes_bytes, lut_bytes = vq.vq_norm_info(dev.fmt, nbc)
    assert codes.shape == (spec.N, row_bytes) and codes.nbytes == codes_bytes and lut.nbytes == lut_bytes
    d_codes, d_lut = torch.from_numpy(codes).cuda(), torch.from_numpy(lut).cuda()
    dW, raw = guarded((spec.N, spec.K), torch.float16, "cuda")
    vq.vq_decode_weights_normalized(dev.fmt, dev.idx, dev.cb, dev.scale, d_codes, d_lut, nbc, dW)
    torch.cuda.synchronize()
    assert_guards_intact(raw, spec.name)
    _, W16 = orc.normalized_decode(f, L.idx, L.cb, L.scale, codes, lut, nbc)
    assert np.array_equal(dW.cpu().numpy().view(np.uint16), W16), f"{spec.name}: normalised decode not bit-exact"
    for batch in (1, 3, 8, 16):
        X = vq_synth.make_x(spec, 73, batch)
        dY, rawy = guarded((batch, spec.N), torch.float16, "cuda")
        vq.vq_gemm_small_batch_normalized(dev.fmt, dev.idx, dev.cb, dev.scale, d_codes, d_lut, nbc, torch.from_numpy(X).cuda(), dY, batch)
        torch.cuda.synchronize()
        assert_guards_intact(rawy, spec.name)
        Y, A = orc.normalized_gemm(f, L.idx, L.cb, L.scale, codes, lut, nbc, X)
        assert_outputs_close(dY.cpu().numpy(), Y, A, f"{spec.name} normalised batch={batch}")


def test_normalized_gemm_layer_size():
    """A 2048 x 4096 layer in the deployed 2-D 6-bit format with 32-column sub-rows (the pair-table kernel
    with the normalisation multiply, in the launch shape a layer of that size gets): every output row."""
    import torch
    spec = vq_synth.LayerSpec("nm_layer", N=2048, K=4096, d=2, b=6, Br=32, Bc=256, int8=True)
    f = oracle_fmt(spec)
    L = draw(spec, 81)
    codes, lut = vq_synth.make_norm(spec, 32, 82)
    dev = DeviceLayer(spec, L)
    d_codes, d_lut = torch.from_numpy(codes).cuda(), torch.from_numpy(lut).cuda()
    for batch in (1, 9):
        X = vq_synth.make_x(spec, 83, batch)
        dY, rawy = guarded((batch, spec.N), torch.float16, "cuda")
        vq.vq_gemm_small_batch_normalized(dev.fmt, dev.idx, dev.cb, dev.scale, d_codes, d_lut, 32, torch.from_numpy(X).cuda(), dY, batch)
        torch.cuda.synchronize()
        assert_guards_intact(rawy, spec.name)
        Y, A = orc.normalized_gemm(f, L.idx, L.cb, L.scale, codes, lut, 32, X)
        assert_outputs_close(dY.cpu().numpy(), Y, A, f"{spec.name} batch={batch}")


def test_normalized_with_unit_table_equals_plain_entry_points():
    """A table of ones switches the normalisation off: the decode equals vq_decode_weights bit for bit."""
    import torch
    spec = vq_synth.LayerSpec("nm_unit", N=128, K=512, d=2, b=6, Br=128, Bc=128, int8=False)
    L = draw(spec, 5)
    dev = DeviceLayer(spec, L)
    codes, _ = vq_synth.make_norm(spec, 32, 6)
    ones = torch.ones((spec.n_blocks, 16), dtype=torch.float16, device="cuda")
    dW = torch.empty((spec.N, spec.K), dtype=torch.float16, device="cuda")
    vq.vq_decode_weights_normalized(dev.fmt, dev.idx, dev.cb, dev.scale, torch.from_numpy(codes).cuda(), ones, 32, dW)
    torch.cuda.synchronize()
    assert np.array_equal(dW.cpu().numpy().view(np.uint16), dev.decode().view(np.uint16))


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned", "pageable"])
def test_grouped_host_buffer_entry_point(pinned):
    """vq_gemm_small_batch_grouped_host: activations from host memory once for the group, every member's
    result in its own host buffer; pinned buffers (direct path) and pageable ones (copies) against the
    oracle, and bit-identical to the device-pointer grouped call."""
    import torch
    rows = [512, 136, 128]
    tmpl = dict(K=4096, d=2, b=4, Br=1, Bc=2048, int8=True)
    specs = [vq_synth.LayerSpec(f"gh{i}", N=n, **tmpl) for i, n in enumerate(rows)]
    layers = [draw(sp, 61, i) for i, sp in enumerate(specs)]
    fmt = lib_fmt(vq_synth.LayerSpec("gh", N=sum(rows), **tmpl))
    dev = [(torch.from_numpy(L.idx).cuda(), torch.from_numpy(L.cb).cuda(), torch.from_numpy(L.scale).cuda()) for L in layers]
    for batch in (1, 6):
        X = vq_synth.make_x(specs[0], 62, batch)
        hX = torch.from_numpy(X)
        hYs = [torch.full((batch, n), float("nan"), dtype=torch.float16) for n in rows]
        if pinned:
            hX, hYs = hX.pin_memory(), [y.pin_memory() for y in hYs]
        ws = torch.zeros(vq.vq_workspace_bytes_grouped_host(fmt, len(rows), batch), dtype=torch.uint8, device="cuda")
        vq.vq_gemm_small_batch_grouped_host(fmt, [(d[0], d[1], d[2], y, n) for d, y, n in zip(dev, hYs, rows)], hX, batch, ws)
        torch.cuda.synchronize()
        dYs = [torch.empty((batch, n), dtype=torch.float16, device="cuda") for n in rows]
        ws2 = torch.zeros(vq.vq_workspace_bytes(fmt, batch), dtype=torch.uint8, device="cuda")
        vq.vq_gemm_small_batch_grouped(fmt, [(d[0], d[1], d[2], y, n) for d, y, n in zip(dev, dYs, rows)], torch.from_numpy(X).cuda(), batch, ws2)
        torch.cuda.synchronize()
        for sp, L, hY, dY in zip(specs, layers, hYs, dYs):
            Yr, A = orc.gemm(oracle_fmt(sp), L.idx, L.cb, L.scale, X, threads=4)
            assert_outputs_close(hY.numpy(), Yr, A, f"{sp.name} batch {batch}")
            assert np.array_equal(hY.numpy().view(np.uint16), dY.cpu().numpy().view(np.uint16))
    with pytest.raises(vq.VQError) as err:   # workspace too small
        vq.vq_gemm_small_batch_grouped_host(fmt, [(d[0], d[1], d[2], y, n) for d, y, n in zip(dev, hYs, rows)], hX, 6,
                                            torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert err.value.code == 5


def test_host_buffer_entry_point():
    import torch
    spec = vq_synth.LayerSpec("host", N=256, K=1024, d=2, b=6, Br=128, Bc=128, int8=False)
    L = draw(spec, 12)
    dev = DeviceLayer(spec, L)
    batch = 4
    X = vq_synth.make_x(spec, 2, batch)
    hX = torch.from_numpy(X).pin_memory()
    hY = torch.zeros((batch, spec.N), dtype=torch.float16).pin_memory()
    ws = torch.zeros(vq.vq_workspace_bytes_host(dev.fmt, batch), dtype=torch.uint8, device="cuda")
    vq.vq_gemm_small_batch_host(dev.fmt, dev.idx, dev.cb, dev.scale, hX, hY, batch, ws)
    torch.cuda.synchronize()
    assert np.array_equal(hY.numpy().view(np.uint16), dev.gemm(X).view(np.uint16))


def test_runtime_argument_errors_on_device_pointers():
    import torch
    spec = vq_synth.LayerSpec("err", N=16, K=64, d=2, b=4, Br=1, Bc=64, int8=False)
    L = draw(spec, 1)
    dev = DeviceLayer(spec, L)
    X = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    Y = torch.zeros((1, 16), dtype=torch.float16, device="cuda")
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(vq.VQError) as e:
        vq.vq_gemm_small_batch(dev.fmt, dev.idx, dev.cb, None, X, Y, 1, small)
    assert e.value.code == 5
    with pytest.raises(vq.VQError) as e:
        buf = torch.zeros(256, dtype=torch.uint8, device="cuda")
        vq.vq_gemm_small_batch(dev.fmt, dev.idx, dev.cb, None, buf[2:130].view(torch.float16), Y, 1, dev.ws)
    assert e.value.code == 4
    with pytest.raises(vq.VQError) as e:
        vq.vq_gemm_small_batch_impl(dev.fmt, dev.idx, dev.cb, None, X, Y, 1, dev.ws, 9)
    assert e.value.code == 7
