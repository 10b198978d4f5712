"""CPU-only checks of the C-ABI library: it loads, exports what include/vq.h declares, sizes and
bits-per-value agree with the paper's printed rows, and every argument error is caught on the
host before any CUDA call (fake non-null pointers are never dereferenced)."""
import ctypes
import os
import re

import pytest

import paper_2402_15319_b200 as vq
from paper_2402_15319_b200 import build as vq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLD = os.path.join(ROOT, "tests", "golden")


@pytest.fixture(scope="module", autouse=True)
def _built():
    vq_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "vq.h")).read()
    declared = set(re.findall(r"\b(vq_[a-z0-9_]+)\s*\(", header))
    assert {"vq_pack_info", "vq_decode_weights", "vq_gemv", "vq_gemm_small_batch"} <= declared
    lib = ctypes.CDLL(vq.lib_path())
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(vq.exported_symbols())


def test_pack_info_matches_paper_bpv_rows():
    # rows of the paper's tables that are expressible as a block of l weights: take 1 x l blocks
    for line in open(os.path.join(GOLD, "bpv_rows.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, d, b_c, l, printed = line.split()[:5]
        k, d, b_c, l = int(k), int(d), int(b_c), int(l)
        b = k.bit_length() - 1
        f = vq.VQFormat(4, l * 2, d, b, 1, l, vq.VQ_CB_FP16 if b_c == 16 else vq.VQ_CB_INT8_SCALED)
        assert vq.vq_pack_info(f).bpv_paper == pytest.approx(float(printed), abs=1e-12), line


def test_pack_info_benchmark_sizes():
    # compressed bytes of the benchmark layers (index + codebook + scale)
    f1 = vq.VQFormat(4096, 4096, 2, 4, 1, 1024, vq.VQ_CB_FP16)
    i1 = vq.vq_pack_info(f1)
    assert (i1.index_bytes, i1.codebook_bytes, i1.scale_bytes, i1.total_bytes) == (4194304, 1048576, 0, 5242880)
    assert i1.bpv_paper == 2.5 and i1.bpv_stored == 2.5 and i1.row_stride_bytes == 1024
    f2 = vq.VQFormat(4096, 4096, 1, 4, 1, 2048, vq.VQ_CB_INT8_SCALED)
    i2 = vq.vq_pack_info(f2)
    assert (i2.index_bytes, i2.codebook_bytes, i2.scale_bytes) == (8388608, 131072, 16384)
    assert i2.bpv_paper == 4.0625 and i2.bpv_stored == pytest.approx(4.0703125)
    f3 = vq.VQFormat(11008, 4096, 2, 6, 128, 128, vq.VQ_CB_FP16)
    i3 = vq.vq_pack_info(f3)
    assert i3.bpv_paper == 3.125 and i3.row_stride_bytes == 1536 and i3.entries == 64
    assert vq.vq_pack_info(vq.VQFormat(4096, 11008, 2, 6, 128, 128, 0)).row_stride_bytes == 4128
    f4 = vq.VQFormat(5120, 13824, 4, 8, 256, 512, vq.VQ_CB_FP16)
    i4 = vq.vq_pack_info(f4)
    assert i4.bpv_paper == 2.125 and i4.codebook_bytes_per_block == 2048 and i4.row_stride_bytes == 3456
    f5 = vq.VQFormat(28672, 8192, 2, 4, 1, 2048, vq.VQ_CB_INT8_SCALED)
    i5 = vq.vq_pack_info(f5)
    assert i5.bpv_paper == 2.125 and i5.bpv_stored == pytest.approx(2.1328125)
    # ragged stride: 3 indices of 5 bits -> 2 bytes -> padded to 16
    assert vq.vq_pack_info(vq.VQFormat(2, 3, 1, 5, 1, 3, 0)).row_stride_bytes == 16


GOOD = vq.VQFormat(8, 16, 2, 4, 1, 16, vq.VQ_CB_FP16)
FAKE = ctypes.c_void_p(0x10000)       # aligned, never dereferenced: every call below fails validation first
ODD = ctypes.c_void_p(0x10008)


def _call_gemm(fmt, idx=FAKE, cb=FAKE, scale=None, X=FAKE, Y=FAKE, batch=1, ws=FAKE, ws_bytes=1 << 30):
    c = fmt.c()
    return vq.load().vq_gemm_small_batch(ctypes.byref(c), idx, cb, scale, X, Y, batch, ws, ws_bytes, None)


def _replace(fmt, **kw):
    d = dict(fmt.__dict__)
    d.update(kw)
    return vq.VQFormat(**d)


@pytest.mark.parametrize("kw,code", [
    (dict(vq_dim=3), 2), (dict(vq_dim=0), 2), (dict(index_bits=0), 2), (dict(index_bits=9), 2),
    (dict(cb_type=3), 2), (dict(cb_type=-1), 2), (dict(n_rows=0), 3), (dict(k_cols=-4), 3), (dict(block_rows=3), 3),
    (dict(block_cols=5), 3), (dict(block_cols=0), 3), (dict(vq_dim=4, block_cols=2, k_cols=16), 3),
])
def test_bad_formats_rejected(kw, code):
    f = _replace(GOOD, **kw)
    with pytest.raises(vq.VQError) as e:
        vq.vq_pack_info(f)
    assert e.value.code == code
    assert vq.vq_workspace_bytes(f, 1) == 0
    assert _call_gemm(f) == code


def test_argument_errors_before_any_launch():
    lib = vq.load()
    c = GOOD.c()
    assert lib.vq_pack_info(None, None) == 1
    assert lib.vq_pack_info(ctypes.byref(c), None) == 1
    assert _call_gemm(GOOD, idx=None) == 1
    assert _call_gemm(GOOD, cb=None) == 1
    assert _call_gemm(GOOD, X=None) == 1
    assert _call_gemm(GOOD, Y=None) == 1
    assert _call_gemm(GOOD, scale=FAKE) == 1                      # fp16 codebook must not carry a scale
    assert _call_gemm(_replace(GOOD, cb_type=1), scale=None) == 1  # int8 codebook needs one
    for k in ("idx", "cb", "X", "Y", "ws"):
        assert _call_gemm(GOOD, **{k: ODD}) == 4
    assert _call_gemm(_replace(GOOD, cb_type=1), scale=ODD) == 4
    assert _call_gemm(GOOD, batch=0) == 6
    assert _call_gemm(GOOD, batch=17) == 6
    assert _call_gemm(GOOD, ws=None) == 5
    assert _call_gemm(GOOD, ws_bytes=vq.vq_workspace_bytes(GOOD, 1) - 1) == 5
    assert vq.vq_workspace_bytes(GOOD, 0) == 0 and vq.vq_workspace_bytes(GOOD, 17) == 0
    assert vq.vq_workspace_bytes(GOOD, 16) >= vq.vq_workspace_bytes(GOOD, 1) > 0
    assert vq.vq_workspace_bytes_host(GOOD, 2) > vq.vq_workspace_bytes(GOOD, 2)
    # decode
    assert lib.vq_decode_weights(ctypes.byref(c), FAKE, FAKE, None, None, None) == 1
    assert lib.vq_decode_weights(ctypes.byref(c), FAKE, FAKE, None, ODD, None) == 4
    assert lib.vq_decode_weights(ctypes.byref(c), None, FAKE, None, FAKE, None) == 1
    # impl selector out of range
    assert lib.vq_gemm_small_batch_impl(ctypes.byref(c), FAKE, FAKE, None, FAKE, FAKE, 1, FAKE, 1 << 30, None, 9) == 7
    # host-buffer variant
    assert lib.vq_gemm_small_batch_host(ctypes.byref(c), FAKE, FAKE, None, None, FAKE, 1, FAKE, 1 << 30, None) == 1
    assert lib.vq_gemm_small_batch_host(ctypes.byref(c), FAKE, FAKE, None, FAKE, FAKE, 1, FAKE, 16, None) == 5
    # INT4 yard-stick
    assert lib.vq_int4g128_gemm_small_batch(8, 100, FAKE, FAKE, FAKE, FAKE, 1, FAKE, 1 << 30, None) == 3
    assert lib.vq_int4g128_gemm_small_batch(8, 256, None, FAKE, FAKE, FAKE, 1, FAKE, 1 << 30, None) == 1
    assert lib.vq_int4g128_gemm_small_batch(8, 256, FAKE, FAKE, ODD, FAKE, 1, FAKE, 1 << 30, None) == 4
    assert lib.vq_int4g128_gemm_small_batch(8, 256, FAKE, FAKE, FAKE, FAKE, 0, FAKE, 1 << 30, None) == 6
    assert lib.vq_int4g128_gemm_small_batch(8, 256, FAKE, FAKE, FAKE, FAKE, 1, None, 1 << 30, None) == 5
    assert lib.vq_int4g128_gemm_small_batch(8, 256, FAKE, FAKE, FAKE, FAKE, 1, FAKE, 16, None) == 5
    assert vq.vq_int4g128_workspace_bytes(8, 1) > 0 and vq.vq_int4g128_workspace_bytes(8, 17) == 0


def test_status_strings():
    names = [vq.vq_status_string(i) for i in range(9)]
    assert names[0] == "VQ_OK" and len(set(names)) == 9
    assert "unknown" in vq.vq_status_string(99)


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    from paper_2402_15319_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="missing"):
        binding.load()


def test_pack_info_int4_codebook_with_group_scales():
    """INT4 codebooks (Sec. 4.2): 4 bits per codebook value, one binary16 scale per row and 128 columns."""
    f = vq.VQFormat(256, 1024, 2, 3, 32, 256, vq.VQ_CB_INT4_G128)
    info = vq.vq_pack_info(f)
    assert info.codebook_bits == 4 and info.entries == 8
    assert info.codebook_bytes_per_block == 8 * 2 // 2
    assert info.n_blocks == (256 // 32) * (1024 // 256)
    assert info.scale_bytes == 2 * 256 * (1024 // 128)
    assert info.total_bytes == info.index_bytes + info.codebook_bytes + info.scale_bytes
    assert abs(info.bpv_paper - (3 / 2 + 8 * 2 * 4 / (32 * 256))) < 1e-12
    with pytest.raises(vq.VQError) as e:          # K must hold whole groups of 128 columns
        vq.vq_pack_info(vq.VQFormat(256, 1024 + 64, 2, 3, 32, 32, vq.VQ_CB_INT4_G128))
    assert e.value.code == 3



def test_grouped_call_argument_errors_and_launch_counts():
    """vq_gemm_small_batch_grouped validates on the host (member pointers, row sums, workspace) before
    any launch, and vq_grouped_kernel_launches tells one kernel for the formats a kernel family takes
    as a group (per-row 4-bit formats, shared-codebook formats, pair-table formats), n_members for the rest."""
    from paper_2402_15319_b200.binding import _CGroupMember
    lib = vq.load()
    total = _replace(GOOD, n_rows=16)
    c = total.c()

    def call(members, n=None, X=FAKE, batch=1, ws=FAKE, ws_bytes=1 << 30, fmt=c):
        arr = (_CGroupMember * max(1, len(members)))()
        for i, m in enumerate(members):
            arr[i] = _CGroupMember(*m)
        return lib.vq_gemm_small_batch_grouped(ctypes.byref(fmt), arr, len(members) if n is None else n, X, batch, ws, ws_bytes, None)

    two = [(FAKE, FAKE, None, FAKE, 8), (FAKE, FAKE, None, FAKE, 8)]
    assert lib.vq_gemm_small_batch_grouped(ctypes.byref(c), None, 2, FAKE, 1, FAKE, 1 << 30, None) == 1
    assert call(two, n=0) == 3 and call(two, n=5) == 3                     # 1..VQ_MAX_GROUP members
    assert call(two, batch=0) == 6 and call(two, batch=17) == 6
    assert call(two, X=None) == 1 and call(two, X=ODD) == 4
    assert call(two, ws=None) == 5 and call(two, ws_bytes=16) == 5 and call(two, ws=ODD) == 4
    assert call([(FAKE, FAKE, None, None, 8), two[1]]) == 1                # member without an output
    assert call([(FAKE, FAKE, None, ODD, 8), two[1]]) == 4
    assert call([(None, FAKE, None, FAKE, 8), two[1]]) == 1
    assert call([(FAKE, FAKE, FAKE, FAKE, 8), two[1]]) == 1                # fp16 codebook must not carry a scale
    assert call([(FAKE, FAKE, None, FAKE, 8), (FAKE, FAKE, None, FAKE, 4)]) == 3   # rows do not add up to fmt.n_rows
    # launch counts (host only)
    row4 = vq.VQFormat(10240, 8192, 2, 4, 1, 2048, vq.VQ_CB_INT8_SCALED)
    blk6 = vq.VQFormat(12288, 4096, 2, 6, 128, 128, vq.VQ_CB_FP16)
    odd5 = vq.VQFormat(42, 312, 1, 5, 1, 156, vq.VQ_CB_FP16)
    # small blocks / index widths only the pair-table kernel takes: 2-D 5-bit 4x256, 1-D 2-bit 1x256, 4-D 8-bit 128x256
    pair = [vq.VQFormat(6144, 4096, 2, 5, 4, 256, vq.VQ_CB_INT8_SCALED), vq.VQFormat(6144, 4096, 1, 2, 1, 256, vq.VQ_CB_INT8_SCALED),
            vq.VQFormat(6144, 4096, 4, 8, 128, 256, vq.VQ_CB_FP16)]
    i4 = vq.VQFormat(6142, 4096, 2, 5, 37, 256, vq.VQ_CB_INT4_G128)   # INT4 codebooks on 37-row blocks: generic kernel, member by member
    pair.append(vq.VQFormat(6144, 4096, 2, 5, 4, 256, vq.VQ_CB_INT4_G128))
    for batch in (1, 4, 16):
        assert vq.vq_grouped_kernel_launches(row4, 3, batch) == 1
        assert vq.vq_grouped_kernel_launches(blk6, 3, batch) == 1
        assert all(vq.vq_grouped_kernel_launches(f, 3, batch) == 1 for f in pair)
        assert vq.vq_grouped_kernel_launches(i4, 3, batch) == 3
        assert vq.vq_grouped_kernel_launches(odd5, 2, batch) == 2
        assert vq.vq_grouped_kernel_launches(row4, 1, batch) == 1
    assert vq.vq_grouped_kernel_launches(row4, 0, 1) == 0 and vq.vq_grouped_kernel_launches(row4, 5, 1) == 0
    assert vq.vq_grouped_kernel_launches(row4, 2, 17) == 0


def test_grouped_host_call_argument_errors():
    from paper_2402_15319_b200.binding import _CGroupMember
    lib = vq.load()
    total = _replace(GOOD, n_rows=16)
    c = total.c()
    arr = (_CGroupMember * 2)(_CGroupMember(FAKE, FAKE, None, FAKE, 8), _CGroupMember(FAKE, FAKE, None, FAKE, 8))
    big = vq.vq_workspace_bytes_grouped_host(total, 2, 1)
    assert big > vq.vq_workspace_bytes(total, 1)
    assert vq.vq_workspace_bytes_grouped_host(total, 0, 1) == 0 and vq.vq_workspace_bytes_grouped_host(total, 2, 17) == 0
    call = lambda n=2, X=FAKE, batch=1, ws=FAKE, nbytes=big: lib.vq_gemm_small_batch_grouped_host(
        ctypes.byref(c), arr, n, X, batch, ws, nbytes, None)
    assert call(X=None) == 1 and call(n=0) == 3 and call(n=5) == 3
    assert call(batch=0) == 6 and call(batch=17) == 6
    assert call(ws=None) == 5 and call(nbytes=big - 600) == 5 and call(ws=ODD) == 4
    arr[1].n_rows = 4       # rows no longer add up
    assert call() == 3
    arr[1].n_rows = 8
    arr[0].d_Y = None
    assert call() == 1


def test_normalized_entry_points_argument_errors_and_sizes():
    """Block-wise normalisation: buffer sizes on the host, and every argument error before any launch."""
    lib = vq.load()
    fmt = vq.VQFormat(12, 256, 2, 5, 4, 128, vq.VQ_CB_INT8_SCALED)
    assert vq.vq_norm_info(fmt, 32) == (4, 48, 3 * 2 * 16 * 2)            # 8 sub-rows -> 4 bytes per row; 6 blocks
    assert vq.vq_norm_info(fmt, 128)[0] == 1                               # 2 sub-rows per row
    assert vq.vq_norm_info(vq.VQFormat(3, 48, 1, 3, 1, 48, vq.VQ_CB_FP16), 16) == (2, 6, 3 * 16 * 2)   # 3 codes -> 2 bytes
    c = fmt.c()

    def dec(codes=FAKE, lut=FAKE, nbc=32, W=FAKE, scale=FAKE):
        return lib.vq_decode_weights_normalized(ctypes.byref(c), FAKE, FAKE, scale, codes, lut, nbc, W, None)

    def gemm(codes=FAKE, lut=FAKE, nbc=32, X=FAKE, Y=FAKE, batch=1):
        return lib.vq_gemm_small_batch_normalized(ctypes.byref(c), FAKE, FAKE, FAKE, codes, lut, nbc, X, Y, batch, None)

    assert dec(codes=None) == 1 and dec(lut=None) == 1 and dec(W=None) == 1 and dec(scale=None) == 1
    assert dec(nbc=0) == 3 and dec(nbc=48) == 3 and dec(nbc=256) == 3       # must divide block_cols = 128
    assert lib.vq_decode_weights_normalized(ctypes.byref(vq.VQFormat(12, 256, 4, 8, 4, 128, vq.VQ_CB_INT8_SCALED).c()),
                                            FAKE, FAKE, FAKE, FAKE, FAKE, 2, FAKE, None) == 3            # not a multiple of vq_dim
    assert dec(codes=ODD) == 4 and dec(lut=ODD) == 4 and dec(W=ODD) == 4
    assert gemm(codes=None) == 1 and gemm(X=None) == 1 and gemm(Y=None) == 1
    assert gemm(batch=0) == 6 and gemm(batch=17) == 6 and gemm(nbc=5) == 3 and gemm(X=ODD) == 4
    out = ctypes.c_void_p(0)
    assert lib.vq_norm_info(ctypes.byref(c), 32, None) == 1 and lib.vq_norm_info(ctypes.byref(c), 3, FAKE) == 3
