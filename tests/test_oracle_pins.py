"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself or with the CUDA path: expected values are
the paper's printed numbers (tests/golden/*.txt, each with its citation), hand-written
matrices, an independent big-integer / exact-rational brute force, numpy's float16, or
algebraic invariants.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import vq_synth
from oracle import vq_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line)
    return out


# --------------------------------------------------------------------------------------
# P1 / P2: bits per value, Sec. 4 "Total bits per value", against rows the paper prints
# --------------------------------------------------------------------------------------
def test_bpv_matches_paper_rows():
    rows = _rows("bpv_rows.txt")
    assert len(rows) >= 15
    for r in rows:
        k, d, b_c, l, printed = r.split()[:5]
        assert orc.bpv(int(k), int(d), int(b_c), int(l)) == pytest.approx(float(printed), abs=1e-12), r


def test_bpv_uniform_rows():
    for r in _rows("uniform_bpv_rows.txt"):
        bits, sb, g, printed = r.split()[:4]
        assert orc.bpv_uniform(int(bits), int(sb), int(g)) == pytest.approx(float(printed), abs=1e-12)


def test_relative_footprint_column():
    # App. B table prints bpv/4 to two decimals
    for r in _rows("rel_footprint_rows.txt"):
        bpv, printed = r.split()[:2]
        rel = float(bpv) / 4.0
        assert abs(rel - float(printed)) <= 0.005 + 1e-12, r
    # and the VQ rows of that table are reachable by the closed form
    assert orc.bpv(16, 2, 8, 2048) / 4 == pytest.approx(0.53125)
    assert orc.bpv(64, 2, 8, 8192) / 4 == pytest.approx(0.78125)


def test_bpv_of_benchmark_formats():
    # 2-D, 6-bit indices, fp16 codebook per 128x128 block -> 3.125; 4-D 8-bit per 256x512 -> 2.125
    assert orc.bpv(64, 2, 16, 128 * 128) == pytest.approx(3.125)
    assert orc.bpv(256, 4, 16, 256 * 512) == pytest.approx(2.125)
    assert orc.bpv(16, 2, 16, 1024) == pytest.approx(2.5)
    # Sec. 2.1: 3 bits per value in pairs -> 2^6 = 64 centroids
    assert 2 ** (3 * 2) == 64


# --------------------------------------------------------------------------------------
# binary16 conversions against numpy (an independent implementation)
# --------------------------------------------------------------------------------------
def test_f16_to_f64_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([orc.f16_bits_to_f64(int(b)) for b in bits])
    fin = np.isfinite(want)
    assert np.array_equal(got[fin], want[fin])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want))
    assert np.array_equal(np.signbit(got[fin]), np.signbit(want[fin]))


def test_f64_to_f16_rounding():
    rng = np.random.default_rng(0)
    xs = np.concatenate([
        rng.normal(size=20000), rng.normal(size=5000) * 1e-5, rng.normal(size=5000) * 1e-7,
        rng.normal(size=2000) * 3e4, rng.normal(size=200) * 1e5,
        np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25,
                  2.0 ** -14, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 1.0 + 2.0 ** -11 + 2.0 ** -30]),
    ])
    # exact ties between neighbouring halves
    h = rng.integers(0, 0x7BFF, size=4000).astype(np.uint16)
    lo = h.view(np.float16).astype(np.float64)
    hi = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    xs = np.concatenate([xs, (lo + hi) / 2, -(lo + hi) / 2])
    with np.errstate(over="ignore"):
        want = xs.astype(np.float16).view(np.uint16)
    got = np.array([orc.f64_to_f16_bits(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(got, want)


# --------------------------------------------------------------------------------------
# P5: packing — hand-derived bytes, identity
# --------------------------------------------------------------------------------------
def test_pack_golden_bytes():
    for r in _rows("pack_bytes.txt"):
        b_s, idx_s, bytes_s = [p.strip() for p in r.split("|")]
        b = int(b_s)
        I = np.array([int(v) for v in idx_s.split()], dtype=np.uint8)[None, :]
        want = bytes(int(v, 16) for v in bytes_s.split())
        f = orc.Fmt(N=1, K=I.shape[1], d=1, b=b, Br=1, Bc=I.shape[1], int8=False)
        packed = orc.pack(f, I)
        assert packed.shape == (1, 16)  # stride is rounded up to 16 bytes
        assert bytes(packed[0, : len(want)]) == want, r
        assert not packed[0, len(want):].any()
        assert np.array_equal(orc.unpack(f, packed), I)


def test_row_stride_rule():
    # ceil(K/d*b/8) rounded up to 16; values for the benchmark shapes
    assert orc.row_stride_bytes(4096, 2, 4) == 1024
    assert orc.row_stride_bytes(4096, 1, 4) == 2048
    assert orc.row_stride_bytes(4096, 2, 6) == 1536
    assert orc.row_stride_bytes(11008, 2, 6) == 4128
    assert orc.row_stride_bytes(5120, 4, 8) == 1280
    assert orc.row_stride_bytes(13824, 4, 8) == 3456
    assert orc.row_stride_bytes(8192, 2, 4) == 2048
    assert orc.row_stride_bytes(28672, 2, 4) == 7168
    assert orc.row_stride_bytes(16, 1, 1) == 16
    assert orc.row_stride_bytes(136, 1, 1) == 32


@pytest.mark.parametrize("b", range(1, 9))
@pytest.mark.parametrize("d", [1, 2, 4])
def test_pack_unpack_identity_and_padding_ignored(b, d):
    rng = np.random.default_rng(100 * b + d)
    N, K = 5, 24 * d
    f = orc.Fmt(N, K, d, b, 1, K, False)
    I = rng.integers(0, 1 << b, size=(N, K // d)).astype(np.uint8)
    zero_pad = orc.pack(f, I)
    junk = rng.integers(0, 256, size=(N, f.stride)).astype(np.uint8)
    junk_pad = orc.pack(f, I, fill=junk)
    assert np.array_equal(orc.unpack(f, zero_pad), I)
    assert np.array_equal(orc.unpack(f, junk_pad), I)
    used_bits = (K // d) * b
    # bytes wholly inside the used range are identical whatever the padding was
    assert np.array_equal(zero_pad[:, : used_bits // 8], junk_pad[:, : used_bits // 8])


# --------------------------------------------------------------------------------------
# P4: brute force — big-integer bit reader + exact rationals, no code shared with the oracle
# --------------------------------------------------------------------------------------
def _brute_index(row_bytes: bytes, j: int, b: int) -> int:
    big = int.from_bytes(row_bytes, "little")
    return (big // (2 ** (j * b))) % (2 ** b)


def _frac_half(v) -> Fraction:
    return Fraction(float(np.float16(v)))


def _brute_layer(f, idx, cb, scale, X):
    """W as exact Fractions and Y = W X exactly, straight from the definition."""
    W = [[None] * f.K for _ in range(f.N)]
    for n in range(f.N):
        rb = bytes(idx[n])
        for k in range(f.K):
            e = _brute_index(rb, k // f.d, f.b)
            blk = (n // f.Br) * (f.K // f.Bc) + (k // f.Bc)
            c = cb[blk][e][k % f.d]
            W[n][k] = Fraction(int(c)) * _frac_half(scale[blk]) if f.int8 else _frac_half(c)
    Y = [[sum(W[n][k] * _frac_half(X[m][k]) for k in range(f.K)) for n in range(f.N)] for m in range(X.shape[0])]
    A = [[sum(abs(W[n][k] * _frac_half(X[m][k])) for k in range(f.K)) for n in range(f.N)] for m in range(X.shape[0])]
    return W, Y, A


BLOCKS_8x16 = [(1, 16), (1, 8), (8, 16), (2, 4), (4, 8), (8, 4)]


@pytest.mark.parametrize("int8", [False, True])
@pytest.mark.parametrize("b", range(1, 9))
@pytest.mark.parametrize("d", [1, 2, 4])
def test_bruteforce_8x16(d, b, int8):
    N, K = 8, 16
    Br, Bc = BLOCKS_8x16[(b + d) % len(BLOCKS_8x16)]
    spec = vq_synth.LayerSpec("t", N, K, d, b, Br, Bc, int8)
    f = orc.Fmt(N, K, d, b, Br, Bc, int8)
    L = vq_synth.make_layer(spec, f.stride, seed=1000 + 31 * b + d)
    X = vq_synth.make_x(spec, seed=7, batch=3)
    Wb, Yb, Ab = _brute_layer(f, L.idx, L.cb, L.scale, X)

    I = orc.unpack(f, L.idx)
    for n in range(N):
        for j in range(K // d):
            assert I[n, j] == _brute_index(bytes(L.idx[n]), j, b)

    We, Wh = orc.decode(f, L.idx, L.cb, L.scale)
    for n in range(N):
        for k in range(K):
            assert Fraction(We[n, k]) == Wb[n][k]          # exact in fp64
            want_half = np.float16(float(Wb[n][k]))         # numpy RN-even from the exact value
            assert Wh[n, k] == want_half.view(np.uint16)
    Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X)
    for m in range(3):
        for n in range(N):
            tol = 1e-13 * float(Ab[m][n]) + 1e-300
            assert abs(Y[m, n] - float(Yb[m][n])) <= tol
            assert abs(A[m, n] - float(Ab[m][n])) <= tol


# --------------------------------------------------------------------------------------
# P3: exact decode on a hand-built codebook — expected matrix written out by hand
# --------------------------------------------------------------------------------------
def test_decode_hand_built_fp16():
    # N=2, K=8, d=2, b=2 (4 entries), blocks 1x4 -> 4 blocks: (row0,c0-3) (row0,c4-7) (row1,..) (row1,..)
    f = orc.Fmt(2, 8, 2, 2, 1, 4, False)
    cb = np.zeros((4, 4, 2), np.float16)
    for blk in range(4):
        for e in range(4):
            cb[blk, e] = [blk * 10 + e, -(blk * 10 + e) - 0.5]
    # row 0 indices (per pair of columns): 0 1 | 2 3 ; row 1: 3 3 | 0 2
    I = np.array([[0, 1, 2, 3], [3, 3, 0, 2]], np.uint8)
    idx = orc.pack(f, I)
    assert idx[0, 0] == 0b11100100 and idx[1, 0] == 0b10001111
    want = np.array([
        [0, -0.5, 1, -1.5, 12, -12.5, 13, -13.5],
        [23, -23.5, 23, -23.5, 30, -30.5, 32, -32.5],
    ], np.float64)
    We, Wh = orc.decode(f, idx, cb)
    assert np.array_equal(We, want)
    assert np.array_equal(Wh, want.astype(np.float16).view(np.uint16))


def test_decode_hand_built_int8_block_rows():
    # N=4, K=4, d=1, b=1 (2 entries), blocks 2x2 -> blk = (n//2)*2 + k//2
    f = orc.Fmt(4, 4, 1, 1, 2, 2, True)
    cb = np.array([[[-3], [5]], [[7], [-127]], [[0], [1]], [[100], [-100]]], np.int8)
    scale = np.array([0.5, 2.0, 0.25, 1.0], np.float16)
    I = np.array([[0, 1, 1, 0], [1, 1, 0, 0], [1, 0, 0, 1], [0, 0, 1, 1]], np.uint8)
    idx = orc.pack(f, I)
    want = np.array([
        [-1.5, 2.5, -254.0, 14.0],
        [2.5, 2.5, 14.0, 14.0],
        [0.25, 0.0, 100.0, -100.0],
        [0.0, 0.0, -100.0, -100.0],
    ])
    We, _ = orc.decode(f, idx, cb, scale)
    assert np.array_equal(We, want)
    # y = W x with x = (1, 2, 3, 4), by hand
    x = np.array([[1, 2, 3, 4]], np.float16)
    Y, A = orc.gemm(f, idx, cb, scale, x)
    assert np.array_equal(Y[0], [-1.5 + 5 - 762 + 56, 2.5 + 5 + 42 + 56, 0.25 + 0 + 300 - 400, -300 - 400])
    assert np.array_equal(A[0], [1.5 + 5 + 762 + 56, 105.5, 700.25, 700])


# --------------------------------------------------------------------------------------
# P6 / P7: invariants
# --------------------------------------------------------------------------------------
def _rand_layer(seed, N=12, K=48, d=2, b=6, Br=4, Bc=16, int8=False):
    spec = vq_synth.LayerSpec("t", N, K, d, b, Br, Bc, int8)
    f = orc.Fmt(N, K, d, b, Br, Bc, int8)
    return f, spec, vq_synth.make_layer(spec, f.stride, seed)


@pytest.mark.parametrize("int8", [False, True])
def test_unit_vector_returns_decoded_column(int8):
    f, spec, L = _rand_layer(11, int8=int8)
    We, _ = orc.decode(f, L.idx, L.cb, L.scale)
    X = np.eye(f.K, dtype=np.float16)[:16]
    Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X)
    for k in range(16):
        assert np.array_equal(Y[k], We[:, k])
        assert np.array_equal(A[k], np.abs(We[:, k]))


@pytest.mark.parametrize("d,b,int8", [(1, 4, True), (2, 4, False), (4, 8, False), (2, 5, True), (1, 3, False)])
def test_fused_equals_decode_then_dense(d, b, int8):
    f, spec, L = _rand_layer(5, N=8, K=32 * d, d=d, b=b, Br=2, Bc=8 * d, int8=int8)
    X = vq_synth.make_x(spec, 3, batch=4)
    We, _ = orc.decode(f, L.idx, L.cb, L.scale)
    Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X)
    assert np.array_equal(Y, orc.dense_gemm(We, X))  # same summation order -> same bits
    # and against numpy's own matmul (different order -> tolerance)
    ref = X.astype(np.float64) @ We.T
    assert np.allclose(Y, ref, rtol=0, atol=1e-12 * A.max())
    assert np.allclose(A, np.abs(X.astype(np.float64)) @ np.abs(We).T, rtol=1e-12)


def test_linearity_in_x():
    f, spec, L = _rand_layer(21)
    # small integers: sums are exact in fp64 so linearity holds exactly
    rng = np.random.default_rng(3)
    x1 = rng.integers(-8, 9, size=(1, f.K)).astype(np.float16)
    x2 = rng.integers(-8, 9, size=(1, f.K)).astype(np.float16)
    cb = (rng.integers(-64, 65, size=L.cb.shape) / 64.0).astype(np.float16)
    y1, _ = orc.gemm(f, L.idx, cb, None, x1)
    y2, _ = orc.gemm(f, L.idx, cb, None, x2)
    y12, _ = orc.gemm(f, L.idx, cb, None, (x1 + 2 * x2).astype(np.float16))
    assert np.array_equal(y12, y1 + 2 * y2)


def test_all_indices_equal_closed_form():
    # every index = e  =>  y[n] = sum_j <cb[blk(n,j)][e], x_j>
    N, K, d, b, Br, Bc = 6, 32, 2, 3, 3, 8
    f = orc.Fmt(N, K, d, b, Br, Bc, False)
    rng = np.random.default_rng(5)
    cb = (rng.integers(-32, 33, size=(f.n_blocks, 8, d)) / 8.0).astype(np.float16)
    x = rng.integers(-4, 5, size=(1, K)).astype(np.float16)
    for e in (0, 5, 7):
        idx = orc.pack(f, np.full((N, K // d), e, np.uint8))
        Y, _ = orc.gemm(f, idx, cb, None, x)
        for n in range(N):
            want = 0.0
            for cbk in range(K // Bc):
                blk = (n // Br) * (K // Bc) + cbk
                seg = x[0, cbk * Bc:(cbk + 1) * Bc].astype(np.float64).reshape(-1, d)
                want += float((seg * cb[blk, e].astype(np.float64)).sum())
            assert Y[0, n] == want


def test_codebook_permutation_invariance():
    # App. "Codebook compression": sorting a codebook and re-assigning indices leaves the tensor unchanged
    f, spec, L = _rand_layer(33, d=2, b=4, Br=4, Bc=16)
    X = vq_synth.make_x(spec, 1, batch=2)
    I = orc.unpack(f, L.idx)
    rng = np.random.default_rng(9)
    cb2 = L.cb.copy()
    I2 = I.copy()
    for blk in range(f.n_blocks):
        perm = rng.permutation(f.entries)           # new position p holds old entry perm[p]
        inv = np.argsort(perm)
        cb2[blk] = L.cb[blk][perm]
        r0 = (blk // (f.K // f.Bc)) * f.Br
        c0 = (blk % (f.K // f.Bc)) * f.Bc // f.d
        sub = I[r0:r0 + f.Br, c0:c0 + f.Bc // f.d]
        I2[r0:r0 + f.Br, c0:c0 + f.Bc // f.d] = inv[sub]
    idx2 = orc.pack(f, I2)
    W1, H1 = orc.decode(f, L.idx, L.cb)
    W2, H2 = orc.decode(f, idx2, cb2)
    assert np.array_equal(W1, W2) and np.array_equal(H1, H2)
    assert np.array_equal(orc.gemm(f, L.idx, L.cb, None, X)[0], orc.gemm(f, idx2, cb2, None, X)[0])


def test_gemm_row_equals_gemv_and_row_subset():
    f, spec, L = _rand_layer(44, int8=True)
    X = vq_synth.make_x(spec, 2, batch=5)
    Y, A = orc.gemm(f, L.idx, L.cb, L.scale, X)
    for m in range(5):
        y, a = orc.gemm(f, L.idx, L.cb, L.scale, X[m])
        assert np.array_equal(y[0], Y[m]) and np.array_equal(a[0], A[m])
    rows = np.array([7, 0, 11, 3], np.int32)
    Ys, As = orc.gemm(f, L.idx, L.cb, L.scale, X, rows=rows)
    assert np.array_equal(Ys, Y[:, rows]) and np.array_equal(As, A[:, rows])
    Yt, At = orc.gemm(f, L.idx, L.cb, L.scale, X, threads=3)
    assert np.array_equal(Yt, Y) and np.array_equal(At, A)


def test_int8_unit_scale_integer_inputs_exact():
    f, spec, L = _rand_layer(55, int8=True, d=2, b=4)
    scale = np.ones(f.n_blocks, np.float16)
    rng = np.random.default_rng(1)
    x = rng.integers(-16, 17, size=(1, f.K)).astype(np.float16)
    Y, _ = orc.gemm(f, L.idx, L.cb, scale, x)
    I = orc.unpack(f, L.idx)
    for n in range(f.N):
        want = 0
        for k in range(f.K):
            blk = (n // f.Br) * (f.K // f.Bc) + k // f.Bc
            want += int(L.cb[blk, I[n, k // f.d], k % f.d]) * int(x[0, k])
        assert Y[0, n] == want


def test_int4g128_bruteforce():
    N, K = 3, 256
    q, s = vq_synth.make_int4g128(N, K, seed=2)
    spec = vq_synth.LayerSpec("t", N, K, 1, 4, 1, 128, True)
    X = vq_synth.make_x(spec, 5, batch=2)
    Y, A = orc.int4g128_gemm(q, s, X)
    for m in range(2):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                byte = int(q[n, k // 2])
                nib = (byte // 16) if k % 2 else (byte % 16)
                acc += Fraction(nib - 8) * _frac_half(s[n, k // 128]) * _frac_half(X[m, k])
            assert abs(Y[m, n] - float(acc)) <= 1e-13 * A[m, n]
    # hand case: all nibbles 0x9 -> +1, scale 2 -> y = 2*sum(x)
    q1 = np.full((1, 64), 0x99, np.uint8)
    s1 = np.full((1, 1), 2.0, np.float16)
    x1 = np.arange(128, dtype=np.float16)[None, :]
    Y1, A1 = orc.int4g128_gemm(q1, s1, x1)
    assert Y1[0, 0] == 2 * (127 * 128 // 2) and A1[0, 0] == Y1[0, 0]
    # low nibble first: byte 0x1f -> column 0 holds 15-8 = 7, column 1 holds 1-8 = -7
    q2 = np.zeros((1, 64), np.uint8) + 0x88
    q2[0, 0] = 0x1F
    x2 = np.zeros((1, 128), np.float16)
    x2[0, 0] = 1
    assert orc.int4g128_gemm(q2, np.ones((1, 1), np.float16), x2)[0][0, 0] == 7
    x2[0, 0], x2[0, 1] = 0, 1
    assert orc.int4g128_gemm(q2, np.ones((1, 1), np.float16), x2)[0][0, 0] == -7


def test_synth_is_deterministic_and_distributed():
    a = vq_synth.normal(3, 1, 200001)
    b = vq_synth.normal(3, 1, 200001)
    assert np.array_equal(a, b)
    assert abs(a.mean()) < 0.01 and abs(a.std() - 1) < 0.01
    u = vq_synth.uniform01(3, 2, 100000)
    assert 0 <= u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 0.01
    by = vq_synth.random_bytes(1, 1, 100003)
    assert by.size == 100003 and abs(by.mean() - 127.5) < 1.5
    spec = vq_synth.CONFIGS["cfg2"]["layers"][0]
    L = vq_synth.make_layer(vq_synth.LayerSpec("s", 64, 4096, 1, 4, 1, 2048, True), 2048, 1)
    assert L.cb.min() >= -127 and L.cb.max() <= 127
    assert 0.0005 <= float(L.scale.min()) and float(L.scale.max()) <= 0.002
    assert spec.N == 4096 and spec.K == 4096


def test_unpack_uniform_hand_values():
    """Yard-stick unpackers against values worked out by hand (Sec. 2.1: w = s * q)."""
    # int4 g128: nibble 0 -> -8, nibble 15 -> +7; low nibble is the lower column; scale per 128 columns
    b = np.zeros((1, 128), np.uint8)        # K = 256: two groups
    b[0, 0] = 0xF0                          # columns 0, 1 = nibbles 0, 15
    b[0, 64] = 0x9A                         # columns 128, 129 = nibbles 10, 9
    s = np.array([[0.5, 2.0]], np.float16)
    W = orc.unpack_uniform("int4g128", b, s)
    assert W.dtype == np.float16 and W.shape == (1, 256)
    assert W[0, 0] == -4.0 and W[0, 1] == 3.5 and W[0, 2] == -4.0
    assert W[0, 128] == 4.0 and W[0, 129] == 2.0 and W[0, 130] == -16.0
    # int8 with a row scale; 0.1 is not a binary16 value: s = 0.0999755859375, s * 127 rounds once
    q = np.array([[-128, 127, 0, 3]], np.int8)
    W8 = orc.unpack_uniform("int8row", q, np.array([0.1], np.float16))
    s16 = float(np.float16(0.1))
    assert s16 == 0.0999755859375
    assert W8[0, 0] == np.float16(-128 * s16) and W8[0, 1] == np.float16(127 * s16) and W8[0, 2] == 0 and W8[0, 3] == np.float16(3 * s16)
    assert float(W8[0, 0]) == -12.796875      # -128 * s is a power-of-two multiple: exact
    # the rounding is one rounding of the exact product, not of a float32-rounded scale times q twice
    exact = 127 * s16
    lo, hi = np.float16(12.6953125), np.float16(12.703125)   # neighbours around 12.696899...
    assert float(lo) < exact < float(hi) and W8[0, 1] == lo
    # fp16 is a copy
    w = np.array([[1.5, -0.0, 65504.0]], np.float16)
    assert np.array_equal(orc.unpack_uniform("fp16", w).view(np.uint16), w.view(np.uint16))


# ---- E-step (Eq. 5) and SQNR (Sec. 2.2) ------------------------------------------------------------
def _exact_assign(x, C, D):
    """Brute force in exact rational arithmetic: all minimisers of sum_t D_t (x_t - c_mt)^2."""
    from fractions import Fraction as Fr
    dist = [sum(Fr(float(D[t])) * (Fr(float(x[t])) - Fr(float(c[t]))) ** 2 for t in range(len(x))) for c in C]
    best = min(dist)
    return [m for m, v in enumerate(dist) if v == best], dist


@pytest.mark.parametrize("d,b,int8", [(1, 3, False), (2, 4, True), (2, 6, False), (4, 5, True)])
def test_assign_is_an_exact_minimiser_or_a_rounding_tie(d, b, int8):
    """Every index the oracle picks minimises the weighted distance exactly, or is within binary32
    rounding (2^-20 relative) of the exact minimum; plain brute force with Fractions."""
    spec = vq_synth.LayerSpec("e", N=8, K=16 * d, d=d, b=b, Br=4, Bc=8 * d, int8=int8)
    f = orc.Fmt(spec.N, spec.K, d, b, spec.Br, spec.Bc, int8)
    L = vq_synth.make_layer(spec, f.stride, 5)
    W = (0.03 * vq_synth.normal(5, 40, spec.N * spec.K)).astype(np.float16).reshape(spec.N, spec.K)
    h = (0.5 + vq_synth.uniform01(5, 41, spec.K)).astype(np.float32)
    I = orc.assign(f, W, L.cb, L.scale, h)
    assert I.shape == (spec.N, spec.K // d) and I.max() < (1 << b)
    bpr = spec.K // spec.Bc
    exact_hits = 0
    for n in range(spec.N):
        for j in range(spec.K // d):
            blk = (n // spec.Br) * bpr + (j * d) // spec.Bc
            C = L.cb[blk].astype(np.float64) * (float(L.scale[blk]) if int8 else 1.0)
            mins, dist = _exact_assign(W[n, j * d:(j + 1) * d], C, h[j * d:(j + 1) * d])
            if I[n, j] in mins:
                exact_hits += 1
            else:
                assert float(dist[I[n, j]] - dist[mins[0]]) <= 2.0 ** -20 * float(dist[mins[0]])
    assert exact_hits >= 0.99 * spec.N * (spec.K // d)


def test_assign_identity_weights_is_nearest_centroid():
    """D = I: the E-step is K-means' assignment (Sec. 3); scipy's vector quantiser is the library routine."""
    from scipy.cluster.vq import vq as scipy_vq
    spec = vq_synth.LayerSpec("km", N=16, K=64, d=2, b=4, Br=16, Bc=64, int8=False)
    f = orc.Fmt(16, 64, 2, 4, 16, 64, False)
    L = vq_synth.make_layer(spec, f.stride, 6)
    W = (0.02 * vq_synth.normal(6, 40, 16 * 64)).astype(np.float16).reshape(16, 64)
    I = orc.assign(f, W, L.cb, None, None)
    code, _ = scipy_vq(W.astype(np.float64).reshape(-1, 2), L.cb[0].astype(np.float64))
    # scipy decides in binary64: allow only disagreements that are binary32-level ties
    diff = np.flatnonzero(code != I.reshape(-1))
    X = W.astype(np.float64).reshape(-1, 2)
    C = L.cb[0].astype(np.float64)
    for i in diff:
        da = ((X[i] - C[code[i]]) ** 2).sum()
        db = ((X[i] - C[I.reshape(-1)[i]]) ** 2).sum()
        assert abs(da - db) <= 2.0 ** -20 * da
    assert diff.size <= 2


def test_assign_special_cases():
    # 1-D, centroids on a uniform grid: the E-step is round-to-nearest of x / step (Sec. 2.1 uniform quantizer)
    f = orc.Fmt(2, 32, 1, 3, 1, 32, False)
    grid = (np.arange(8) - 4) * 0.25
    cb = np.tile(grid.astype(np.float16), (2, 1)).reshape(2, 8, 1)
    W = np.linspace(-1.2, 0.9, 64).astype(np.float16).reshape(2, 32)
    I = orc.assign(f, W, cb)
    want = np.clip(np.floor(W.astype(np.float64) / 0.25 + 0.5), -4, 3) + 4     # half-way cases go up = lower |distance| tie -> check separately
    ties = np.isclose((W.astype(np.float64) / 0.25) % 1.0, 0.5)
    assert np.array_equal(I[~ties], want[~ties].astype(np.uint8))
    # exact ties go to the lower index
    assert orc.assign(orc.Fmt(1, 1, 1, 1, 1, 1, False), np.array([[0.5]], np.float16), np.array([[[0.0], [1.0]]], np.float16))[0, 0] == 0
    # the weights matter: x = (1, 0) between c0 = (0, 0) and c1 = (1, 1); D = (1, 9) -> c0, D = (9, 1) -> c1
    f2 = orc.Fmt(1, 2, 2, 1, 1, 2, False)
    cb2 = np.array([[[0.0, 0.0], [1.0, 1.0]]], np.float16)
    x = np.array([[1.0, 0.0]], np.float16)
    assert orc.assign(f2, x, cb2, None, np.array([1.0, 9.0], np.float32))[0, 0] == 0
    assert orc.assign(f2, x, cb2, None, np.array([9.0, 1.0], np.float32))[0, 0] == 1
    # a weight that is itself a centroid maps to it; decode(pack(assign)) then returns the weight
    f3 = orc.Fmt(4, 8, 2, 3, 2, 4, True)
    spec3 = vq_synth.LayerSpec("rt", 4, 8, 2, 3, 2, 4, True)
    L3 = vq_synth.make_layer(spec3, f3.stride, 8)
    _, W16 = orc.decode(f3, L3.idx, L3.cb, L3.scale, exact=False)
    Wq = W16.view(np.float16)
    I3 = orc.assign(f3, Wq, L3.cb, L3.scale)
    _, W16b = orc.decode(f3, orc.pack(f3, I3), L3.cb, L3.scale, exact=False)
    assert np.array_equal(W16b, W16)          # idempotent: quantising a quantised matrix changes nothing


def test_sqnr_closed_forms():
    assert abs(orc.sqnr_db(np.array([1.0, -1.0]), np.array([0.5, -0.5])) - 10 * np.log10(4.0)) < 1e-12
    # uniform quantizer with step q on a signal uniform in [-A, A]: noise power q^2/12, signal A^2/3
    A, q = 1.0, 2.0 / 256
    w = (np.arange(1 << 16) + 0.5) / (1 << 16) * 2 * A - A
    qw = (np.floor(w / q) + 0.5) * q
    assert abs(orc.sqnr_db(w, qw) - 10 * np.log10((A * A / 3) / (q * q / 12))) < 1e-3


def test_int4_codebook_with_group_scales_hand_values():
    """INT4 codebooks decoded with a scale per row and group of 128 columns (Sec. 4.2): values by hand."""
    f = orc.Fmt(2, 256, 2, 2, 2, 256, 2)            # one block, 4 entries of 2 nibbles, two groups per row
    cb = np.array([[0x10, 0xF7, 0x8F, 0x23]], np.uint8)   # entries: (0,1) (7,-1) (-1,-8) (3,2)
    I = np.zeros((2, 128), np.uint8)
    I[0, 0], I[0, 1], I[0, 64], I[1, 127] = 1, 2, 3, 2
    idx = orc.pack(f, I)
    scale = np.array([[0.5, 2.0], [0.25, 3.0]], np.float16)
    W, W16 = orc.decode(f, idx, cb, scale)
    assert W[0, 0] == 3.5 and W[0, 1] == -0.5           # entry 1 = (7,-1), group 0 of row 0: x0.5
    assert W[0, 2] == -0.5 and W[0, 3] == -4.0          # entry 2 = (-1,-8)
    assert W[0, 4] == 0.0 and W[0, 5] == 0.5            # entry 0 = (0,1)
    assert W[0, 128] == 6.0 and W[0, 129] == 4.0        # entry 3 = (3,2), group 1 of row 0: x2
    assert W[1, 254] == -3.0 and W[1, 255] == -24.0     # row 1, group 1: x3
    assert np.array_equal(W16.view(np.float16).astype(np.float64), W)   # all exactly representable here
    # bits per value: 2/2 index + 4*2*4/512 codebook = 1.0625 (Sec. 4 formula, b_c = 4)
    assert abs(orc.bpv(4, 2, 4, 512) - 1.0625) < 1e-12
    # mat-vec = dense product on the decoded matrix
    x = vq_synth.normal(3, 1, 256).astype(np.float16)
    Y, A = orc.gemm(f, idx, cb, scale, x)
    assert np.allclose(Y[0], W @ x.astype(np.float64), rtol=1e-14, atol=0)



# ---- block-wise normalisation at decode (App. on blockwise data normalization) ------------------------
def test_norm_lut_log2_hand_values():
    """2^(a*s + z): a = 1, z = -3 gives the powers of two 1/8 .. 4096 exactly; a = 0.5 puts sqrt(2) at s = 1,
    whose nearest binary16 is 1.4140625 (0x3DA8: 1.4140625 < 1.41421356 < 1.415039, nearer the lower)."""
    lut = orc.norm_lut_log2(1.0, -3.0)
    assert lut.dtype == np.float16 and [float(v) for v in lut] == [2.0 ** (s - 3) for s in range(16)]
    half = orc.norm_lut_log2(0.5, 0.0)
    assert float(half[0]) == 1.0 and float(half[2]) == 2.0 and float(half[4]) == 4.0
    assert half.view(np.uint16)[1] == 0x3DA8 and float(half[1]) == 1.4140625
    assert float(orc.norm_lut_log2(0.0, 0.0)[7]) == 1.0                      # zero step: unit scaling whatever the code


def test_normalized_decode_hand_built():
    """2 x 8 weights, 2-D entries, 1-bit indices, one codebook for the whole matrix, sub-rows of 4 columns:
    every number below is written by hand."""
    f = orc.Fmt(N=2, K=8, d=2, b=1, Br=2, Bc=8, int8=False)
    cb = np.array([[1.0, 2.0], [-3.0, 0.5]], np.float16)                       # entry 0 = (1, 2), entry 1 = (-3, 0.5)
    I = np.array([[0, 1, 1, 0], [1, 1, 0, 0]], np.int32)                       # 4 indices per row
    idx = orc.pack(f, I)
    lut = np.zeros((1, 16), np.float16)
    lut[0, 0], lut[0, 3], lut[0, 9], lut[0, 15] = 1.0, 0.5, 4.0, 0.25
    # codes: row 0 -> sub-rows (3, 9) = byte 0x93; row 1 -> (15, 0) = byte 0x0F   (low nibble = first sub-row)
    codes = np.array([[0x93], [0x0F]], np.uint8)
    assert orc.norm_code_row_bytes(8, 4) == 1
    W, W16 = orc.normalized_decode(f, idx, cb, None, codes, lut, 4)
    expect = np.array([[0.5, 1.0, -1.5, 0.25, -12.0, 2.0, 4.0, 8.0],
                       [-0.75, 0.125, -0.75, 0.125, 1.0, 2.0, 1.0, 2.0]])
    assert np.array_equal(W, expect)
    assert np.array_equal(W16.view(np.float16).astype(np.float64), expect)
    x = np.array([[1, 1, 1, 1, 1, 1, 1, 1], [2, 0, 0, 0, 0, 0, 0, -1]], np.float16)
    Y, A = orc.normalized_gemm(f, idx, cb, None, codes, lut, 4, x)
    assert Y.tolist() == [[2.25, 4.75], [-7.0, -3.5]]
    assert A.tolist() == [[29.25, 7.75], [9.0, 3.5]]


def test_normalized_decode_int8_rounds_once_and_unit_lut_is_plain_decode():
    """int8 codebook: w = fp16(scale * c * norm), one rounding of the exact product: scale 0.0999755859375
    (0x2E66 = 819/8192), c = 127, norm 1.4140625 (= 181/128): exact 819 * 127 * 181 / 2^20 = 18826353 / 1048576
    = 17.9542..., between the binary16 neighbours 17.953125 and 17.96875 and nearer the first.  With every
    table entry 1.0 the result is the plain decode."""
    f = orc.Fmt(N=1, K=2, d=1, b=1, Br=1, Bc=2, int8=True)
    cb = np.array([127, -128], np.int8)
    scale = np.array([0x2E66], np.uint16)
    idx = orc.pack(f, np.array([[0, 1]], np.int32))
    lut = np.full((1, 16), 1.4140625, np.float16)
    W, W16 = orc.normalized_decode(f, idx, cb, scale, np.array([[5]], np.uint8), lut, 2)
    assert Fraction(float(W[0, 0])) == Fraction(18826353, 1048576)
    assert Fraction(float(W[0, 1])) == Fraction(819 * -128 * 181, 1048576)
    assert float(W16.view(np.float16)[0, 0]) == 17.953125
    spec = vq_synth.LayerSpec("n", N=6, K=32, d=2, b=3, Br=3, Bc=16, int8=True)
    fo = orc.Fmt(spec.N, spec.K, spec.d, spec.b, spec.Br, spec.Bc, spec.int8)
    L = vq_synth.make_layer(spec, fo.stride, 3)
    ones = np.ones((fo.n_blocks, 16), np.float16)
    codes = vq_synth.random_bytes(1, 2, spec.N * orc.norm_code_row_bytes(spec.K, 8)).reshape(spec.N, -1)
    _, plain = orc.decode(fo, L.idx, L.cb, L.scale, exact=False)
    _, normed = orc.normalized_decode(fo, L.idx, L.cb, L.scale, codes, ones, 8)
    assert np.array_equal(plain, normed)
