"""ctypes front-end of the CPU oracle (oracle/vq_oracle.cpp).

TEST INFRASTRUCTURE ONLY: the parity reference and the timed CPU baseline.  Nothing in the
product package imports this module, and this module imports nothing from the product.

All arrays are numpy; binary16 data travels as uint16 bit patterns or np.float16 views.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vq_oracle.cpp")
_LIB = os.path.join(_HERE, "libvq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-o", _LIB, _SRC]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        c_ll, c_i, c_d, c_p = ctypes.c_longlong, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        L.ref_bpv.restype = c_d
        L.ref_bpv.argtypes = [c_i, c_i, c_i, c_ll]
        L.ref_bpv_uniform.restype = c_d
        L.ref_bpv_uniform.argtypes = [c_i, c_i, c_i]
        L.ref_row_stride_bytes.restype = c_ll
        L.ref_row_stride_bytes.argtypes = [c_i, c_i, c_i]
        L.ref_f64_to_f16.restype = ctypes.c_uint16
        L.ref_f64_to_f16.argtypes = [c_d]
        L.ref_f16_to_f64.restype = c_d
        L.ref_f16_to_f64.argtypes = [ctypes.c_uint16]
        L.ref_pack.restype = None
        L.ref_pack.argtypes = [c_i, c_i, c_i, c_i, c_p, c_p, c_ll]
        L.ref_unpack.restype = None
        L.ref_unpack.argtypes = [c_i, c_i, c_i, c_i, c_p, c_ll, c_p]
        L.ref_decode.restype = None
        L.ref_decode.argtypes = [c_i] * 7 + [c_p, c_ll, c_p, c_p, c_p, c_p]
        L.ref_gemm.restype = None
        L.ref_gemm.argtypes = [c_i] * 7 + [c_p, c_ll, c_p, c_p, c_p, c_i, c_p, c_ll, c_p, c_p, c_i]
        L.ref_dense_gemm.restype = None
        L.ref_dense_gemm.argtypes = [c_i, c_i, c_p, c_p, c_i, c_p]
        L.ref_int4g128_gemm.restype = None
        L.ref_int4g128_gemm.argtypes = [c_i, c_i, c_p, c_p, c_p, c_i, c_p, c_p, c_i]
        L.ref_hardware_threads.restype = c_i
        L.ref_hardware_threads.argtypes = []
        _lib = L
    return _lib


@dataclass(frozen=True)
class Fmt:
    """One VQ-compressed matrix: N x K weights, VQ dim d, b index bits, Br x Bc blocks."""

    N: int
    K: int
    d: int
    b: int
    Br: int
    Bc: int
    int8: bool   # False: fp16 codebook; True: int8 codebook + scale per block; 2: int4 codebook + scale per row and 128 columns

    @property
    def entries(self) -> int:
        return 1 << self.b

    @property
    def n_blocks(self) -> int:
        return (self.N // self.Br) * (self.K // self.Bc)

    @property
    def stride(self) -> int:
        return row_stride_bytes(self.K, self.d, self.b)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    return a.view(np.uint16) if a.dtype == np.float16 else a.astype(np.uint16, copy=False)


def bpv(k: int, d: int, b_c: int, l: int) -> float:
    return _load().ref_bpv(k, d, b_c, l)


def bpv_uniform(bits: int, scale_bits: int, group: int) -> float:
    return _load().ref_bpv_uniform(bits, scale_bits, group)


def row_stride_bytes(K: int, d: int, b: int) -> int:
    return _load().ref_row_stride_bytes(K, d, b)


def f64_to_f16_bits(x: float) -> int:
    return _load().ref_f64_to_f16(float(x))


def f16_bits_to_f64(h: int) -> float:
    return _load().ref_f16_to_f64(int(h))


def pack(f: Fmt, I: np.ndarray, fill: np.ndarray | None = None) -> np.ndarray:
    """Indices I[N][K/d] (uint8) -> packed rows uint8[N][stride]; `fill` pre-sets padding."""
    I = np.ascontiguousarray(I, dtype=np.uint8)
    assert I.shape == (f.N, f.K // f.d)
    out = np.zeros((f.N, f.stride), np.uint8) if fill is None else np.array(fill, dtype=np.uint8, copy=True)
    assert out.shape == (f.N, f.stride) and out.flags.c_contiguous
    _load().ref_pack(f.N, f.K, f.d, f.b, _p(I), _p(out), f.stride)
    return out


def unpack(f: Fmt, idx: np.ndarray) -> np.ndarray:
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    assert idx.size == f.N * f.stride
    I = np.empty((f.N, f.K // f.d), np.uint8)
    _load().ref_unpack(f.N, f.K, f.d, f.b, _p(idx), f.stride, _p(I))
    return I


def _check_layer(f: Fmt, idx, cb, scale):
    idx = np.ascontiguousarray(idx, dtype=np.uint8)
    assert idx.size == f.N * f.stride
    if int(f.int8) == 2:      # int4 codebook, scales per (row, 128-column group)
        cb = np.ascontiguousarray(cb, dtype=np.uint8)
        scale = _u16(scale)
        assert f.K % 128 == 0 and scale.size == f.N * (f.K // 128)
        assert cb.size == f.n_blocks * f.entries * f.d // 2
        return idx, cb, scale
    if f.int8:
        cb = np.ascontiguousarray(cb, dtype=np.int8)
        scale = _u16(scale)
        assert scale.size == f.n_blocks
    else:
        cb = _u16(cb)
        scale = None
    assert cb.size == f.n_blocks * f.entries * f.d
    return idx, cb, scale


def decode(f: Fmt, idx, cb, scale=None, exact: bool = True, half: bool = True):
    """Returns (W_exact float64 [N][K] or None, W16 uint16 [N][K] or None)."""
    idx, cb, scale = _check_layer(f, idx, cb, scale)
    We = np.empty((f.N, f.K), np.float64) if exact else None
    Wh = np.empty((f.N, f.K), np.uint16) if half else None
    _load().ref_decode(f.N, f.K, f.d, f.b, f.Br, f.Bc, int(f.int8), _p(idx), f.stride, _p(cb),
                       _p(scale), _p(We), _p(Wh))
    return We, Wh


def gemm(f: Fmt, idx, cb, scale, X, rows=None, threads: int = 1):
    """Y[m][r], A[m][r] in float64 for X[batch][K] (float16).  rows: optional row subset."""
    idx, cb, scale = _check_layer(f, idx, cb, scale)
    X = _u16(np.atleast_2d(X))
    batch = X.shape[0]
    assert X.shape[1] == f.K
    if rows is not None:
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        n_out = rows.size
    else:
        n_out = f.N
    Y = np.empty((batch, n_out), np.float64)
    A = np.empty((batch, n_out), np.float64)
    _load().ref_gemm(f.N, f.K, f.d, f.b, f.Br, f.Bc, int(f.int8), _p(idx), f.stride, _p(cb),
                     _p(scale), _p(X), batch, _p(rows), n_out, _p(Y), _p(A), int(threads))
    return Y, A


# ---- block-wise data normalisation (App. on blockwise data normalization) ---------------------------
# The quantizer divides every sub-row of `block_cols` columns by a scale before clustering and stores the
# scale as a 4-bit integer on a log2 grid; the decoder multiplies the looked-up values by the inverse.
# What the decoder needs is, per codebook block, the 16 values the 4-bit code can stand for: a table
# lut[blk][16] (binary16) and a code per (row, sub-row).  The grid itself (norm_lut_log2 below) belongs
# to the quantizer; its printed formula is garbled in the paper, the reading taken is
#   value(s) = 2^(a*s + z),  s = 0..15,  a = step of the group, z = floating-point offset,
# rounded once to binary16.  norm_lut_log2 is "parity unpinned" as to the paper's intent (pinned by
# mathematics only); the decode functions below take the table as given and are pinned by hand values.
def norm_lut_log2(a: float, z: float) -> np.ndarray:
    """The 16 scales of one group on the log2 grid: float16 [16]."""
    return np.array([2.0 ** (a * s + z) for s in range(16)], dtype=np.float64).astype(np.float16)


def norm_code_row_bytes(K: int, block_cols: int) -> int:
    """Bytes of one row of 4-bit codes (two per byte, low nibble first)."""
    return (K // block_cols + 1) // 2


def norm_factors(f: Fmt, codes, lut, block_cols: int) -> np.ndarray:
    """F[n][k] (float64) = lut[blk(n, k)][code(n, k // block_cols)]; blk ordered as the codebooks are."""
    assert f.Bc % block_cols == 0 and block_cols % f.d == 0
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(f.N, norm_code_row_bytes(f.K, block_cols))
    lut = _u16(lut).view(np.float16).astype(np.float64).reshape(f.n_blocks, 16)
    F = np.empty((f.N, f.K), np.float64)
    for n in range(f.N):
        for j in range(f.K // block_cols):
            byte = int(codes[n, j // 2])
            code = (byte >> 4) if (j % 2) else (byte & 15)
            k0 = j * block_cols
            blk = (n // f.Br) * (f.K // f.Bc) + k0 // f.Bc
            F[n, k0:k0 + block_cols] = lut[blk, code]
    return F


def normalized_decode(f: Fmt, idx, cb, scale, codes, lut, block_cols: int):
    """(W exact float64, W16 uint16): the decoded weight times its sub-row's scale; the product of at most
    three short significands (30 bits) is exact in float64 and rounded once to binary16."""
    We, _ = decode(f, idx, cb, scale, exact=True, half=False)
    Wn = We * norm_factors(f, codes, lut, block_cols)
    return Wn, Wn.astype(np.float16).view(np.uint16)


def normalized_gemm(f: Fmt, idx, cb, scale, codes, lut, block_cols: int, X, rows=None):
    """Y[m][r], A[m][r] (float64, k ascending) on the normalised weights."""
    Wn, _ = normalized_decode(f, idx, cb, scale, codes, lut, block_cols)
    if rows is not None:
        Wn = Wn[np.asarray(rows)]
    Xd = _u16(np.atleast_2d(X)).view(np.float16).astype(np.float64)
    Y = np.empty((Xd.shape[0], Wn.shape[0]), np.float64)
    A = np.empty_like(Y)
    for m in range(Xd.shape[0]):
        P = Wn * Xd[m][None, :]
        Y[m] = np.cumsum(P, axis=1)[:, -1]      # left to right over k
        A[m] = np.abs(P).sum(axis=1)
    return Y, A


def dense_gemm(W: np.ndarray, X) -> np.ndarray:
    W = np.ascontiguousarray(W, dtype=np.float64)
    X = _u16(np.atleast_2d(X))
    N, K = W.shape
    Y = np.empty((X.shape[0], N), np.float64)
    _load().ref_dense_gemm(N, K, _p(W), _p(X), X.shape[0], _p(Y))
    return Y


def int4g128_gemm(q: np.ndarray, scale, X, threads: int = 1):
    q = np.ascontiguousarray(q, dtype=np.uint8)
    N, K = q.shape[0], q.shape[1] * 2
    scale = _u16(scale)
    assert scale.size == N * (K // 128)
    X = _u16(np.atleast_2d(X))
    Y = np.empty((X.shape[0], N), np.float64)
    A = np.empty((X.shape[0], N), np.float64)
    _load().ref_int4g128_gemm(N, K, _p(q), _p(scale), _p(X), X.shape[0], _p(Y), _p(A), int(threads))
    return Y, A


def unpack_uniform(kind: str, src: np.ndarray, scale=None) -> np.ndarray:
    """Uniformly quantized weights expanded to binary16, the yard-sticks of the transfer + decode
    experiment (App. B; Sec. 2.1 symmetric uniform quantizer w = s * q):
      "fp16":     the weights themselves, copied;
      "int8row":  signed 8-bit q [N][K], one binary16 scale per row;
      "int4g128": unsigned nibbles [N][K/2] (low nibble = lower column) meaning q - 8, one binary16
                  scale per row and group of 128 columns.
    The product s * q is exact in float64 (11-bit by 8-bit significands); it is rounded once to
    binary16 (round to nearest even), as decode() does for int8 codebooks."""
    if kind == "fp16":
        return np.array(src, dtype=np.float16, copy=True)
    if kind == "int8row":
        q = np.asarray(src, dtype=np.int8).astype(np.float64)
        s = np.asarray(scale, dtype=np.float16).astype(np.float64).reshape(-1, 1)
        return (q * s).astype(np.float16)
    if kind == "int4g128":
        b = np.asarray(src, dtype=np.uint8)
        N, K = b.shape[0], b.shape[1] * 2
        q = np.empty((N, K), np.float64)
        q[:, 0::2] = (b & 15).astype(np.float64) - 8.0
        q[:, 1::2] = (b >> 4).astype(np.float64) - 8.0
        s = np.asarray(scale, dtype=np.float16).astype(np.float64).reshape(N, K // 128)
        return (q * np.repeat(s, 128, axis=1)).astype(np.float16)
    raise ValueError(kind)


def assign(f: Fmt, W: np.ndarray, cb, scale=None, hdiag=None) -> np.ndarray:
    """E-step / VQ_quant (Sec. 3, Eq. 5): for every d-vector x of W (d adjacent columns of one row)
    the index m of the centroid of its block that minimises (x - c_m)^T D (x - c_m), D = the diagonal
    weights of the vector's columns (hdiag[k] = 1 / [H^-1]_kk; None = identity, plain K-means).
    Returns I[N][K/d] uint8.

    The decision is taken in binary32, the arithmetic of the CUDA kernel, so that both sides break
    near-ties alike: per coordinate t  diff = x_t - c_t,  sq = diff * diff,  term = D_t * sq, every
    operation rounded to binary32, the terms added left to right; the lowest index wins among equal
    distances.  int8 centroids are c = scale * c_int (exact in binary32)."""
    W = np.ascontiguousarray(W, dtype=np.float16)
    assert W.shape == (f.N, f.K)
    assert int(f.int8) != 2, "the E-step is defined here for fp16 and int8 codebooks"
    e, d = f.entries, f.d
    if f.int8:
        C = np.asarray(cb, dtype=np.int8).reshape(f.n_blocks, e, d).astype(np.float32)
        C = C * np.asarray(scale, dtype=np.float16).astype(np.float32).reshape(f.n_blocks, 1, 1)
    else:
        C = np.asarray(cb, dtype=np.float16).reshape(f.n_blocks, e, d).astype(np.float32)
    D = np.ones(f.K, np.float32) if hdiag is None else np.ascontiguousarray(hdiag, dtype=np.float32)
    assert D.shape == (f.K,)
    I = np.empty((f.N, f.K // d), np.uint8)
    bpr = f.K // f.Bc
    for br in range(f.N // f.Br):
        for bc in range(bpr):
            r0, k0 = br * f.Br, bc * f.Bc
            X = W[r0:r0 + f.Br, k0:k0 + f.Bc].astype(np.float32).reshape(f.Br, f.Bc // d, d)
            Dv = D[k0:k0 + f.Bc].reshape(f.Bc // d, d)
            Cb = C[br * bpr + bc]                                   # [e][d]
            acc = None
            for t in range(d):
                diff = X[:, :, t, None] - Cb[None, None, :, t]       # binary32 throughout
                term = Dv[None, :, t, None] * (diff * diff)
                acc = term if acc is None else acc + term
            assert acc.dtype == np.float32
            I[r0:r0 + f.Br, k0 // d:(k0 + f.Bc) // d] = np.argmin(acc, axis=2)   # first minimum = lowest index
    return I


def sqnr_db(W: np.ndarray, Q: np.ndarray) -> float:
    """Signal-to-quantization-noise ratio in dB (Sec. 2.2): 10 log10( E[W^2] / E[(W - Q)^2] )."""
    W = np.asarray(W, dtype=np.float64)
    Q = np.asarray(Q, dtype=np.float64)
    return float(10.0 * np.log10(np.mean(W * W) / np.mean((W - Q) ** 2)))


def hardware_threads() -> int:
    return _load().ref_hardware_threads()
