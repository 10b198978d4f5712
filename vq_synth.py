"""Seeded synthetic inputs for the VQ-decode linear layer.

This module only draws numbers: random bytes for the packed index stream, random codebook
entries, scales and activations, with the shapes and value distributions of the benchmark
configurations.  It contains none of the method's arithmetic (no bit unpacking, no look-up, no
products); the row stride of the index stream is supplied by the caller.  Both the CPU oracle's
tests and the CUDA library's tests and benchmark draw their inputs from here.

Random source: a counter-based splitmix64 (the i-th 64-bit draw of a stream is a pure function
of (seed, stream id, i)), uniform doubles from the top 53 bits, normals by Box-Muller in fp64,
one round-to-nearest-even conversion to binary16 (numpy astype).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def raw_u64(seed: int, stream: int, n: int) -> np.ndarray:
    """n 64-bit draws of stream `stream` under `seed` (wrapping uint64 arithmetic)."""
    with np.errstate(over="ignore"):
        base = _mix(np.array([(seed * 0x100000001B3 + stream * 0x9E3779B1 + 0x1234567) % (1 << 64)], dtype=np.uint64))[0]
        ctr = (np.arange(1, n + 1, dtype=np.uint64)) * _GOLDEN + base
        return _mix(ctr)


def uniform01(seed: int, stream: int, n: int) -> np.ndarray:
    return (raw_u64(seed, stream, n) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normal(seed: int, stream: int, n: int) -> np.ndarray:
    m = (n + 1) // 2
    u = uniform01(seed, stream, 2 * m)
    u1 = 1.0 - u[:m]  # (0, 1]
    u2 = u[m:]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.concatenate([r * np.cos(2 * np.pi * u2), r * np.sin(2 * np.pi * u2)])
    return out[:n]


def random_bytes(seed: int, stream: int, n: int) -> np.ndarray:
    return raw_u64(seed, stream, (n + 7) // 8).view(np.uint8)[:n].copy()


@dataclass(frozen=True)
class LayerSpec:
    """Shape and format of one synthetic VQ layer (N out x K in)."""

    name: str
    N: int
    K: int
    d: int          # VQ dimension
    b: int          # index bits
    Br: int         # block rows
    Bc: int         # block cols
    int8: bool      # int8 codebook with one fp16 scale per block, else fp16 codebook; 2 = int4 codebook, scale per row and 128 columns
    cb_sigma: float = 0.02                 # fp16 codebook entries ~ N(0, sigma^2)
    scale_range: tuple = (0.0005, 0.002)   # int8: block scale ~ U(lo, hi)

    @property
    def entries(self) -> int:
        return 1 << self.b

    @property
    def n_blocks(self) -> int:
        return (self.N // self.Br) * (self.K // self.Bc)

    @property
    def n_weights(self) -> int:
        return self.N * self.K


@dataclass
class Layer:
    spec: LayerSpec
    stride: int
    idx: np.ndarray            # uint8 [N][stride]
    cb: np.ndarray             # float16 or int8, [n_blocks][entries][d]
    scale: np.ndarray | None   # float16 [n_blocks] or None
    x: dict = field(default_factory=dict)


def make_layer(spec: LayerSpec, stride: int, seed: int, layer_id: int = 0) -> Layer:
    """Draw one layer.  Uniform random bytes in the index stream are uniform random indices
    (every b-bit pattern is a valid entry); padding bytes are random too and must be ignored."""
    s0 = 16 * layer_id
    idx = random_bytes(seed, s0 + 1, spec.N * stride).reshape(spec.N, stride)
    n_cb = spec.n_blocks * spec.entries * spec.d
    if int(spec.int8) == 2:   # int4 codebook (two nibbles per byte), scale per row and group of 128 columns
        cb = random_bytes(seed, s0 + 2, n_cb // 2).reshape(spec.n_blocks, spec.entries * spec.d // 2)
        scale = (0.001 + 0.003 * uniform01(seed, s0 + 3, spec.N * (spec.K // 128))).astype(np.float16).reshape(spec.N, spec.K // 128)
    elif spec.int8:
        cb = (raw_u64(seed, s0 + 2, n_cb) % np.uint64(255)).astype(np.int64) - 127
        cb = cb.astype(np.int8).reshape(spec.n_blocks, spec.entries, spec.d)
        lo, hi = spec.scale_range
        scale = (lo + (hi - lo) * uniform01(seed, s0 + 3, spec.n_blocks)).astype(np.float16)
    else:
        cb = (spec.cb_sigma * normal(seed, s0 + 2, n_cb)).astype(np.float16)
        cb = cb.reshape(spec.n_blocks, spec.entries, spec.d)
        scale = None
    return Layer(spec, stride, idx, cb, scale)


def make_norm(spec: LayerSpec, block_cols: int, seed: int, layer_id: int = 0):
    """Block-wise normalisation inputs of one layer: uniform random 4-bit codes per row and sub-row of
    `block_cols` columns (uint8 [N][ceil(K / block_cols / 2)], two codes per byte) and, per codebook block,
    16 scales drawn uniformly from [0.25, 4) as float16 (the decoder treats the table as opaque values)."""
    s0 = 16 * layer_id
    row_bytes = (spec.K // block_cols + 1) // 2
    codes = random_bytes(seed, s0 + 10, spec.N * row_bytes).reshape(spec.N, row_bytes)
    lut = (0.25 + 3.75 * uniform01(seed, s0 + 11, spec.n_blocks * 16)).astype(np.float16).reshape(spec.n_blocks, 16)
    return codes, lut


def make_x(spec: LayerSpec, seed: int, batch: int, layer_id: int = 0) -> np.ndarray:
    """Activations X[batch][K] ~ N(0,1) as float16."""
    return normal(seed, 16 * layer_id + 4, batch * spec.K).astype(np.float16).reshape(batch, spec.K)


def _set(prefix, shapes, **fmt):
    return [LayerSpec(name=f"{prefix}.{nm}", N=n, K=k, **fmt) for nm, n, k in shapes]


# The five benchmark configurations (seeded synthetic layers with LLM projection shapes) and, last,
# the paper's deployed format on the shapes of the model it was deployed for.
CONFIGS = {
    # single 4096x4096 layer, 2-D VQ, 4-bit indices, 16-entry fp16 codebook per 1x1024 block
    "cfg1": dict(seed=0, batches=(1,), layers=_set("l4096", [("w", 4096, 4096)],
                 d=2, b=4, Br=1, Bc=1024, int8=False, cb_sigma=0.02)),
    # same layer, 1-D mobile-LUT style: 16-entry int8 codebook + fp16 scale per 1x2048 block
    "cfg2": dict(seed=1, batches=(1,), layers=_set("l4096", [("w", 4096, 4096)],
                 d=1, b=4, Br=1, Bc=2048, int8=True)),
    # Llama-2-7B-shaped layer set, 2-D, 6-bit indices, 64-entry fp16 codebook per 128x128 block
    "cfg3": dict(seed=2, batches=(1,), layers=_set("llama2_7b", [
                 ("q", 4096, 4096), ("k", 4096, 4096), ("v", 4096, 4096), ("o", 4096, 4096),
                 ("gate", 11008, 4096), ("up", 11008, 4096), ("down", 4096, 11008)],
                 d=2, b=6, Br=128, Bc=128, int8=False, cb_sigma=0.02)),
    # Llama-2-13B-shaped layer set, 4-D, 8-bit indices, 256-entry fp16 codebook per 256x512 block
    "cfg4": dict(seed=3, batches=(1, 8), layers=_set("llama2_13b", [
                 ("q", 5120, 5120), ("k", 5120, 5120), ("v", 5120, 5120), ("o", 5120, 5120),
                 ("gate", 13824, 5120), ("up", 13824, 5120), ("down", 5120, 13824)],
                 d=4, b=8, Br=256, Bc=512, int8=False, cb_sigma=0.015)),
    # Llama-2-70B-shaped (GQA) layer set, 2-D, 4-bit indices, int8 codebook + scale per 1x2048
    "cfg5": dict(seed=4, batches=(1, 2, 4, 8, 16), layers=_set("llama2_70b", [
                 ("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
                 ("gate", 28672, 8192), ("up", 28672, 8192), ("down", 8192, 28672)],
                 d=2, b=4, Br=1, Bc=2048, int8=True)),
    # Llama-3-8B-shaped (GQA) layer set in the format the paper deploys (Sec. 4.1, Table 1, App. B):
    # 2-D, 6-bit indices, int8 codebook + scale per group of 8192 weights of at most 256 columns
    "llama3_8b": dict(seed=5, batches=(1, 8), layers=_set("llama3_8b", [
                 ("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
                 ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)],
                 d=2, b=6, Br=32, Bc=256, int8=True)),
    # the same shapes with INT4 codebooks (Sec. 4.2: 2-D, 3 bits per dimension, blocks of 4096 weights,
    # entries quantized to 4 bits, one scale per row and group of 128 columns)
    "llama3_8b_int4cb": dict(seed=6, batches=(1, 8), layers=_set("llama3_8b_i4", [
                 ("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
                 ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)],
                 d=2, b=6, Br=32, Bc=128, int8=2)),
    # the same shapes at the 2.75-bit row of the paper's table of VQ configurations (App. on VQ
    # configurations): 2-D, 2.5 bits per dimension (5-bit indices), 8-bit codebooks, blocks of 4 x 256
    "llama3_8b_d2b5_4x256": dict(seed=7, batches=(1, 8), layers=_set("llama3_8b_b5", [
                 ("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
                 ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336)],
                 d=2, b=5, Br=4, Bc=256, int8=True)),
}


def make_int4g128(N: int, K: int, seed: int, layer_id: int = 0):
    """Uniform INT4 group-128 yard-stick layer: random nibbles, scales ~ U(0.001, 0.004)."""
    s0 = 16 * layer_id
    q = random_bytes(seed, s0 + 8, N * (K // 2)).reshape(N, K // 2)
    scale = (0.001 + 0.003 * uniform01(seed, s0 + 9, N * (K // 128))).astype(np.float16).reshape(N, K // 128)
    return q, scale
