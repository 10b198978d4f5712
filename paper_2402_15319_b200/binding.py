"""ctypes binding with the same names as include/vq.h.  Argument marshalling only: every step
of the computation runs in the CUDA library.  Tensors are torch CUDA tensors (device memory and
streams are torch's); there is no CPU fallback — a missing library is an error."""
from __future__ import annotations

import ctypes
import functools
import os
from dataclasses import dataclass

VQ_CB_FP16, VQ_CB_INT8_SCALED, VQ_CB_INT4_G128 = 0, 1, 2
VQ_IMPL_AUTO, VQ_IMPL_GENERIC, VQ_IMPL_TUNED, VQ_IMPL_STREAM = 0, 1, 2, 3

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libvq_b200.so")
_lib = None


class VQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {vq_status_string(code)}")


class _CFormat(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_rows", "k_cols", "vq_dim", "index_bits", "block_rows", "block_cols", "cb_type")]


class _CPackInfo(ctypes.Structure):
    _fields_ = [("entries", ctypes.c_int32), ("codebook_bits", ctypes.c_int32),
                ("indices_per_row", ctypes.c_int64), ("row_stride_bytes", ctypes.c_int64),
                ("index_bytes", ctypes.c_int64), ("n_blocks", ctypes.c_int64),
                ("codebook_bytes_per_block", ctypes.c_int64), ("codebook_bytes", ctypes.c_int64),
                ("scale_bytes", ctypes.c_int64), ("total_bytes", ctypes.c_int64),
                ("bpv_paper", ctypes.c_double), ("bpv_stored", ctypes.c_double)]


@dataclass(frozen=True)
class VQFormat:
    n_rows: int
    k_cols: int
    vq_dim: int
    index_bits: int
    block_rows: int
    block_cols: int
    cb_type: int

    def c(self) -> _CFormat:
        return _c_format(self)


@functools.lru_cache(maxsize=4096)
def _c_format(f: "VQFormat") -> _CFormat:
    # one struct per distinct format, reused by every call (the library only reads it)
    return _CFormat(f.n_rows, f.k_cols, f.vq_dim, f.index_bits, f.block_rows, f.block_cols, f.cb_type)


@dataclass(frozen=True)
class PackInfo:
    entries: int
    codebook_bits: int
    indices_per_row: int
    row_stride_bytes: int
    index_bytes: int
    n_blocks: int
    codebook_bytes_per_block: int
    codebook_bytes: int
    scale_bytes: int
    total_bytes: int
    bpv_paper: float
    bpv_stored: float


_SIGNATURES = {
    "vq_pack_info": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "vq_workspace_bytes": (ctypes.c_size_t, [ctypes.c_void_p, ctypes.c_int]),
    "vq_workspace_bytes_host": (ctypes.c_size_t, [ctypes.c_void_p, ctypes.c_int]),
    "vq_decode_weights": (ctypes.c_int, [ctypes.c_void_p] * 6),
    "vq_norm_info": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]),
    "vq_decode_weights_normalized": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]),
    "vq_gemm_small_batch_normalized": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                                       ctypes.c_int, ctypes.c_void_p]),
    "vq_gemv": (ctypes.c_int, [ctypes.c_void_p] * 7 + [ctypes.c_size_t, ctypes.c_void_p]),
    "vq_gemm_small_batch": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "vq_gemm_small_batch_impl": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_int]),
    "vq_gemm_small_batch_grouped": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                                                   ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "vq_grouped_kernel_launches": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]),
    "vq_gemm_small_batch_grouped_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
                                                        ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "vq_workspace_bytes_grouped_host": (ctypes.c_size_t, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]),
    "vq_gemm_small_batch_host": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "vq_gemm_small_batch_host_static": (ctypes.c_int, [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_void_p]),
    "vq_static_scratch_bytes": (ctypes.c_size_t, []),
    "vq_int4g128_gemm_small_batch": (ctypes.c_int, [ctypes.c_int32, ctypes.c_int32] + [ctypes.c_void_p] * 4 + [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]),
    "vq_int4g128_workspace_bytes": (ctypes.c_size_t, [ctypes.c_int32, ctypes.c_int]),
    "vq_assign_indices": (ctypes.c_int, [ctypes.c_void_p] * 7),
    "vq_unpack_uniform": (ctypes.c_int, [ctypes.c_int, ctypes.c_int32, ctypes.c_int32] + [ctypes.c_void_p] * 4),
    "vq_device_wait_failures": (ctypes.c_int, [ctypes.c_void_p]),
    "vq_probe_decode_loop": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t,
                                            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "vq_probe_read": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]),
    "vq_status_string": (ctypes.c_char_p, [ctypes.c_int]),
}


def lib_path() -> str:
    return _LIB_PATH


def exported_symbols():
    return sorted(_SIGNATURES)


def load():
    """Load libvq_b200.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2402_15319_b200.build`")
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def vq_status_string(code: int) -> str:
    return load().vq_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise VQError(code, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def vq_pack_info(fmt: VQFormat) -> PackInfo:
    c, out = fmt.c(), _CPackInfo()
    _check(load().vq_pack_info(ctypes.byref(c), ctypes.byref(out)), "vq_pack_info")
    return PackInfo(*[getattr(out, n) for n, _ in _CPackInfo._fields_])


def vq_workspace_bytes(fmt: VQFormat, batch: int) -> int:
    c = fmt.c()
    return load().vq_workspace_bytes(ctypes.byref(c), int(batch))


def vq_workspace_bytes_host(fmt: VQFormat, batch: int) -> int:
    c = fmt.c()
    return load().vq_workspace_bytes_host(ctypes.byref(c), int(batch))


def vq_decode_weights(fmt: VQFormat, d_idx, d_cb, d_scale, d_W, stream=None) -> None:
    c = fmt.c()
    _check(load().vq_decode_weights(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_W),
                                    _stream(stream)), "vq_decode_weights")


class _CNormInfo(ctypes.Structure):
    _fields_ = [("code_row_bytes", ctypes.c_size_t), ("codes_bytes", ctypes.c_size_t), ("lut_bytes", ctypes.c_size_t)]


def vq_norm_info(fmt: VQFormat, norm_block_cols: int):
    """(code_row_bytes, codes_bytes, lut_bytes) of the block-wise normalisation buffers."""
    c = fmt.c()
    out = _CNormInfo()
    _check(load().vq_norm_info(ctypes.byref(c), int(norm_block_cols), ctypes.byref(out)), "vq_norm_info")
    return int(out.code_row_bytes), int(out.codes_bytes), int(out.lut_bytes)


def vq_decode_weights_normalized(fmt: VQFormat, d_idx, d_cb, d_scale, d_norm_codes, d_norm_lut, norm_block_cols: int, d_W,
                                 stream=None) -> None:
    c = fmt.c()
    _check(load().vq_decode_weights_normalized(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_norm_codes),
                                               _ptr(d_norm_lut), int(norm_block_cols), _ptr(d_W), _stream(stream)),
           "vq_decode_weights_normalized")


def vq_gemm_small_batch_normalized(fmt: VQFormat, d_idx, d_cb, d_scale, d_norm_codes, d_norm_lut, norm_block_cols: int, d_X, d_Y,
                                   batch: int, stream=None) -> None:
    c = fmt.c()
    _check(load().vq_gemm_small_batch_normalized(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_norm_codes),
                                                 _ptr(d_norm_lut), int(norm_block_cols), _ptr(d_X), _ptr(d_Y), int(batch),
                                                 _stream(stream)), "vq_gemm_small_batch_normalized")


def vq_gemv(fmt: VQFormat, d_idx, d_cb, d_scale, d_x, d_y, d_ws, stream=None) -> None:
    c = fmt.c()
    _check(load().vq_gemv(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_x), _ptr(d_y),
                          _ptr(d_ws), d_ws.numel() * d_ws.element_size(), _stream(stream)), "vq_gemv")


def vq_gemm_small_batch(fmt: VQFormat, d_idx, d_cb, d_scale, d_X, d_Y, batch: int, d_ws, stream=None) -> None:
    c = fmt.c()
    _check(load().vq_gemm_small_batch(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_X),
                                      _ptr(d_Y), int(batch), _ptr(d_ws), d_ws.numel() * d_ws.element_size(),
                                      _stream(stream)), "vq_gemm_small_batch")


class _CGroupMember(ctypes.Structure):
    _fields_ = [("d_idx", ctypes.c_void_p), ("d_cb", ctypes.c_void_p), ("d_scale", ctypes.c_void_p),
                ("d_Y", ctypes.c_void_p), ("n_rows", ctypes.c_int32)]


def vq_gemm_small_batch_grouped(fmt: VQFormat, members, d_X, batch: int, d_ws, stream=None) -> None:
    """members: sequence of (d_idx, d_cb, d_scale, d_Y, n_rows); fmt.n_rows = the sum of the members' rows."""
    arr = (_CGroupMember * len(members))()
    for i, (idx, cb, sc, Y, n) in enumerate(members):
        arr[i] = _CGroupMember(_ptr(idx), _ptr(cb), _ptr(sc), _ptr(Y), int(n))
    c = fmt.c()
    _check(load().vq_gemm_small_batch_grouped(ctypes.byref(c), arr, len(members), _ptr(d_X), int(batch), _ptr(d_ws),
                                              d_ws.numel() * d_ws.element_size(), _stream(stream)),
           "vq_gemm_small_batch_grouped")


def vq_gemm_small_batch_grouped_host(fmt: VQFormat, members, h_X, batch: int, d_ws, stream=None) -> None:
    """members: sequence of (d_idx, d_cb, d_scale, h_Y, n_rows) with HOST outputs; h_X a host tensor (pinned for
    the direct path).  Synchronise before reading the outputs."""
    arr = (_CGroupMember * len(members))()
    for i, (idx, cb, sc, Y, n) in enumerate(members):
        arr[i] = _CGroupMember(_ptr(idx), _ptr(cb), _ptr(sc), _ptr(Y), int(n))
    c = fmt.c()
    _check(load().vq_gemm_small_batch_grouped_host(ctypes.byref(c), arr, len(members), _ptr(h_X), int(batch), _ptr(d_ws),
                                                   d_ws.numel() * d_ws.element_size(), _stream(stream)),
           "vq_gemm_small_batch_grouped_host")


def vq_workspace_bytes_grouped_host(fmt: VQFormat, n_members: int, batch: int) -> int:
    c = fmt.c()
    return load().vq_workspace_bytes_grouped_host(ctypes.byref(c), int(n_members), int(batch))


def vq_grouped_kernel_launches(fmt: VQFormat, n_members: int, batch: int) -> int:
    c = fmt.c()
    return load().vq_grouped_kernel_launches(ctypes.byref(c), int(n_members), int(batch))


def vq_gemm_small_batch_impl(fmt: VQFormat, d_idx, d_cb, d_scale, d_X, d_Y, batch: int, d_ws, impl: int,
                             stream=None) -> None:
    c = fmt.c()
    _check(load().vq_gemm_small_batch_impl(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(d_X),
                                           _ptr(d_Y), int(batch), _ptr(d_ws),
                                           d_ws.numel() * d_ws.element_size(), _stream(stream), int(impl)),
           "vq_gemm_small_batch_impl")


def vq_gemm_small_batch_host(fmt: VQFormat, d_idx, d_cb, d_scale, h_X, h_Y, batch: int, d_ws, stream=None) -> None:
    """h_X / h_Y are host tensors (pinned for asynchronous copies); synchronise before reading h_Y."""
    c = fmt.c()
    _check(load().vq_gemm_small_batch_host(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale), _ptr(h_X),
                                           _ptr(h_Y), int(batch), _ptr(d_ws),
                                           d_ws.numel() * d_ws.element_size(), _stream(stream)),
           "vq_gemm_small_batch_host")


def vq_gemm_small_batch_host_static(fmt: VQFormat, d_idx, d_cb, d_scale, h_X, h_Y, batch: int, stream=None) -> None:
    """Host-buffer skinny GEMM that allocates nothing: the device copies of X and Y live in a
    fixed 2 MiB array inside the library (vq_static_scratch_bytes()).  For callers that may not
    call cudaMalloc.  Calls on one device share that array: keep them ordered on the GPU.
    Synchronise before reading h_Y."""
    c = fmt.c()
    _check(load().vq_gemm_small_batch_host_static(ctypes.byref(c), _ptr(d_idx), _ptr(d_cb), _ptr(d_scale),
                                                  _ptr(h_X), _ptr(h_Y), int(batch), _stream(stream)),
           "vq_gemm_small_batch_host_static")


def vq_static_scratch_bytes() -> int:
    return load().vq_static_scratch_bytes()


def vq_probe_decode_loop(policy: int, warps: int, batch: int, iters: int, d_scratch, stream=None):
    """(clocks per pass, weights decoded per pass and SM) of one policy's decode loop on resident data."""
    clocks, weights = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(load().vq_probe_decode_loop(int(policy), int(warps), int(batch), int(iters), _ptr(d_scratch),
                                       d_scratch.numel() * d_scratch.element_size(), ctypes.byref(clocks), ctypes.byref(weights),
                                       _stream(stream)), "vq_probe_decode_loop")
    return clocks.value, weights.value


def vq_probe_read(d_buf, d_out4, stream=None) -> None:
    _check(load().vq_probe_read(_ptr(d_buf), d_buf.numel() * d_buf.element_size(), _ptr(d_out4), _stream(stream)), "vq_probe_read")


def vq_device_wait_failures() -> int:
    """Bounded in-kernel waits that ran out on the current device (0 in a healthy run); synchronises."""
    out = ctypes.c_int(-1)
    _check(load().vq_device_wait_failures(ctypes.byref(out)), "vq_device_wait_failures")
    return out.value


def vq_int4g128_workspace_bytes(n_rows: int, batch: int) -> int:
    return load().vq_int4g128_workspace_bytes(int(n_rows), int(batch))


def vq_int4g128_gemm_small_batch(n_rows: int, k_cols: int, d_q, d_scale, d_X, d_Y, batch: int, d_ws, stream=None) -> None:
    _check(load().vq_int4g128_gemm_small_batch(int(n_rows), int(k_cols), _ptr(d_q), _ptr(d_scale), _ptr(d_X),
                                               _ptr(d_Y), int(batch), _ptr(d_ws), d_ws.numel() * d_ws.element_size(),
                                               _stream(stream)),
           "vq_int4g128_gemm_small_batch")


VQ_UNPACK_FP16, VQ_UNPACK_INT8_ROW, VQ_UNPACK_INT4_G128 = 0, 1, 2


def vq_unpack_uniform(kind: int, n_rows: int, k_cols: int, d_src, d_scale, d_W, stream=None) -> None:
    _check(load().vq_unpack_uniform(int(kind), int(n_rows), int(k_cols), _ptr(d_src), _ptr(d_scale), _ptr(d_W),
                                    _stream(stream)), "vq_unpack_uniform")


def vq_assign_indices(fmt: "VQFormat", d_W, d_cb, d_scale, d_hdiag, d_idx, stream=None) -> None:
    """E-step (Eq. 5): nearest centroid under diagonal weights; writes the packed index stream d_idx."""
    c = fmt.c()
    _check(load().vq_assign_indices(ctypes.byref(c), _ptr(d_W), _ptr(d_cb), _ptr(d_scale), _ptr(d_hdiag), _ptr(d_idx),
                                    _stream(stream)), "vq_assign_indices")

