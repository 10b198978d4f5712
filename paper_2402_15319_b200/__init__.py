"""B200-native VQ-decode linear layer (GPTVQ storage format): thin Python binding over the
C-ABI library libvq_b200.so.  Importing the package loads nothing; the first call loads the
shared library and raises if it has not been built."""
from .binding import (  # noqa: F401
    VQ_CB_FP16, VQ_CB_INT8_SCALED, VQ_CB_INT4_G128, VQ_IMPL_AUTO, VQ_IMPL_GENERIC, VQ_IMPL_TUNED, VQ_IMPL_STREAM,
    VQError, VQFormat, PackInfo, lib_path, load, exported_symbols,
    vq_norm_info, vq_decode_weights_normalized, vq_gemm_small_batch_normalized,
    vq_pack_info, vq_workspace_bytes, vq_workspace_bytes_host, vq_decode_weights, vq_gemv,
    vq_gemm_small_batch, vq_gemm_small_batch_grouped, vq_grouped_kernel_launches, vq_gemm_small_batch_impl, vq_gemm_small_batch_host,
    vq_gemm_small_batch_host_static, vq_static_scratch_bytes, vq_gemm_small_batch_grouped_host, vq_workspace_bytes_grouped_host,
    vq_int4g128_gemm_small_batch, vq_int4g128_workspace_bytes, vq_status_string, vq_device_wait_failures,
    vq_assign_indices, vq_unpack_uniform, vq_probe_decode_loop, vq_probe_read, VQ_UNPACK_FP16, VQ_UNPACK_INT8_ROW, VQ_UNPACK_INT4_G128,
)
