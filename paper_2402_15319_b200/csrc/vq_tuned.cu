// Dispatch to the tuned kernel families.
#include "vq_common.cuh"

namespace vq {

namespace {
// Incremented by a kernel whenever one of its bounded waits gives up; stays 0 in a healthy run.
static __device__ int g_wait_failures;
}  // namespace

vq_status encode_index_map(CUtensorMap* tm, const uint8_t* idx, long long stride, int N, int box_bytes, int box_rows) {
  using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                     const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  // the driver's encoder, looked up once through the runtime (no link against libcuda)
  static EncodeTiledFn encode = nullptr;
  if (!encode) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !p)
      return VQ_ERR_CUDA;
    encode = reinterpret_cast<EncodeTiledFn>(p);
  }
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(stride), static_cast<cuuint64_t>(N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(stride)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_bytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem_strides[2] = {1u, 1u};
  if (encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(idx), dims, strides, box, elem_strides,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VQ_ERR_CUDA;
  return VQ_OK;
}

vq_status device_error_counter(int** d_counter) {
  static int* addr_of[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (!addr_of[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_wait_failures) != cudaSuccess || !p) return VQ_ERR_CUDA;
    addr_of[dev] = static_cast<int*>(p);
  }
  *d_counter = addr_of[dev];
  return VQ_OK;
}

vq_status launch_gemm_tuned(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, float* ws,
                            cudaStream_t s) {
  (void)ws;
  if (g.cb_int4) return VQ_ERR_UNSUPPORTED;   // int4 codebooks: format-generic kernels only
  vq_status st = launch_gemm_blockcb(g, p, X, Y, batch, s);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  return launch_gemm_rowcb(g, p, X, Y, batch, s);
}


}  // namespace vq

// Number of in-kernel waits that ran out on the current device since the library was loaded
// (synchronises the device).  0 in a healthy run.
extern "C" vq_status vq_device_wait_failures(int* h_count) {
  if (!h_count) return VQ_ERR_NULL;
  int* d = nullptr;
  vq_status st = vq::device_error_counter(&d);
  if (st != VQ_OK) return st;
  if (cudaMemcpy(h_count, d, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return VQ_ERR_CUDA;
  return VQ_OK;
}
