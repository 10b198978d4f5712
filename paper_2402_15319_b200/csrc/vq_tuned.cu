// Dispatch to the tuned kernel families.
#include "vq_common.cuh"

namespace vq {

namespace {
// Incremented by a kernel whenever one of its bounded waits gives up; stays 0 in a healthy run.
static __device__ int g_wait_failures;
}  // namespace

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
  vq_status st = launch_gemm_blockcb(g, p, X, Y, batch, s);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  return launch_gemm_rowcb(g, p, X, Y, batch, s);
}

vq_status launch_decode_tuned(const Geometry&, const LayerPtrs&, __half*, cudaStream_t) {
  return VQ_ERR_UNSUPPORTED;
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
