// vq_gemm_small_batch_host_static: the host-buffer skinny GEMM for callers that cannot allocate
// device memory.  Its device-side staging buffers (a copy of X, room for Y) live in a fixed array
// that is part of the library image instead of in a workspace the caller would have to allocate.
#include "vq_common.cuh"

namespace vq {
namespace {

constexpr size_t kStaticScratchBytes = 2u << 20;   // 2 MiB per GPU that loads the library

// Device scratch shared by every call on a device.  In host code this NAME is only a handle for
// cudaGetSymbolAddress; the address kernels and copies may use is what that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

size_t round256(size_t v) { return (v + 255) / 256 * 256; }

// Device address of the scratch array on the current device, looked up once per device.
vq_status scratch_address(unsigned char** out) {
  static unsigned char* addr_of[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (addr_of[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return VQ_ERR_CUDA;
    addr_of[dev] = static_cast<unsigned char*>(p);
  }
  *out = addr_of[dev];
  return VQ_OK;
}

}  // namespace
}  // namespace vq

using namespace vq;

extern "C" size_t vq_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" vq_status vq_gemm_small_batch_host_static(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                                     const void* d_scale, const void* h_X, void* h_Y, int batch,
                                                     void* stream) {
  Geometry g;
  vq_status st = make_geometry(fmt, &g);
  if (st != VQ_OK) return st;
  if (!d_idx || !d_cb || !h_X || !h_Y) return VQ_ERR_NULL;
  if ((g.cb_int8 || g.cb_int4) ? d_scale == nullptr : d_scale != nullptr) return VQ_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(d_idx) | reinterpret_cast<uintptr_t>(d_cb) | reinterpret_cast<uintptr_t>(d_scale)) & 15u)
    return VQ_ERR_ALIGN;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  const size_t x_bytes = static_cast<size_t>(batch) * g.K * 2, y_bytes = static_cast<size_t>(batch) * g.N * 2;
  if (round256(x_bytes) + round256(y_bytes) > kStaticScratchBytes) return VQ_ERR_WORKSPACE;   // beyond the fixed scratch
  unsigned char* scratch = nullptr;
  st = scratch_address(&scratch);
  if (st != VQ_OK) return st;
  // Nothing in the scratch has to start at zero: X is overwritten by the copy, Y by the kernel.
  __half* d_X = reinterpret_cast<__half*>(scratch);
  __half* d_Y = reinterpret_cast<__half*>(scratch + round256(x_bytes));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(d_X, h_X, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return VQ_ERR_CUDA;
  LayerPtrs p;
  p.idx = static_cast<const uint8_t*>(d_idx);
  p.cb = d_cb;
  p.scale = static_cast<const __half*>(d_scale);
  st = launch_gemm_tuned(g, p, d_X, d_Y, batch, nullptr, 0, s);
  if (st == VQ_ERR_UNSUPPORTED) st = launch_gemm_generic(g, p, d_X, d_Y, batch, s);
  if (st != VQ_OK) return st;
  if (cudaMemcpyAsync(h_Y, d_Y, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VQ_ERR_CUDA;
  return VQ_OK;
}
