// Shared declarations of the CUDA side of the VQ-decode library (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "vq.h"

namespace vq {

// Format with derived quantities, passed by value to kernels.
struct Geometry {
  int N, K, d, b, Br, Bc;
  int cb_int8;            // 0: fp16 codebook, 1: int8 codebook + fp16 block scale
  int cb_int4;            // 1: int4 codebook + fp16 scale per row and group of 128 columns (cb_int8 is 0 then)
  int entries;            // 2^b
  int J;                  // indices per row = K/d
  int blocks_per_row;     // K/Bc
  long long stride;       // bytes between index rows
};

struct LayerPtrs {
  const uint8_t* idx;
  const void* cb;
  const __half* scale;
};

// Maximum number of K-splits any kernel uses; fixes the workspace size.
constexpr int kMaxSplits = 8;
// Devices per process the launchers keep per-device set-up state for.
constexpr int kMaxDevices = 64;

vq_status make_geometry(const vq_format* fmt, Geometry* g);

// Kernel launchers.  Each returns VQ_OK, VQ_ERR_UNSUPPORTED (format/shape not covered by this
// family) or VQ_ERR_CUDA.
vq_status launch_decode_generic(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s);
vq_status launch_gemm_generic(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y,
                              int batch, cudaStream_t s);
vq_status launch_gemm_tuned(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y,
                            int batch, float* ws, cudaStream_t s);
vq_status launch_gemm_blockcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s);
vq_status launch_gemm_rowcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                            cudaStream_t s);
vq_status launch_int4g128_rowcb(int N, int K, const uint8_t* q, const __half* scale, const __half* X, __half* Y, int batch,
                                cudaStream_t s);
vq_status launch_decode_tuned(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s);
// E-step: nearest centroid under diagonal weights, packed into the index stream `idx` (output).
vq_status launch_assign(const Geometry& g, const LayerPtrs& p, const __half* W, const float* hdiag, uint8_t* idx,
                        cudaStream_t s);

// Device address of this device's counter of bounded waits that ran out inside a kernel (a copy
// that never completed); looked up once per device.
vq_status device_error_counter(int** d_counter);

// Tensor map of the packed index stream seen as a 2-D byte tensor (N rows of `stride` bytes) with
// boxes of box_rows rows x box_bytes bytes, for tiled TMA loads without swizzle or multicast.
vq_status encode_index_map(CUtensorMap* tm, const uint8_t* idx, long long stride, int N, int box_bytes, int box_rows);

inline vq_status check_launch() {
  return cudaGetLastError() == cudaSuccess ? VQ_OK : VQ_ERR_CUDA;
}

}  // namespace vq
