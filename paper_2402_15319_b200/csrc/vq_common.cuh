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

// Workspace of the persistent kernel (vq_stream.cu): one ticket counter per 16 rows at most, and
// two slabs (at most 256 rows each) of fp32 partial sums per persistent CTA.
constexpr int kMaxStreamCtas = 448;
constexpr int kMaxSlabRows = 256;
// Layers of one grouped call (they share the activations).
constexpr int kMaxSegments = 4;
// Devices per process the launchers keep per-device set-up state for.
constexpr int kMaxDevices = 64;

vq_status make_geometry(const vq_format* fmt, Geometry* g);

// Kernel launchers.  Each returns VQ_OK, VQ_ERR_UNSUPPORTED (format/shape not covered by this
// family) or VQ_ERR_CUDA.
vq_status launch_decode_generic(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s);
vq_status launch_gemm_generic(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y,
                              int batch, cudaStream_t s);
vq_status launch_gemm_tuned(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y,
                            int batch, void* ws, size_t ws_bytes, cudaStream_t s);

// One call of the persistent kernel: n_seg layers of one format and one K that share X.
struct StreamCall {
  Geometry g;          // format and K; g.N is not used (rows per layer are in N[])
  int n_seg;
  const uint8_t* idx[kMaxSegments];
  const void* cb[kMaxSegments];
  const __half* scale[kMaxSegments];
  __half* Y[kMaxSegments];
  int N[kMaxSegments];
  const __half* X;
  int batch;
  void* ws;            // ticket counters (zero on entry, zero on exit) + partial sums
  size_t ws_bytes;
};
size_t stream_workspace_bytes(long long rows, int batch);
size_t stream_ticket_bytes(long long rows);   // the counters at the start of the workspace
vq_status launch_gemm_stream(const StreamCall& call, cudaStream_t s);
bool stream_covers(const Geometry& g);
vq_status launch_int4g128_stream(int N, int K, const uint8_t* q, const __half* scale, const __half* X, __half* Y, int batch,
                                 void* ws, size_t ws_bytes, cudaStream_t s);
vq_status launch_gemm_blockcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s);
// The same kernels over several layers of one format and K in one launch (rows per layer in call.N;
// call.ws is not used), and whether they take the format (member rows must be multiples of 128 too).
vq_status launch_gemm_blockcb_group(const StreamCall& call, cudaStream_t s);
bool blockcb_covers(const Geometry& g);
vq_status launch_gemm_rowcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                            cudaStream_t s);
// Warp-private pair tables: small codebook blocks (1, 2, 4, 8 or a multiple of 16 rows), 2-D indices of
// any width, 1-D indices of up to 4 bits, 4-D 8-bit indices, every codebook type, K and block columns
// multiples of 64.
vq_status launch_gemm_warptab(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s);
// ... over several layers of one format and K in one launch (rows per layer in call.N; call.ws is not used)
vq_status launch_gemm_warptab_group(const StreamCall& call, cudaStream_t s);
bool warptab_covers(const Geometry& g);
// ... with block-wise normalisation (one layer; sub-rows of a power of two >= 16 columns; fp16 / int8 codebooks)
vq_status launch_gemm_warptab_norm(const Geometry& g, const LayerPtrs& p, const void* norm_codes, const void* norm_lut,
                                   int norm_block_cols, const __half* X, __half* Y, int batch, cudaStream_t s);
vq_status launch_int4g128_rowcb(int N, int K, const uint8_t* q, const __half* scale, const __half* X, __half* Y, int batch,
                                cudaStream_t s);
// Block-wise normalisation at decode (format-generic kernels): codes = 4-bit code per row and sub-row of
// block_cols columns, lut = 16 binary16 scales per codebook block.
vq_status launch_decode_norm(const Geometry& g, const LayerPtrs& p, const void* codes, const void* lut, int block_cols,
                             __half* W, cudaStream_t s);
vq_status launch_gemm_norm(const Geometry& g, const LayerPtrs& p, const void* codes, const void* lut, int block_cols,
                           const __half* X, __half* Y, int batch, cudaStream_t s);
vq_status launch_decode_tuned(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s, const void* norm_codes = nullptr,
                              const void* norm_lut = nullptr, int norm_block_cols = 0);
// E-step: nearest centroid under diagonal weights, packed into the index stream `idx` (output).
vq_status launch_assign(const Geometry& g, const LayerPtrs& p, const __half* W, const float* hdiag, uint8_t* idx,
                        cudaStream_t s);

// Device address of this device's counter of bounded waits that ran out inside a kernel (a copy
// that never completed); looked up once per device.
vq_status device_error_counter(int** d_counter);
// SM count of the current device (looked up once per device).
vq_status device_sms(int* out);

// Tensor map of the packed index stream seen as a 2-D byte tensor (N rows of `stride` bytes) with
// boxes of box_rows rows x box_bytes bytes, for tiled TMA loads without swizzle, into the issuing CTA only.
// swizzle128: rows of the box (box_bytes == 128) land with the 128-byte swizzle pattern.
vq_status encode_index_map(CUtensorMap* tm, const uint8_t* idx, long long stride, int N, int box_bytes, int box_rows,
                           bool swizzle128 = false);

// General tiled tensor map (loads with it always target the issuing CTA alone): elements of 1 or 2 bytes, rank <= 5,
// dims / box in elements, strides of dimensions 1.. in bytes; swizzle 0 none, 1 64-byte, 2 128-byte.
vq_status encode_tensor_map(CUtensorMap* tm, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                            const uint64_t* strides, const uint32_t* box, int swizzle);

inline vq_status check_launch() {
  return cudaGetLastError() == cudaSuccess ? VQ_OK : VQ_ERR_CUDA;
}

}  // namespace vq
