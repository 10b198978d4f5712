// Uniform INT4 group-128 GEMV/skinny GEMM: the bandwidth yard-stick reported beside the VQ
// kernels (paper Sec. 2.1 symmetric uniform quantiser; Sec. 5: uniform 4-bit weights, one scale per 128 columns, 4.125 bits per value).
#include "vq_common.cuh"

namespace vq {
namespace {

template <int MB>
__global__ void __launch_bounds__(256) int4g128_kernel(int N, int K, const uint32_t* __restrict__ q,
                                                       const __half* __restrict__ scale,
                                                       const __half* __restrict__ X, __half* __restrict__ Y,
                                                       int batch) {
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  const int words = K / 8;  // 8 nibbles per 32-bit word
  for (int n = warp_global; n < N; n += warps_total) {
    const uint32_t* row = q + static_cast<long long>(n) * words;
    const __half* srow = scale + static_cast<long long>(n) * (K / 128);
    float acc[MB];
#pragma unroll
    for (int m = 0; m < MB; ++m) acc[m] = 0.f;
    for (int w = lane; w < words; w += 32) {
      const uint32_t bits = __ldg(row + w);
      const float s = __half2float(__ldg(srow + w / 16));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float wv = s * static_cast<float>(static_cast<int>((bits >> (4 * i)) & 15u) - 8);
#pragma unroll
        for (int m = 0; m < MB; ++m)
          if (m < batch) acc[m] = fmaf(wv, __half2float(__ldg(X + static_cast<long long>(m) * K + w * 8 + i)), acc[m]);
      }
    }
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      float v = acc[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && m < batch) Y[static_cast<long long>(m) * N + n] = __float2half_rn(v);
    }
  }
}

// Uniform yard-stick unpackers (App. B transfer + decode experiment): one thread writes 8 adjacent
// weights with one 128-bit store; a warp reads 512 / 256 / 128 contiguous bytes and writes 512.
template <int KIND>
__global__ void __launch_bounds__(256) unpack_uniform_kernel(long long groups8, int k8, const void* __restrict__ src,
                                                             const __half* __restrict__ scale, uint4* __restrict__ W) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < groups8;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    uint4 out;
    if constexpr (KIND == VQ_UNPACK_FP16) {
      out = __ldg(static_cast<const uint4*>(src) + i);
    } else {
      int q[8];
      float s;
      if constexpr (KIND == VQ_UNPACK_INT8_ROW) {
        const uint2 raw = __ldg(static_cast<const uint2*>(src) + i);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          q[j] = static_cast<int8_t>((raw.x >> (8 * j)) & 0xff);
          q[4 + j] = static_cast<int8_t>((raw.y >> (8 * j)) & 0xff);
        }
        s = __half2float(__ldg(scale + i / k8));   // one scale per row of k8 groups
      } else {
        const uint32_t raw = __ldg(static_cast<const uint32_t*>(src) + i);
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = static_cast<int>((raw >> (4 * j)) & 15u) - 8;
        s = __half2float(__ldg(scale + i / 16));   // 16 groups of 8 columns share a scale
      }
      __half2 h[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)   // exact fp32 products, one rounding each
        h[j] = __halves2half2(__float2half_rn(s * static_cast<float>(q[2 * j])), __float2half_rn(s * static_cast<float>(q[2 * j + 1])));
      out = make_uint4(*reinterpret_cast<uint32_t*>(&h[0]), *reinterpret_cast<uint32_t*>(&h[1]),
                       *reinterpret_cast<uint32_t*>(&h[2]), *reinterpret_cast<uint32_t*>(&h[3]));
    }
    W[i] = out;
  }
}

}  // namespace
}  // namespace vq

using namespace vq;

extern "C" size_t vq_int4g128_workspace_bytes(int32_t N, int batch) {
  if (N <= 0 || batch < 1 || batch > 16) return 0;
  return stream_workspace_bytes(N, batch);
}

extern "C" vq_status vq_int4g128_gemm_small_batch(int32_t N, int32_t K, const void* d_q, const void* d_scale,
                                                  const void* d_X, void* d_Y, int batch, void* d_ws, size_t ws_bytes,
                                                  void* stream) {
  if (!d_q || !d_scale || !d_X || !d_Y) return VQ_ERR_NULL;
  if (N <= 0 || K <= 0 || K % 128 || (K / 2) % 16) return VQ_ERR_SHAPE;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  const uintptr_t bitsor = reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_scale) |
                           reinterpret_cast<uintptr_t>(d_X) | reinterpret_cast<uintptr_t>(d_Y);
  if (bitsor & 15u) return VQ_ERR_ALIGN;
  if (!d_ws || ws_bytes < vq_int4g128_workspace_bytes(N, batch)) return VQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(d_ws) & 15u) return VQ_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (N < 8192) {   // few slabs: the cluster kernel's K-split is the cheaper one (4096 x 4096: 5.8 against 11 us)
    const vq_status st = launch_int4g128_rowcb(N, K, static_cast<const uint8_t*>(d_q), static_cast<const __half*>(d_scale),
                                               static_cast<const __half*>(d_X), static_cast<__half*>(d_Y), batch, s);
    if (st != VQ_ERR_UNSUPPORTED) return st;
  }
  {
    // the persistent tensor-core kernel shared with the per-row VQ formats; the plain kernel below
    // covers rows that are not whole 128-byte chunks
    const vq_status st = launch_int4g128_stream(N, K, static_cast<const uint8_t*>(d_q), static_cast<const __half*>(d_scale),
                                                static_cast<const __half*>(d_X), static_cast<__half*>(d_Y), batch, d_ws,
                                                ws_bytes, s);
    if (st != VQ_ERR_UNSUPPORTED) return st;
  }
  long long blocks = (N + 7) / 8;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 8) blocks = static_cast<long long>(sms) * 8;
  const unsigned nb = static_cast<unsigned>(blocks);
  const uint32_t* q = static_cast<const uint32_t*>(d_q);
  const __half* sc = static_cast<const __half*>(d_scale);
  const __half* X = static_cast<const __half*>(d_X);
  __half* Y = static_cast<__half*>(d_Y);
  if (batch == 1) int4g128_kernel<1><<<nb, 256, 0, s>>>(N, K, q, sc, X, Y, batch);
  else if (batch == 2) int4g128_kernel<2><<<nb, 256, 0, s>>>(N, K, q, sc, X, Y, batch);
  else if (batch <= 4) int4g128_kernel<4><<<nb, 256, 0, s>>>(N, K, q, sc, X, Y, batch);
  else if (batch <= 8) int4g128_kernel<8><<<nb, 256, 0, s>>>(N, K, q, sc, X, Y, batch);
  else int4g128_kernel<16><<<nb, 256, 0, s>>>(N, K, q, sc, X, Y, batch);
  return check_launch();
}

extern "C" vq_status vq_unpack_uniform(int kind, int32_t N, int32_t K, const void* d_src, const void* d_scale,
                                       void* d_W, void* stream) {
  if (kind != VQ_UNPACK_FP16 && kind != VQ_UNPACK_INT8_ROW && kind != VQ_UNPACK_INT4_G128) return VQ_ERR_FORMAT;
  if (!d_src || !d_W || (kind != VQ_UNPACK_FP16 && !d_scale)) return VQ_ERR_NULL;
  if (N <= 0 || K <= 0 || K % 128) return VQ_ERR_SHAPE;
  uintptr_t bitsor = reinterpret_cast<uintptr_t>(d_src) | reinterpret_cast<uintptr_t>(d_W);
  if (kind != VQ_UNPACK_FP16) bitsor |= reinterpret_cast<uintptr_t>(d_scale);
  if (bitsor & 15u) return VQ_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const long long groups8 = static_cast<long long>(N) * (K / 8);
  long long blocks = (groups8 + 255) / 256;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 64) blocks = static_cast<long long>(sms) * 64;
  const unsigned nb = static_cast<unsigned>(blocks);
  const __half* sc = static_cast<const __half*>(d_scale);
  uint4* W = static_cast<uint4*>(d_W);
  if (kind == VQ_UNPACK_FP16) unpack_uniform_kernel<VQ_UNPACK_FP16><<<nb, 256, 0, s>>>(groups8, K / 8, d_src, sc, W);
  else if (kind == VQ_UNPACK_INT8_ROW) unpack_uniform_kernel<VQ_UNPACK_INT8_ROW><<<nb, 256, 0, s>>>(groups8, K / 8, d_src, sc, W);
  else unpack_uniform_kernel<VQ_UNPACK_INT4_G128><<<nb, 256, 0, s>>>(groups8, K / 8, d_src, sc, W);
  return check_launch();
}
