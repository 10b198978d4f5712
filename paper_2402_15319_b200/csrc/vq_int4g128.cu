// Uniform INT4 group-128 GEMV/skinny GEMM: the bandwidth yard-stick reported beside the VQ
// kernels (paper Sec. 2.1 symmetric uniform quantiser; Sec. 5 "INT4 g128", 4.125 bits per value).
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

}  // namespace
}  // namespace vq

using namespace vq;

extern "C" vq_status vq_int4g128_gemm_small_batch(int32_t N, int32_t K, const void* d_q, const void* d_scale,
                                                  const void* d_X, void* d_Y, int batch, void* stream) {
  if (!d_q || !d_scale || !d_X || !d_Y) return VQ_ERR_NULL;
  if (N <= 0 || K <= 0 || K % 128 || (K / 2) % 16) return VQ_ERR_SHAPE;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  const uintptr_t bitsor = reinterpret_cast<uintptr_t>(d_q) | reinterpret_cast<uintptr_t>(d_scale) |
                           reinterpret_cast<uintptr_t>(d_X) | reinterpret_cast<uintptr_t>(d_Y);
  if (bitsor & 15u) return VQ_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  {
    // tensor-core path shared with the per-row VQ kernels; the plain kernel below covers the rest
    const vq_status st = launch_int4g128_rowcb(N, K, static_cast<const uint8_t*>(d_q), static_cast<const __half*>(d_scale),
                                               static_cast<const __half*>(d_X), static_cast<__half*>(d_Y), batch, s);
    if (st != VQ_ERR_UNSUPPORTED) return st;
  }
  long long blocks = (N + 7) / 8;
  if (blocks > 148LL * 8) blocks = 148LL * 8;
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
