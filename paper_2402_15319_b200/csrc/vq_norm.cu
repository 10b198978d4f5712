// Block-wise data normalisation applied at decode (paper App. on blockwise data normalization): every
// sub-row of `block_cols` columns carries a 4-bit code that selects one of 16 scales of its codebook
// block; the decoded weight is the looked-up value times that scale.  The 16 scales per block come as a
// table (the quantizer's log2 grid is its own business: the decoder needs the values only).
//
// Format-generic kernels (any valid VQ format): a thread takes 8 indices (= b whole bytes of the stream)
// at a time, as the format-generic kernels without normalisation do.
//   decode: w = binary16(value * scale), the product formed exactly in fp64 (at most 11 + 8 + 11
//           significand bits for int8 codebooks, 11 + 4 + 11 for int4 ones) and rounded once.
//   GEMM  : fp32 multiply-adds, one warp per output row, lanes summed by shuffles, one rounding to fp16.
#include "vq_common.cuh"

namespace vq {
namespace {

struct NormArgs {
  const uint8_t* codes;     // [N][code_row_bytes], two 4-bit codes per byte, low nibble = lower sub-row
  const __half* lut;        // [blocks][16]
  int block_cols;           // columns per sub-row
  int code_row_bytes;       // (K / block_cols + 1) / 2
};

__device__ __forceinline__ unsigned long long group_bits(const uint8_t* row, long long stride, int g, int b) {
  unsigned long long bits = 0;
  const long long off = static_cast<long long>(g) * b;
  for (int i = 0; i < b; ++i) {
    const long long at = off + i;
    if (at < stride) bits |= static_cast<unsigned long long>(__ldg(row + at)) << (8 * i);
  }
  return bits;
}

// Looked-up value before normalisation, exact in fp32 (scale * c has at most 19 significand bits).
__device__ __forceinline__ float entry_value(const Geometry& g, const LayerPtrs& p, long long blk, int e, int t, int n, int k) {
  const long long at = (blk * g.entries + e) * g.d + t;
  if (g.cb_int4) {
    const uint8_t byte = static_cast<const uint8_t*>(p.cb)[at >> 1];
    const int nib = (at & 1) ? (byte >> 4) : (byte & 15);
    return __half2float(p.scale[static_cast<long long>(n) * (g.K / 128) + k / 128]) * static_cast<float>(nib >= 8 ? nib - 16 : nib);
  }
  if (g.cb_int8) return __half2float(p.scale[blk]) * static_cast<float>(static_cast<const int8_t*>(p.cb)[at]);
  return __half2float(static_cast<const __half*>(p.cb)[at]);
}

// Scale of the sub-row that column k of row n lies in.
__device__ __forceinline__ float sub_row_scale(const NormArgs& na, long long blk, int n, int k) {
  const int j = k / na.block_cols;
  const uint8_t byte = __ldg(na.codes + static_cast<long long>(n) * na.code_row_bytes + (j >> 1));
  const int code = (j & 1) ? (byte >> 4) : (byte & 15);
  return __half2float(__ldg(na.lut + blk * 16 + code));
}

__global__ void __launch_bounds__(256) decode_norm_kernel(Geometry g, LayerPtrs p, NormArgs na, __half* __restrict__ W) {
  const int groups = (g.J + 7) / 8;
  const long long total = static_cast<long long>(g.N) * groups;
  for (long long it = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; it < total;
       it += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int n = static_cast<int>(it / groups);
    const int grp = static_cast<int>(it % groups);
    const unsigned long long bits = group_bits(p.idx + n * g.stride, g.stride, grp, g.b);
    const long long blk_row = static_cast<long long>(n / g.Br) * g.blocks_per_row;
    for (int i = 0; i < 8; ++i) {
      const int j = grp * 8 + i;
      if (j >= g.J) break;
      const int e = static_cast<int>((bits >> (i * g.b)) & (g.entries - 1));
      const int k0 = j * g.d;
      const long long blk = blk_row + k0 / g.Bc;
      const double s = static_cast<double>(sub_row_scale(na, blk, n, k0));   // (a VQ vector lies inside one sub-row)
      for (int t = 0; t < g.d; ++t)
        W[static_cast<long long>(n) * g.K + k0 + t] = __double2half(static_cast<double>(entry_value(g, p, blk, e, t, n, k0 + t)) * s);
    }
  }
}

template <int MB>
__global__ void __launch_bounds__(256) gemm_norm_kernel(Geometry g, LayerPtrs p, NormArgs na, const __half* __restrict__ X,
                                                        __half* __restrict__ Y, int batch) {
  const int lane = threadIdx.x & 31;
  const int warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int warps_total = (gridDim.x * blockDim.x) >> 5;
  const int groups = (g.J + 7) / 8;
  for (int n = warp_global; n < g.N; n += warps_total) {
    const uint8_t* row = p.idx + n * g.stride;
    const long long blk_row = static_cast<long long>(n / g.Br) * g.blocks_per_row;
    float acc[MB];
#pragma unroll
    for (int m = 0; m < MB; ++m) acc[m] = 0.f;
    for (int grp = lane; grp < groups; grp += 32) {
      const unsigned long long bits = group_bits(row, g.stride, grp, g.b);
      for (int i = 0; i < 8; ++i) {
        const int j = grp * 8 + i;
        if (j >= g.J) break;
        const int e = static_cast<int>((bits >> (i * g.b)) & (g.entries - 1));
        const int k0 = j * g.d;
        const long long blk = blk_row + k0 / g.Bc;
        const float s = sub_row_scale(na, blk, n, k0);
        for (int t = 0; t < g.d; ++t) {
          const float w = entry_value(g, p, blk, e, t, n, k0 + t) * s;
#pragma unroll
          for (int m = 0; m < MB; ++m)
            if (m < batch) acc[m] = fmaf(w, __half2float(__ldg(X + static_cast<long long>(m) * g.K + k0 + t)), acc[m]);
        }
      }
    }
#pragma unroll
    for (int m = 0; m < MB; ++m) {
      float v = acc[m];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0 && m < batch) Y[static_cast<long long>(m) * g.N + n] = __float2half_rn(v);
    }
  }
}

NormArgs norm_args(const Geometry& g, const void* codes, const void* lut, int block_cols) {
  NormArgs na;
  na.codes = static_cast<const uint8_t*>(codes);
  na.lut = static_cast<const __half*>(lut);
  na.block_cols = block_cols;
  na.code_row_bytes = (g.K / block_cols + 1) / 2;
  return na;
}

}  // namespace

vq_status launch_decode_norm(const Geometry& g, const LayerPtrs& p, const void* codes, const void* lut, int block_cols,
                             __half* W, cudaStream_t s) {
  const long long total = static_cast<long long>(g.N) * ((g.J + 7) / 8);
  long long blocks = (total + 255) / 256;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 64) blocks = static_cast<long long>(sms) * 64;
  decode_norm_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(g, p, norm_args(g, codes, lut, block_cols), W);
  return check_launch();
}

vq_status launch_gemm_norm(const Geometry& g, const LayerPtrs& p, const void* codes, const void* lut, int block_cols,
                           const __half* X, __half* Y, int batch, cudaStream_t s) {
  long long blocks = (g.N + 7) / 8;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 8) blocks = static_cast<long long>(sms) * 8;
  const unsigned nb = static_cast<unsigned>(blocks);
  const NormArgs na = norm_args(g, codes, lut, block_cols);
  if (batch == 1) gemm_norm_kernel<1><<<nb, 256, 0, s>>>(g, p, na, X, Y, batch);
  else if (batch == 2) gemm_norm_kernel<2><<<nb, 256, 0, s>>>(g, p, na, X, Y, batch);
  else if (batch <= 4) gemm_norm_kernel<4><<<nb, 256, 0, s>>>(g, p, na, X, Y, batch);
  else if (batch <= 8) gemm_norm_kernel<8><<<nb, 256, 0, s>>>(g, p, na, X, Y, batch);
  else gemm_norm_kernel<16><<<nb, 256, 0, s>>>(g, p, na, X, Y, batch);
  return check_launch();
}

}  // namespace vq
