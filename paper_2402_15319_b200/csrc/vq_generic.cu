// Format-generic kernels: correct for every valid (d, b, block shape, codebook type).
// They read the index stream in groups of 8 indices (= b whole bytes), look entries up straight
// from global memory (L1/L2 cached) and accumulate in fp32.  The tuned kernels replace them for
// the benchmark format families; these remain the path for everything else.
#include "vq_common.cuh"

namespace vq {
namespace {

// Bits [8*g*b, 8*(g+1)*b) of a row: the b bytes holding indices 8g..8g+7 (Sec. 3.2 "packed
// tightly").  Bytes past the row stride read as zero.
__device__ __forceinline__ unsigned long long load_group_bits(const uint8_t* row, long long stride, int g, int b) {
  unsigned long long bits = 0;
  const long long off = static_cast<long long>(g) * b;
  for (int i = 0; i < b; ++i) {
    const long long at = off + i;
    if (at < stride) bits |= static_cast<unsigned long long>(__ldg(row + at)) << (8 * i);
  }
  return bits;
}

// One codebook value as fp32; for int8 codebooks scale*c, exact in fp32 (App. A look-up,
// Sec. 3.1 scale factor).
// int4 codebooks: scale of row n's group of 128 columns times the signed nibble, exact in fp32.
__device__ __forceinline__ float lut_value(const Geometry& g, const LayerPtrs& p, long long blk, int e, int t, int n, int k) {
  const long long at = (blk * g.entries + e) * g.d + t;
  if (g.cb_int4) {
    const uint8_t byte = static_cast<const uint8_t*>(p.cb)[at >> 1];
    const int nib = (at & 1) ? (byte >> 4) : (byte & 15);
    return __half2float(p.scale[static_cast<long long>(n) * (g.K / 128) + k / 128]) * static_cast<float>(nib >= 8 ? nib - 16 : nib);
  }
  if (g.cb_int8) {
    const float c = static_cast<float>(static_cast<const int8_t*>(p.cb)[at]);
    return __half2float(p.scale[blk]) * c;
  }
  return __half2float(static_cast<const __half*>(p.cb)[at]);
}

__global__ void decode_generic_kernel(Geometry g, LayerPtrs p, __half* __restrict__ W) {
  const int groups = (g.J + 7) / 8;
  const long long total = static_cast<long long>(g.N) * groups;
  for (long long it = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; it < total;
       it += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int n = static_cast<int>(it / groups);
    const int grp = static_cast<int>(it % groups);
    const uint8_t* row = p.idx + n * g.stride;
    const unsigned long long bits = load_group_bits(row, g.stride, grp, g.b);
    const long long blk_row = static_cast<long long>(n / g.Br) * g.blocks_per_row;
    for (int i = 0; i < 8; ++i) {
      const int j = grp * 8 + i;
      if (j >= g.J) break;
      const int e = static_cast<int>((bits >> (i * g.b)) & (g.entries - 1));
      const int k0 = j * g.d;
      const long long blk = blk_row + k0 / g.Bc;
      for (int t = 0; t < g.d; ++t) {
        __half h;
        if (g.cb_int8 || g.cb_int4) {
          h = __float2half_rn(lut_value(g, p, blk, e, t, n, k0 + t));
        } else {
          h = static_cast<const __half*>(p.cb)[(blk * g.entries + e) * g.d + t];  // bit copy
        }
        W[static_cast<long long>(n) * g.K + k0 + t] = h;
      }
    }
  }
}

// Vectorised decode for formats whose rows hold a whole number of 8-index groups (K/d % 8 == 0):
// one thread expands one group (b bytes of indices) into 8*D weights and writes them with D
// 128-bit stores; a warp writes 512*D contiguous bytes of one row.  The kernel is bound by the
// fp16 output it has to write (2 B per weight); the codebook look-ups go through L1.
template <int D>
__global__ void __launch_bounds__(256) decode_vec_kernel(Geometry g, LayerPtrs p, __half* __restrict__ W) {
  const int groups = g.J / 8;
  const long long total = static_cast<long long>(g.N) * groups;
  const bool block_per_group = g.Bc % (8 * D) == 0;   // a group never straddles two codebook blocks
  for (long long it = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; it < total;
       it += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int n = static_cast<int>(it / groups);
    const int grp = static_cast<int>(it - static_cast<long long>(n) * groups);
    const uint8_t* src = p.idx + n * g.stride + static_cast<long long>(grp) * g.b;
    unsigned long long bits = 0;
    for (int i = 0; i < g.b; ++i) bits |= static_cast<unsigned long long>(__ldg(src + i)) << (8 * i);
    const long long blk_row = static_cast<long long>(n / g.Br) * g.blocks_per_row;
    const int k0 = grp * 8 * D;
    long long blk = blk_row + k0 / g.Bc;
    float sc = g.cb_int8 ? __half2float(__ldg(p.scale + blk)) : 0.f;
    __align__(16) __half out[8 * D];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int e = static_cast<int>((bits >> (i * g.b)) & (g.entries - 1));
      if (!block_per_group) {
        blk = blk_row + (k0 + i * D) / g.Bc;
        if (g.cb_int8) sc = __half2float(__ldg(p.scale + blk));
      }
      const long long at = (blk * g.entries + e) * D;
      if (g.cb_int8) {
        const int8_t* c = static_cast<const int8_t*>(p.cb) + at;
#pragma unroll
        for (int t = 0; t < D; ++t) out[i * D + t] = __float2half_rn(sc * static_cast<float>(__ldg(c + t)));   // exact product, one rounding
      } else {
        const __half* c = static_cast<const __half*>(p.cb) + at;   // bit copies
        if constexpr (D == 1) out[i] = __ldg(c);
        else if constexpr (D == 2) *reinterpret_cast<uint32_t*>(&out[2 * i]) = __ldg(reinterpret_cast<const uint32_t*>(c));
        else *reinterpret_cast<uint2*>(&out[4 * i]) = __ldg(reinterpret_cast<const uint2*>(c));
      }
    }
    uint4* dst = reinterpret_cast<uint4*>(W + static_cast<long long>(n) * g.K + k0);
#pragma unroll
    for (int q = 0; q < D; ++q) dst[q] = reinterpret_cast<const uint4*>(out)[q];
  }
}

template <int MB>
__global__ void __launch_bounds__(256) gemm_generic_kernel(Geometry g, LayerPtrs p, const __half* __restrict__ X,
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
      const unsigned long long bits = load_group_bits(row, g.stride, grp, g.b);
      for (int i = 0; i < 8; ++i) {
        const int j = grp * 8 + i;
        if (j >= g.J) break;
        const int e = static_cast<int>((bits >> (i * g.b)) & (g.entries - 1));
        const int k0 = j * g.d;
        const long long blk = blk_row + k0 / g.Bc;
        for (int t = 0; t < g.d; ++t) {
          const float w = lut_value(g, p, blk, e, t, n, k0 + t);
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

}  // namespace

vq_status launch_decode_generic(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s) {
  if (g.J % 8 == 0 && !g.cb_int4) {   // K % 8 == 0 follows: every 128-bit store is aligned
    const long long total = static_cast<long long>(g.N) * (g.J / 8);
    long long blocks = (total + 255) / 256;
    int sms = 0;
    if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
    if (blocks > static_cast<long long>(sms) * 32) blocks = static_cast<long long>(sms) * 32;
    const unsigned nb = static_cast<unsigned>(blocks);
    if (g.d == 1) decode_vec_kernel<1><<<nb, 256, 0, s>>>(g, p, W);
    else if (g.d == 2) decode_vec_kernel<2><<<nb, 256, 0, s>>>(g, p, W);
    else decode_vec_kernel<4><<<nb, 256, 0, s>>>(g, p, W);
    return check_launch();
  }
  const long long total = static_cast<long long>(g.N) * ((g.J + 7) / 8);
  long long blocks = (total + 255) / 256;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 64) blocks = static_cast<long long>(sms) * 64;
  decode_generic_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(g, p, W);
  return check_launch();
}

vq_status launch_gemm_generic(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s) {
  long long blocks = (g.N + 7) / 8;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (blocks > static_cast<long long>(sms) * 8) blocks = static_cast<long long>(sms) * 8;
  const unsigned nb = static_cast<unsigned>(blocks);
  if (batch == 1) gemm_generic_kernel<1><<<nb, 256, 0, s>>>(g, p, X, Y, batch);
  else if (batch == 2) gemm_generic_kernel<2><<<nb, 256, 0, s>>>(g, p, X, Y, batch);
  else if (batch <= 4) gemm_generic_kernel<4><<<nb, 256, 0, s>>>(g, p, X, Y, batch);
  else if (batch <= 8) gemm_generic_kernel<8><<<nb, 256, 0, s>>>(g, p, X, Y, batch);
  else gemm_generic_kernel<16><<<nb, 256, 0, s>>>(g, p, X, Y, batch);
  return check_launch();
}

}  // namespace vq
