// Tuned weight materialisation (vq_decode_weights): W[n][jd+t] = cb[blk][i(n,j)][t], times the
// block's scale for int8 codebooks (paper App. A: the quantized matrix is a look-up of the
// codebooks; Sec. 3.2 decode step; App. B transfer + decode experiment).
//
// The kernel is bound by the fp16 output it writes (2 B per weight against 0.27-0.5 B read), so
// everything is arranged around the stores: a warp turns one 256-column segment of one row into 32
// adjacent 128-bit stores (lane l owns columns 8l .. 8l+7 = 8/d indices = m = 8b/d bits).  The
// segment's m index words are fetched by one coalesced 32-bit load (lanes 0..m-1) and handed to
// their owners by two shuffles and a funnel shift.  A CTA works on a tile of 32 rows x 2048 columns
// whose codebooks are first copied into shared memory as final fp16 values (int8 entries as
// fp16(fp32(scale) * c): one rounding, the value the entry point is specified to write), so a
// look-up is one shared-memory load of d halves; bank conflicts among the lanes' random entries
// cost less than the stores.
#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

#ifndef VQ_DEC_TILE_ROWS
#define VQ_DEC_TILE_ROWS 32
#endif
#ifndef VQ_DEC_TILE_COLS
#define VQ_DEC_TILE_COLS 2048
#endif
#ifndef VQ_DEC_UNROLL
#define VQ_DEC_UNROLL 8
#endif
constexpr int kTileRows = VQ_DEC_TILE_ROWS;
constexpr int kTileCols = VQ_DEC_TILE_COLS;
constexpr int kWarps = 8;
constexpr int kUnroll = VQ_DEC_UNROLL;   // segments of a row whose index loads are in flight together

struct DecodeArgs {
  const uint8_t* idx;
  const void* cb;
  const __half* scale;
  const __half* row_scale;   // int4 codebooks: [N][K/128] scales applied after the look-up, else null
  // block-wise normalisation (null codes: off): a 4-bit code per row and sub-row of 1 << norm_shift columns
  // (at least 8: a lane's 8 columns lie in one sub-row) selects one of the 16 scales of the codebook block
  const uint8_t* norm_codes;
  const __half* norm_lut;
  int norm_shift, norm_row_bytes;
  __half* W;
  long long stride;
  int N, K, b, Br, Bc, entries, blocks_per_row;
  int m;              // index bits per lane and segment = 8 b / d
  int tile_cols;      // columns of a tile, a multiple of 256; the last tile of a row may be shorter
  int bc_shift;       // log2(Bc): block columns are a power of two
  int br_per_tile;    // codebook block rows a tile touches
  int bc_per_tile;    // codebook block columns a tile touches
  int rows_per_br;    // tile rows that share a block row = min(Br, kTileRows)
};

template <int D>
__device__ __forceinline__ uint4 lookup8(const __half* tab, uint32_t v, int b, uint32_t emask) {
  // tab: the block's [entry][D] fp16 table in shared memory; v: the lane's 8/D indices
  uint4 out;
  if constexpr (D == 4) {
    const uint2 lo = *reinterpret_cast<const uint2*>(tab + 4 * (v & emask));
    const uint2 hi = *reinterpret_cast<const uint2*>(tab + 4 * ((v >> b) & emask));
    out = make_uint4(lo.x, lo.y, hi.x, hi.y);
  } else if constexpr (D == 2) {
    const uint32_t* t32 = reinterpret_cast<const uint32_t*>(tab);
    out.x = t32[v & emask];
    out.y = t32[(v >> b) & emask];
    out.z = t32[(v >> (2 * b)) & emask];
    out.w = t32[(v >> (3 * b)) & emask];
  } else {
    const uint16_t* t16 = reinterpret_cast<const uint16_t*>(tab);
    uint32_t h[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) h[i] = t16[(v >> (i * b)) & emask];
    out = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
  }
  return out;
}

// Grid (ceil(K / tile_cols), ceil(N / 32)).  Dynamic shared memory: br_per_tile * bc_per_tile
// tables of entries * D halves.
template <int D>
__global__ void __launch_bounds__(32 * kWarps) decode_tile_kernel(const DecodeArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* tables = reinterpret_cast<__half*>(smem_raw);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int row0 = blockIdx.y * kTileRows, col0 = blockIdx.x * a.tile_cols;
  const int table_halves = a.entries * D;

  // ---- codebooks of the tile -> shared memory, as the fp16 values to be written ----
  {
    const long long br0 = row0 / a.Br, bc0 = col0 / a.Bc;
    const long long last_br = (a.N - 1) / a.Br;
    const int n_tab = a.br_per_tile * a.bc_per_tile;
    for (int o = tid; o < n_tab * table_halves; o += 32 * kWarps) {
      const int tb = o / table_halves, within = o - tb * table_halves;
      const int lbr = tb / a.bc_per_tile, lbc = tb - lbr * a.bc_per_tile;
      long long brow = br0 + lbr;
      if (brow > last_br) brow = last_br;   // tile rows past N: any valid block, never stored
      long long bcol = bc0 + lbc;
      if (bcol >= a.blocks_per_row) bcol = a.blocks_per_row - 1;   // short last tile: never looked up
      const long long blk = brow * a.blocks_per_row + bcol;
      __half v;
      if (a.row_scale != nullptr) {   // signed nibble, kept unscaled (exact in fp16)
        const long long at = blk * table_halves + within;
        const uint8_t byte = __ldg(static_cast<const uint8_t*>(a.cb) + (at >> 1));
        const int nib = (at & 1) ? (byte >> 4) : (byte & 15);
        v = __int2half_rn(nib >= 8 ? nib - 16 : nib);
      } else if (a.scale == nullptr) {
        v = __ldg(static_cast<const __half*>(a.cb) + blk * table_halves + within);
      } else if (a.norm_codes != nullptr) {   // normalised int8: entry kept unscaled (exact), block and sub-row scales applied together later
        v = __int2half_rn(static_cast<int>(__ldg(static_cast<const int8_t*>(a.cb) + blk * table_halves + within)));
      } else {
        const float c = static_cast<float>(__ldg(static_cast<const int8_t*>(a.cb) + blk * table_halves + within));
        v = __float2half_rn(__half2float(__ldg(a.scale + blk)) * c);   // exact fp32 product, one rounding
      }
      tables[o] = v;
    }
  }
  __syncthreads();

  const int m = a.m;
  const uint32_t vmask = m == 32 ? 0xffffffffu : ((1u << m) - 1u);
  const uint32_t emask = static_cast<uint32_t>(a.entries - 1);
  const int segs = min(a.tile_cols, a.K - col0) / 256;
  const int bit0 = lane * m, src_lane = bit0 >> 5, sh = bit0 & 31;
  const int src_lane2 = src_lane + 1 < m ? src_lane + 1 : src_lane;
  for (int r = warp; r < kTileRows; r += kWarps) {
    const int n = row0 + r;
    if (n >= a.N) break;
    const uint32_t* row32 = reinterpret_cast<const uint32_t*>(a.idx + n * a.stride) + static_cast<long long>(col0 / 256) * m;
    const __half* row_tabs = tables + (r / a.rows_per_br) * a.bc_per_tile * table_halves;
    uint4* dst = reinterpret_cast<uint4*>(a.W + static_cast<long long>(n) * a.K + col0) + lane;
    // block-column table of the lane's 8 columns: constant per segment group for wide blocks,
    // per-lane offset for blocks narrower than a segment
    const int lane_cols = lane * 8;
    auto emit = [&](int seg, uint32_t word_u) {
      const uint32_t w0 = __shfl_sync(0xffffffffu, word_u, src_lane);
      const uint32_t w1 = __shfl_sync(0xffffffffu, word_u, src_lane2);
      const uint32_t v = __funnelshift_r(w0, w1, sh) & vmask;
      const __half* tab = row_tabs + ((seg * 256 + lane_cols) >> a.bc_shift) * table_halves;
      uint4 out = lookup8<D>(tab, v, a.b, emask);
      if (a.norm_codes != nullptr) {
        // w = binary16(value * scale of the sub-row), the exact product rounded once.  The factor p collects the
        // sub-row's scale and, for int8 / int4 codebooks, the block's / row group's scale: exact in fp32 (22 bits).
        // fp16 entries: p * entry has 22 significand bits, exact in fp32; integer entries: up to 30 bits, formed in fp64.
        const int col = col0 + seg * 256 + lane_cols;
        const long long blk = static_cast<long long>(n / a.Br) * a.blocks_per_row + (col >> a.bc_shift);
        const int j = col >> a.norm_shift;
        const uint32_t code = (static_cast<uint32_t>(__ldg(a.norm_codes + static_cast<long long>(n) * a.norm_row_bytes + (j >> 1))) >> (4 * (j & 1))) & 15u;
        float pf = __half2float(__ldg(a.norm_lut + blk * 16 + code));
        uint32_t* o32 = reinterpret_cast<uint32_t*>(&out);
        if (a.row_scale == nullptr && a.scale == nullptr) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __half2 hv = *reinterpret_cast<const __half2*>(&o32[q]);
            const __half2 r = __halves2half2(__float2half_rn(pf * __low2float(hv)), __float2half_rn(pf * __high2float(hv)));
            o32[q] = *reinterpret_cast<const uint32_t*>(&r);
          }
        } else {
          pf *= a.row_scale != nullptr ? __half2float(__ldg(a.row_scale + static_cast<long long>(n) * (a.K / 128) + col / 128))
                                       : __half2float(__ldg(a.scale + blk));
          const double pd = static_cast<double>(pf);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __half2 hv = *reinterpret_cast<const __half2*>(&o32[q]);
            const __half2 r = __halves2half2(__double2half(pd * static_cast<double>(__low2float(hv))),
                                             __double2half(pd * static_cast<double>(__high2float(hv))));
            o32[q] = *reinterpret_cast<const uint32_t*>(&r);
          }
        }
      } else if (a.row_scale != nullptr) {   // the lane's 8 columns lie in one group of 128: exact fp32 product, one rounding
        const float sc = __half2float(__ldg(a.row_scale + static_cast<long long>(n) * (a.K / 128) + (col0 + seg * 256 + lane_cols) / 128));
        uint32_t* o32 = reinterpret_cast<uint32_t*>(&out);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const __half2 hv = *reinterpret_cast<const __half2*>(&o32[q]);
          const __half2 r = __halves2half2(__float2half_rn(sc * __low2float(hv)), __float2half_rn(sc * __high2float(hv)));
          o32[q] = *reinterpret_cast<const uint32_t*>(&r);
        }
      }
      dst[seg * 32] = out;
    };
    int s0 = 0;
    for (; s0 + kUnroll <= segs; s0 += kUnroll) {   // full groups: no per-segment predicates
      uint32_t word[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) word[u] = lane < m ? __ldg(row32 + (s0 + u) * m + lane) : 0u;
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) emit(s0 + u, word[u]);
    }
    for (; s0 < segs; ++s0) emit(s0, lane < m ? __ldg(row32 + s0 * m + lane) : 0u);
  }
}

}  // namespace

// Formats the tile kernel covers: K a multiple of 256, at most 32 index bits per lane and segment
// (8 b / d <= 32), block columns a power of two >= 8 that divide or are divided by the tile's columns,
// block rows that divide or are divided by 32, tables of the tile within 96 KB of shared memory.
// With norm_codes: block-wise normalisation, sub-rows of a power of two of at least 8 columns.
vq_status launch_decode_tuned(const Geometry& g, const LayerPtrs& p, __half* W, cudaStream_t s, const void* norm_codes,
                              const void* norm_lut, int norm_block_cols) {
  if (g.K % 256 || (8 * g.b) % g.d || 8 * g.b / g.d > 32 || g.Bc % 8) return VQ_ERR_UNSUPPORTED;
  DecodeArgs a;
  a.norm_codes = static_cast<const uint8_t*>(norm_codes);
  a.norm_lut = static_cast<const __half*>(norm_lut);
  a.norm_shift = 0;
  a.norm_row_bytes = 0;
  if (norm_codes) {
    a.norm_shift = -1;
    for (int sft = 3; sft < 31; ++sft)
      if ((1 << sft) == norm_block_cols) a.norm_shift = sft;
    if (a.norm_shift < 0 || !norm_lut) return VQ_ERR_UNSUPPORTED;
    a.norm_row_bytes = (g.K / norm_block_cols + 1) / 2;
  }
  a.tile_cols = g.K < kTileCols ? g.K : kTileCols;
  a.bc_shift = -1;
  for (int sft = 3; sft < 31; ++sft)
    if ((1 << sft) == g.Bc) a.bc_shift = sft;
  if (a.bc_shift < 0) return VQ_ERR_UNSUPPORTED;
  if (a.tile_cols % g.Bc && g.Bc % a.tile_cols) return VQ_ERR_UNSUPPORTED;
  if (kTileRows % g.Br && g.Br % kTileRows) return VQ_ERR_UNSUPPORTED;
  a.idx = p.idx;
  a.cb = p.cb;
  a.scale = g.cb_int8 ? p.scale : nullptr;
  a.row_scale = g.cb_int4 ? p.scale : nullptr;
  a.W = W;
  a.stride = g.stride;
  a.N = g.N;
  a.K = g.K;
  a.b = g.b;
  a.Br = g.Br;
  a.Bc = g.Bc;
  a.entries = g.entries;
  a.blocks_per_row = g.blocks_per_row;
  a.m = 8 * g.b / g.d;
  a.br_per_tile = g.Br >= kTileRows ? 1 : kTileRows / g.Br;
  a.bc_per_tile = g.Bc >= a.tile_cols ? 1 : a.tile_cols / g.Bc;
  a.rows_per_br = g.Br >= kTileRows ? kTileRows : g.Br;
  const size_t smem = static_cast<size_t>(a.br_per_tile) * a.bc_per_tile * g.entries * g.d * sizeof(__half);
  if (smem > 96 * 1024) return VQ_ERR_UNSUPPORTED;
  const dim3 grid((g.K + a.tile_cols - 1) / a.tile_cols, (g.N + kTileRows - 1) / kTileRows, 1);
  static int attr_set[kMaxDevices][3] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  auto launch = [&](auto kern, int slot) {
    if (!__atomic_load_n(&attr_set[dev][slot], __ATOMIC_ACQUIRE)) {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024) != cudaSuccess) return VQ_ERR_CUDA;
      __atomic_store_n(&attr_set[dev][slot], 1, __ATOMIC_RELEASE);
    }
    kern<<<grid, 32 * kWarps, smem, s>>>(a);
    return check_launch();
  };
  if (g.d == 1) return launch(decode_tile_kernel<1>, 0);
  if (g.d == 2) return launch(decode_tile_kernel<2>, 1);
  return launch(decode_tile_kernel<4>, 2);
}

}  // namespace vq
