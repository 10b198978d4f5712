// warptab_kernel<EB, NB>: formats with SMALL codebook blocks (1, 2, 4, 8 rows, or any multiple of 16
// rows) and any index width the other tuned families do not take: 2-D indices of 1..8 bits, 1-D indices
// of 1..4 bits; fp16 or scaled-int8 codebooks; block columns and K multiples of 64.  These are the
// remaining rows of the paper's configuration table (App. on VQ configurations: 1-D 2-bit 1x256 and
// 1x128, 2-D 2.5 bits per dimension on 2x256 and 4x256, 1-D 3-bit 32x256, 2-D 8-bit indices 256x256).
//
// Everything is expressed as PAIR look-ups: EB bits of the index stream select one 32-bit table word
// holding the two fp16 weights of two adjacent columns.  For d = 2 that is the codebook entry itself
// (EB = index_bits); for d = 1 two consecutive indices are looked up at once in the product table
// word[e] = (c[e mod k], c[e div k]) with EB = 2 * index_bits (the decode of Sec. 3.2 / App. A, two values
// per look-up as the paper's LUT instructions do).  Scales of int8 codebooks are folded into the table
// (w = fp16(scale * c), Sec. 3.1).
//
// Work: a CTA owns 16 output rows; its warps split K.  A warp walks its column range in steps of 64
// columns.  In a step, lane (g = lane / 4, t = lane % 4) takes 8 consecutive pairs (EB bytes of the
// stream, columns 16t .. 16t+15 of the step) of rows g and g + 8, gathers their table words and feeds
// them as A fragments to four m16n8k16 tensor-core steps whose B fragments are the activations of the
// same columns (batch rows 0..7, and 8..15 in a second accumulator when NB == 2); fp32 accumulation.
// Tables are private to the warp: one table per codebook block row that the 16 rows touch (16 / Br
// tables, one if Br >= 16), rebuilt whenever the walk enters a new block column.  The warps' partial
// sums meet in shared memory in a fixed order (bit-identical results run to run).
#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

using namespace dev;

constexpr int kMaxWarps = 8;   // per CTA; three CTAs of that size fit an SM's registers

struct WarpTabArgs {
  const uint8_t* idx;
  const void* cb;
  const __half* scale;
  const __half* X;
  __half* Y;
  long long stride;
  int N, K, batch;
  int d, b, entries, cb_int8;
  int Br, br_shift, block_rows;   // br_shift: log2(Br) when Br < 16
  int bsteps;                     // 64-column steps per codebook block (Bc / 64)
  int blocks_per_row;
  int steps_total, steps_per_warp;
  int tbl_words;                  // words of one warp's tables (tables << EB)
  int red_off;                    // byte offset of the reduction buffer in shared memory
};

__device__ __forceinline__ void fence_acc4(float (&c)[4]) {
  asm volatile("" : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])::"memory");
}

// Byte address offset (entry * 4) of pair P of a lane's 8 pairs; (lo, hi, top) hold the lane's EB bytes
// from bit 0 of lo upwards.
template <int EB, int P>
__device__ __forceinline__ uint32_t pair_offset(uint32_t lo, uint32_t hi) {
  constexpr int SH = P * EB;
  constexpr uint32_t M4 = ((1u << EB) - 1u) << 2;
  if constexpr (SH + EB <= 32) {
    if constexpr (SH >= 2) return (lo >> (SH - 2)) & M4;
    else return (lo << (2 - SH)) & M4;
  } else if constexpr (SH >= 32) {
    if constexpr (SH - 32 >= 2) return (hi >> (SH - 34)) & M4;
    else return (hi << (34 - SH)) & M4;
  } else {
    return __funnelshift_r(lo, hi, SH - 2) & M4;   // SH >= 25 here
  }
}

// The EB bytes at byte offset `o` of a row as (lo, hi): aligned 32-bit loads of the words that hold them.
// Every word read lies inside the row pitch: the last byte needed is o + EB - 1 < row bytes <= pitch,
// and both are multiples of 4 past the word's start.
template <int EB>
__device__ __forceinline__ void load_bits(const uint8_t* row, int o, uint32_t& lo, uint32_t& hi) {
  const int sh = (o & 3) * 8;
  const uint32_t* w = reinterpret_cast<const uint32_t*>(row + (o & ~3));
  const uint32_t w0 = __ldg(w);
  uint32_t w1 = 0, w2 = 0;
  if ((o & 3) + EB > 4) w1 = __ldg(w + 1);
  if constexpr (EB == 7) {
    if ((o & 3) + EB > 8) w2 = __ldg(w + 2);
  }
  lo = __funnelshift_r(w0, w1, sh);
  hi = __funnelshift_r(w1, w2, sh);
}

template <int EB, int NB>
__global__ void __launch_bounds__(kMaxWarps * 32, 3) warptab_kernel(const WarpTabArgs a) {
  extern __shared__ __align__(16) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int row0 = blockIdx.x * 16;
  const int rA = min(row0 + g, a.N - 1), rB = min(row0 + g + 8, a.N - 1);   // rows past N: computed, not written
  const int brow0 = a.Br >= 16 ? row0 / a.Br : row0 >> a.br_shift;
  uint32_t* tbl = reinterpret_cast<uint32_t*>(smem) + warp * a.tbl_words;
  uint32_t tA = smem_u32(tbl), tB = tA;
  if (a.Br < 16) {
    tA += static_cast<uint32_t>((rA >> a.br_shift) - brow0) << (EB + 2);
    tB += static_cast<uint32_t>((rB >> a.br_shift) - brow0) << (EB + 2);
  }
  const uint8_t* rowA = a.idx + rA * a.stride;
  const uint8_t* rowB = a.idx + rB * a.stride;

  float acc[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[nb][c] = 0.f;

  // One table word per (table j, pair entry e): the two fp16 weights that the EB index bits stand for.
  auto build = [&](int col_blk) {
    for (int i = lane; i < a.tbl_words; i += 32) {
      const int j = i >> EB, e = i & ((1 << EB) - 1);
      const int brow = min(brow0 + j, a.block_rows - 1);
      const long long blk = static_cast<long long>(brow) * a.blocks_per_row + col_blk;
      long long at0, at1;
      if (a.d == 2) {
        at0 = (blk * a.entries + e) * 2;
        at1 = at0 + 1;
      } else {
        at0 = blk * a.entries + (e & (a.entries - 1));
        at1 = blk * a.entries + (e >> a.b);
      }
      __half h0, h1;
      if (a.cb_int8) {
        const float sc = __half2float(__ldg(a.scale + blk));
        const int8_t* c = static_cast<const int8_t*>(a.cb);
        h0 = __float2half_rn(sc * static_cast<float>(__ldg(c + at0)));   // exact product, one rounding
        h1 = __float2half_rn(sc * static_cast<float>(__ldg(c + at1)));
      } else {
        const __half* c = static_cast<const __half*>(a.cb);
        h0 = __ldg(c + at0);
        h1 = __ldg(c + at1);
      }
      tbl[i] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
    }
  };

  constexpr int U = NB == 1 ? 4 : 2;   // steps whose index words and activations are fetched ahead
  const int s_begin = warp * a.steps_per_warp;
  const int s_end = min(a.steps_total, s_begin + a.steps_per_warp);
  int until_rebuild = 0;   // steps left in the current codebook block column
  for (int s0 = s_begin; s0 < s_end; s0 += U) {
    uint32_t lo[U][2], hi[U][2];
    uint4 xv[U][NB][2];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = min(s0 + u, s_end - 1);   // (steps past the range are loaded again, not used)
      const int o = (s * 4 + t) * EB;
      load_bits<EB>(rowA, o, lo[u][0], hi[u][0]);
      load_bits<EB>(rowB, o, lo[u][1], hi[u][1]);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        const int m = nb * 8 + g;
        if (m < a.batch) {
          const __half* x = a.X + static_cast<long long>(m) * a.K + s * 64 + t * 16;
          xv[u][nb][0] = ldg128_nc(x);
          xv[u][nb][1] = ldg128_nc(x + 8);
        } else {
          xv[u][nb][0] = make_uint4(0u, 0u, 0u, 0u);
          xv[u][nb][1] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = s0 + u;
      if (s < s_end) {
        if (until_rebuild == 0) {
          const int col_blk = s / a.bsteps;
          until_rebuild = a.bsteps - (s - col_blk * a.bsteps);
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) fence_acc4(acc[nb]);   // the gathers of the old tables are done
          __syncwarp();
          build(col_blk);
          __syncwarp();
          fence_value(tA);
          fence_value(tB);
        }
        --until_rebuild;
        uint32_t wa[8], wb[8];
#define VQ_WT_PAIR(P)                                                     \
  wa[P] = lds32(tA + pair_offset<EB, P>(lo[u][0], hi[u][0]));            \
  wb[P] = lds32(tB + pair_offset<EB, P>(lo[u][1], hi[u][1]));
        VQ_WT_PAIR(0) VQ_WT_PAIR(1) VQ_WT_PAIR(2) VQ_WT_PAIR(3)
        VQ_WT_PAIR(4) VQ_WT_PAIR(5) VQ_WT_PAIR(6) VQ_WT_PAIR(7)
#undef VQ_WT_PAIR
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          const uint4 x0 = xv[u][nb][0], x1 = xv[u][nb][1];
          mma16816(acc[nb], wa[0], wb[0], wa[1], wb[1], x0.x, x0.y);
          mma16816(acc[nb], wa[2], wb[2], wa[3], wb[3], x0.z, x0.w);
          mma16816(acc[nb], wa[4], wb[4], wa[5], wb[5], x1.x, x1.y);
          mma16816(acc[nb], wa[6], wb[6], wa[7], wb[7], x1.z, x1.w);
        }
      }
    }
  }

  // K parts of the warps meet in shared memory; thread i then owns output (batch row i / 16, row i % 16).
  float* red = reinterpret_cast<float*>(smem + a.red_off);
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int c = 0; c < 4; ++c) red[(warp * NB * 4 + nb * 4 + c) * 32 + lane] = acc[nb][c];
  __syncthreads();
  const int warps = blockDim.x >> 5;
  for (int i = threadIdx.x; i < 128 * NB; i += blockDim.x) {
    const int r = i & 15, m = i >> 4;
    const int nb = m >> 3, mm = m & 7;
    const int c = (mm & 1) + 2 * (r >> 3);
    const int src_lane = (r & 7) * 4 + (mm >> 1);
    float sum = 0.f;
    for (int w = 0; w < warps; ++w) sum += red[(w * NB * 4 + nb * 4 + c) * 32 + src_lane];
    if (m < a.batch && row0 + r < a.N) a.Y[static_cast<long long>(m) * a.N + row0 + r] = __float2half_rn(sum);
  }
}

int pair_bits(const Geometry& g) {
  if (g.d == 2) return g.b;
  if (g.d == 1 && g.b <= 4) return 2 * g.b;
  return 0;
}

int tables_per_tile(const Geometry& g) { return g.Br >= 16 ? 1 : 16 / g.Br; }

template <int EB>
vq_status launch_eb(const WarpTabArgs& a, int nb, unsigned grid, unsigned threads, size_t smem_bytes, cudaStream_t s) {
  if (nb == 1) warptab_kernel<EB, 1><<<grid, threads, smem_bytes, s>>>(a);
  else warptab_kernel<EB, 2><<<grid, threads, smem_bytes, s>>>(a);
  return check_launch();
}

}  // namespace

bool warptab_covers(const Geometry& g) {
  if (g.cb_int4) return false;
  const int eb = pair_bits(g);
  if (eb < 1 || eb > 8) return false;
  if (g.K % 64 || g.Bc % 64) return false;
  if (!(g.Br == 1 || g.Br == 2 || g.Br == 4 || g.Br == 8 || g.Br % 16 == 0)) return false;
  return (tables_per_tile(g) << eb) <= 1024;
}

vq_status launch_gemm_warptab(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s) {
  if (!warptab_covers(g)) return VQ_ERR_UNSUPPORTED;
  const int eb = pair_bits(g);
  const int nb = batch <= 8 ? 1 : 2;
  WarpTabArgs a = {};
  a.idx = p.idx;
  a.cb = p.cb;
  a.scale = p.scale;
  a.X = X;
  a.Y = Y;
  a.stride = g.stride;
  a.N = g.N;
  a.K = g.K;
  a.batch = batch;
  a.d = g.d;
  a.b = g.b;
  a.entries = g.entries;
  a.cb_int8 = g.cb_int8;
  a.Br = g.Br;
  a.br_shift = g.Br == 1 ? 0 : g.Br == 2 ? 1 : g.Br == 4 ? 2 : 3;
  a.block_rows = g.N / g.Br;
  a.bsteps = g.Bc / 64;
  a.blocks_per_row = g.blocks_per_row;
  a.steps_total = g.K / 64;
  a.tbl_words = tables_per_tile(g) << eb;
  // K split: enough warps to fill the device (about 32 per SM), at most kMaxWarps per CTA, each at least one step
  // and, where the layer is large enough for that, at least one whole codebook block column
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  const long long tiles = (static_cast<long long>(g.N) + 15) / 16;
  int wk = kMaxWarps;
  while (wk > 1 && tiles * wk > 32LL * sms && tiles * (wk / 2) >= 24LL * sms) wk /= 2;
  if (wk > a.steps_total) wk = a.steps_total;
  auto smem_for = [&](int w) { return static_cast<size_t>(w) * (a.tbl_words * 4 + nb * 4 * 32 * 4); };
  while (wk > 1 && smem_for(wk) > 48 * 1024) --wk;
  a.steps_per_warp = (a.steps_total + wk - 1) / wk;
  wk = (a.steps_total + a.steps_per_warp - 1) / a.steps_per_warp;   // no warp without work
  a.red_off = wk * a.tbl_words * 4;
  const size_t smem_bytes = smem_for(wk);
  if (smem_bytes > 48 * 1024) return VQ_ERR_UNSUPPORTED;
  const unsigned grid = static_cast<unsigned>(tiles), threads = static_cast<unsigned>(wk) * 32u;
  switch (eb) {
    case 1: return launch_eb<1>(a, nb, grid, threads, smem_bytes, s);
    case 2: return launch_eb<2>(a, nb, grid, threads, smem_bytes, s);
    case 3: return launch_eb<3>(a, nb, grid, threads, smem_bytes, s);
    case 4: return launch_eb<4>(a, nb, grid, threads, smem_bytes, s);
    case 5: return launch_eb<5>(a, nb, grid, threads, smem_bytes, s);
    case 6: return launch_eb<6>(a, nb, grid, threads, smem_bytes, s);
    case 7: return launch_eb<7>(a, nb, grid, threads, smem_bytes, s);
    default: return launch_eb<8>(a, nb, grid, threads, smem_bytes, s);
  }
}

}  // namespace vq
