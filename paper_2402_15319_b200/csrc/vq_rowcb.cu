// Tuned skinny-GEMM kernels for formats whose codebooks belong to ONE row (block_rows == 1) and
// are indexed by 4-bit indices: the "mobile LUT" layouts (16-entry int8 codebook + fp16 scale per
// row segment) and the 16-entry fp16 2-D codebooks.
//
// Work decomposition.  A warp owns a tile of 16 rows and walks a range of columns in steps of
// STEP_COLS columns.  Lane (g = lane/4, t = lane%4) streams, with one 128-bit load per row and
// step, the 32 indices of rows g and g+8 that cover its quarter of the step, one step ahead of
// their use.  The indices are expanded to fp16 weights in registers and fed, as the A fragment,
// to mma.sync m16n8k16; the activations are the B fragment (batch row = g), accumulation is fp32.
// Two ways of expanding an index:
//   * PrmtI8: the row's 16 int8 entries live in 4 registers per VQ dimension and are looked up
//     with byte permutes - the register-file analogue of the paper's LUT instruction (Sec. 3.2:
//     index -> 8-bit value).  The bytes become fp16 by the 0x6400 exponent trick, exactly.
//   * LdsTbl: the rows' entries are expanded once per block into lane-private fp16 tables in
//     shared memory (bank = lane: conflict-free for any index pattern) and gathered with ld.shared.
// Which weight column sits in which reduction slot of the mma is free; the activations of the
// CTA's column range are staged once in shared memory in exactly the order the lanes consume them.
// int8 codebooks: the block scale multiplies the block's fp32 partial sum (Sec. 3.1 scale factor).
// The K dimension is split over the warps of a CTA and over the CTAs of a thread block cluster;
// partial sums meet in the shared memory of cluster rank 0 and are added in a fixed order.
#include <cstdlib>

#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

using namespace dev;

struct RowArgs {
  const uint8_t* idx;
  const uint8_t* cb;
  const __half* scale;
  const __half* X;
  __half* Y;
  long long stride;     // bytes between index rows
  int N, K, batch;
  int n_steps;          // K / STEP_COLS
  int steps_per_block;  // block_cols / STEP_COLS
  int blocks_per_row;   // K / block_cols
  int WR, WK;           // warps of a CTA: row tiles x K parts
  // dynamic shared memory, from its first 4096-byte boundary: warp-private tables, then the
  // activations (x_offset), then the reduction buffer (red_offset)
  int x_offset;
  int red_offset;
};

constexpr uint32_t kMagic = 0x64646464u;      // high byte of fp16 1024.0
constexpr uint32_t kBias2 = 0x64806480u;      // fp16 pair (1152, 1152) = 1024 + 128

__device__ __forceinline__ uint32_t sub_bias(uint32_t h) {
  uint32_t r;
  asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(h), "r"(kBias2));
  return r;
}

// ---------------------------------------------------------------------------------------------
// PrmtI8<D>: 16 int8 entries of D dims per (row, block); register LUT.
// ---------------------------------------------------------------------------------------------
template <int D_>
struct PrmtI8 {
  static constexpr int D = D_;
  static constexpr int STEP_COLS = 128 * D;   // 4 lanes x 32 indices x D
  static constexpr int CHUNKS = 4 * D;        // 8-column activation chunks per lane and step
  static constexpr bool SCALED = true;
  static constexpr int TABLE_BYTES_PER_WARP = 0;
  static constexpr int CB_ROW_BYTES = 16 * D;

  // order in which a lane consumes the 8 activations of a chunk
  static __device__ __forceinline__ uint4 permute_x(uint4 in) {
    if constexpr (D == 1) {
      return in;
    } else {
      return make_uint4(prmt(in.x, in.z, 0x5410), prmt(in.y, in.w, 0x5410), prmt(in.x, in.z, 0x7632),
                        prmt(in.y, in.w, 0x7632));
    }
  }

  struct State {
    uint32_t T[2][D][4];   // [row g / g+8][plane][entries 4q..4q+3], biased by +128
    const uint8_t* cb_row[2];
    const __half* sc_row[2];
    float sc[2];

    __device__ __forceinline__ void init(const RowArgs& a, int rl, int rh, int, uint32_t) {
      cb_row[0] = a.cb + static_cast<long long>(rl) * a.blocks_per_row * CB_ROW_BYTES;
      cb_row[1] = a.cb + static_cast<long long>(rh) * a.blocks_per_row * CB_ROW_BYTES;
      sc_row[0] = a.scale + static_cast<long long>(rl) * a.blocks_per_row;
      sc_row[1] = a.scale + static_cast<long long>(rh) * a.blocks_per_row;
    }

    __device__ __forceinline__ void load_block(int blk) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint8_t* p = cb_row[h] + static_cast<long long>(blk) * CB_ROW_BYTES;
        if constexpr (D == 1) {
          const uint4 v = ldg128_nc(p);
          T[h][0][0] = v.x ^ 0x80808080u; T[h][0][1] = v.y ^ 0x80808080u;
          T[h][0][2] = v.z ^ 0x80808080u; T[h][0][3] = v.w ^ 0x80808080u;
        } else {
          const uint4 v0 = ldg128_nc(p), v1 = ldg128_nc(p + 16);
          const uint32_t w[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            T[h][0][q] = prmt(w[2 * q], w[2 * q + 1], 0x6420) ^ 0x80808080u;
            T[h][1][q] = prmt(w[2 * q], w[2 * q + 1], 0x7531) ^ 0x80808080u;
          }
        }
        sc[h] = __half2float(__ldg(sc_row[h] + blk));
      }
    }

    // 4 looked-up bytes (indices i0..i0+3 of the word, plane p) of row h
    __device__ __forceinline__ uint32_t look4(int h, int p, uint32_t sel, uint32_t pick) const {
      const uint32_t lo = prmt(T[h][p][0], T[h][p][1], sel);
      const uint32_t hi = prmt(T[h][p][2], T[h][p][3], sel);
      return prmt(lo, hi, pick);
    }

    // One index word of each row (8 indices = 8*D columns) -> A fragments of 2*D mma steps.
    // a[c][q][.]: chunk c of the word, mma q of the chunk, registers a0..a3.
    __device__ __forceinline__ void decode(uint32_t wl, uint32_t wh, uint32_t (&a)[D][2][4]) const {
      const uint32_t w[2] = {wl, wh};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t sel = w[h] & 0x77777777u;
        const uint32_t pick = ((w[h] >> 1) & 0x44444444u) | 0x32103210u;
        const uint32_t selH = sel >> 16, pickH = pick >> 16;
        if constexpr (D == 1) {
          const uint32_t rL = look4(h, 0, sel, pick), rH = look4(h, 0, selH, pickH);
          a[0][0][h] = sub_bias(prmt(rL, kMagic, 0x4140));
          a[0][0][h + 2] = sub_bias(prmt(rL, kMagic, 0x4342));
          a[0][1][h] = sub_bias(prmt(rH, kMagic, 0x4140));
          a[0][1][h + 2] = sub_bias(prmt(rH, kMagic, 0x4342));
        } else {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const uint32_t r0 = look4(h, 0, c ? selH : sel, c ? pickH : pick);
            const uint32_t r1 = look4(h, 1, c ? selH : sel, c ? pickH : pick);
            a[c][0][h] = sub_bias((r0 & 0x00FF00FFu) | 0x64006400u);   // columns 0,4 of the chunk
            a[c][0][h + 2] = sub_bias(prmt(r0, kMagic, 0x4341));         // columns 2,6
            a[c][1][h] = sub_bias((r1 & 0x00FF00FFu) | 0x64006400u);   // columns 1,5
            a[c][1][h + 2] = sub_bias(prmt(r1, kMagic, 0x4341));         // columns 3,7
          }
        }
      }
    }
  };
};

// ---------------------------------------------------------------------------------------------
// LdsTbl<INT8>: 16 entries of 2 dims per (row, block), fp16 or int8; lane-private fp16 tables in
// shared memory: word (half, entry, lane) at half*2048 + entry*128 + lane*4.
// ---------------------------------------------------------------------------------------------
template <bool INT8>
struct LdsTbl {
  static constexpr int D = 2;
  static constexpr int STEP_COLS = 256;
  static constexpr int CHUNKS = 8;
  static constexpr bool SCALED = INT8;
  static constexpr int TABLE_BYTES_PER_WARP = 4096;
  static constexpr int CB_ROW_BYTES = INT8 ? 32 : 64;

  static __device__ __forceinline__ uint4 permute_x(uint4 in) { return in; }

  struct State {
    const uint8_t* cb_row[2];
    const __half* sc_row[2];
    float sc[2];
    uint32_t tbl;   // shared address of this lane's column of the table
    uint32_t fill;  // shared address this lane writes when building the table

    __device__ __forceinline__ void init(const RowArgs& a, int rl, int rh, int lane, uint32_t warp_tbl) {
      const int t = lane & 3, g = lane >> 2;
      cb_row[0] = a.cb + static_cast<long long>(rl) * a.blocks_per_row * CB_ROW_BYTES + t * (CB_ROW_BYTES / 4);
      cb_row[1] = a.cb + static_cast<long long>(rh) * a.blocks_per_row * CB_ROW_BYTES + t * (CB_ROW_BYTES / 4);
      if constexpr (INT8) {
        sc_row[0] = a.scale + static_cast<long long>(rl) * a.blocks_per_row;
        sc_row[1] = a.scale + static_cast<long long>(rh) * a.blocks_per_row;
      }
      tbl = warp_tbl + lane * 4;
      fill = warp_tbl + (4 * t) * 128 + g * 16;   // entries 4t..4t+3, the 4 copies of row g
    }

    // Lane (g, t) fetches entries 4t..4t+3 of rows g and g+8 and writes each 4 times (one copy
    // per lane of the row's quad).
    __device__ __forceinline__ void load_block(int blk) {
      __syncwarp();   // every lane is done with the previous block's table
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint8_t* p = cb_row[h] + static_cast<long long>(blk) * CB_ROW_BYTES;
        uint32_t e[4];
        if constexpr (INT8) {
          const uint2 v = ldg64_nc(p);   // 4 entries x (c0, c1)
          e[0] = sub_bias(prmt(v.x ^ 0x80808080u, kMagic, 0x4140));
          e[1] = sub_bias(prmt(v.x ^ 0x80808080u, kMagic, 0x4342));
          e[2] = sub_bias(prmt(v.y ^ 0x80808080u, kMagic, 0x4140));
          e[3] = sub_bias(prmt(v.y ^ 0x80808080u, kMagic, 0x4342));
          sc[h] = __half2float(__ldg(sc_row[h] + blk));
        } else {
          const uint4 v = ldg128_nc(p);
          e[0] = v.x; e[1] = v.y; e[2] = v.z; e[3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) sts128(fill + h * 2048 + i * 128, make_uint4(e[i], e[i], e[i], e[i]));
      }
      __syncwarp();
    }

    // shared address of entry (index I of word w) in this lane's column: the 4 index bits are
    // moved to bits 7..10 and merged with the lane's constant address bits by one logic op
    template <int I>
    __device__ __forceinline__ uint32_t entry_addr(uint32_t w, uint32_t base) const {
      constexpr int p = 4 * I;
      uint32_t x;
      if constexpr (p < 7) {
        x = w << (7 - p);
      } else {
#ifdef VQ_SHIFT_VIA_MULHI
        asm("mul.hi.u32 %0, %1, %2;" : "=r"(x) : "r"(w), "n"(1u << (32 - (p - 7))));
#else
        x = w >> (p - 7);
#endif
      }
      return (x & 0x780u) | base;
    }

    __device__ __forceinline__ void decode(uint32_t wl, uint32_t wh, uint32_t (&a)[2][2][4]) const {
      // chunk c = indices 4c..4c+3; mma q of the chunk = indices 4c+2q, 4c+2q+1
      const uint32_t lo = tbl, hi = tbl + 2048;
      a[0][0][0] = lds32(entry_addr<0>(wl, lo));        a[0][0][1] = lds32(entry_addr<0>(wh, hi));
      a[0][0][2] = lds32(entry_addr<1>(wl, lo));        a[0][0][3] = lds32(entry_addr<1>(wh, hi));
      a[0][1][0] = lds32(entry_addr<2>(wl, lo));        a[0][1][1] = lds32(entry_addr<2>(wh, hi));
      a[0][1][2] = lds32(entry_addr<3>(wl, lo));        a[0][1][3] = lds32(entry_addr<3>(wh, hi));
      a[1][0][0] = lds32(entry_addr<4>(wl, lo));        a[1][0][1] = lds32(entry_addr<4>(wh, hi));
      a[1][0][2] = lds32(entry_addr<5>(wl, lo));        a[1][0][3] = lds32(entry_addr<5>(wh, hi));
      a[1][1][0] = lds32(entry_addr<6>(wl, lo));        a[1][1][1] = lds32(entry_addr<6>(wh, hi));
      a[1][1][2] = lds32(entry_addr<7>(wl, lo));        a[1][1][3] = lds32(entry_addr<7>(wh, hi));
    }
  };
};

// ---------------------------------------------------------------------------------------------
// The kernel.  Grid (S, ceil(N / (16*WR))), cluster (S, 1, 1); CTA = WR*WK warps.
// ---------------------------------------------------------------------------------------------
template <class P, int NB>
__global__ void __launch_bounds__(256) rowcb_kernel(const RowArgs a) {
  constexpr int D = P::D;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // the tables' address bits 7..11 must be free for the index and the row half
  const uint32_t smem_base = (smem_u32(smem_raw) + 4095u) & ~4095u;
  unsigned char* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int S = gridDim.x, rank = blockIdx.x;
  if (S > 1) cluster_arrive_relaxed();   // matched by the wait in front of the first remote store
  pdl_launch_dependents();

  const int wr = warp % a.WR, wk = warp / a.WR;
  const int T = S * a.WK;
  const int part = rank * a.WK + wk;
  const int cta_s0 = a.n_steps * (rank * a.WK) / T;
  const int cta_s1 = a.n_steps * ((rank + 1) * a.WK) / T;
  const int s0 = a.n_steps * part / T, s1 = a.n_steps * (part + 1) / T;

  const int tile = blockIdx.y * a.WR + wr;
  const int r_lo = tile * 16 + g, r_hi = r_lo + 8;
  const int rl = min(r_lo, a.N - 1), rh = min(r_hi, a.N - 1);   // tail rows load a valid row, store nothing
  const uint8_t* pl = a.idx + rl * a.stride + t * 16;
  const uint8_t* ph = a.idx + rh * a.stride + t * 16;

  typename P::State st;
  st.init(a, rl, rh, lane, smem_base + warp * P::TABLE_BYTES_PER_WARP);

  // indices of the first step and the first block's tables: weights do not depend on the
  // previous kernel, so they are requested before the dependency wait
  uint4 nl = make_uint4(0, 0, 0, 0), nh = nl;
  pl += static_cast<long long>(s0) * 64;
  ph += static_cast<long long>(s0) * 64;
  if (s0 < s1) {
    nl = ldg128_stream(pl);
    nh = ldg128_stream(ph);
    st.load_block(s0 / a.steps_per_block);
  }

  // ---- activations of the CTA's column range, in consumption order ----
  pdl_wait();
  {
    const int col0 = cta_s0 * P::STEP_COLS;
    const int n8 = (cta_s1 - cta_s0) * (P::STEP_COLS / 8);
    uint4* xs = reinterpret_cast<uint4*>(smem + a.x_offset);
    for (int m = 0; m < a.batch; ++m) {
      const uint4* src = reinterpret_cast<const uint4*>(a.X + static_cast<long long>(m) * a.K + col0);
      for (int c8 = tid; c8 < n8; c8 += blockDim.x) {
        const int col = c8 * 8;
        const int step = col / P::STEP_COLS, within = col % P::STEP_COLS;
        const int tt = within / (P::STEP_COLS / 4), chunk = (within % (P::STEP_COLS / 4)) / 8;
        xs[((step * P::CHUNKS + chunk) * a.batch + m) * 4 + tt] = P::permute_x(__ldg(src + c8));
      }
    }
  }
  __syncthreads();

  float acc[NB][4], total[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[nb][e] = total[nb][e] = 0.f;

  bool on[NB];
  uint32_t xaddr[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    on[nb] = nb * 8 + g < a.batch;
    xaddr[nb] = smem_base + a.x_offset + (((s0 - cta_s0) * P::CHUNKS * a.batch + nb * 8 + g) * 4 + t) * 16;
  }
  const uint32_t xstride = a.batch * 64;   // bytes between consecutive chunks

  int in_blk = s0 % a.steps_per_block, blk = s0 / a.steps_per_block;
  for (int s = s0; s < s1; ++s) {
    const uint4 cl = nl, ch = nh;
    pl += 64;
    ph += 64;
    if (s + 1 < s1) {
      nl = ldg128_stream(pl);
      nh = ldg128_stream(ph);
    }
    const uint32_t wl[4] = {cl.x, cl.y, cl.z, cl.w}, wh[4] = {ch.x, ch.y, ch.z, ch.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t af[D][2][4];
      st.decode(wl[j], wh[j], af);
#pragma unroll
      for (int c = 0; c < D; ++c) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          uint4 xb = make_uint4(0, 0, 0, 0);
          if (on[nb]) xb = lds128(xaddr[nb] + (j * D + c) * xstride);
          mma16816(acc[nb], af[c][0][0], af[c][0][1], af[c][0][2], af[c][0][3], xb.x, xb.y);
          mma16816(acc[nb], af[c][1][0], af[c][1][1], af[c][1][2], af[c][1][3], xb.z, xb.w);
        }
      }
    }
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) xaddr[nb] += P::CHUNKS * xstride;
    if (++in_blk == a.steps_per_block || s + 1 == s1) {
      // end of a codebook block: apply its scale to the block's partial sums
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        if constexpr (P::SCALED) {
          total[nb][0] = fmaf(st.sc[0], acc[nb][0], total[nb][0]);
          total[nb][1] = fmaf(st.sc[0], acc[nb][1], total[nb][1]);
          total[nb][2] = fmaf(st.sc[1], acc[nb][2], total[nb][2]);
          total[nb][3] = fmaf(st.sc[1], acc[nb][3], total[nb][3]);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
        }
      }
      in_blk = 0;
      ++blk;
      if (s + 1 < s1) st.load_block(blk);
    }
  }
  if constexpr (!P::SCALED) {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) total[nb][e] = acc[nb][e];
  }

  // ---- combine the K parts ----
  // total[nb][e]: row g + 8*(e/2) of the tile, batch row nb*8 + 2t + (e&1)
  if (T == 1) {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = (e >> 1) ? r_hi : r_lo, n = nb * 8 + 2 * t + (e & 1);
        if (r < a.N && n < a.batch) a.Y[static_cast<long long>(n) * a.N + r] = __float2half_rn(total[nb][e]);
      }
    return;
  }
  // red[part][wr][row 0..15][n 0..8*NB-1] in the shared memory of cluster rank 0
  const uint32_t red_local = smem_base + a.red_offset;
  const uint32_t mine = red_local + (((part * a.WR + wr) * 16 + g) * (8 * NB) + 2 * t) * 4;
  if (S > 1) {
    cluster_wait_acquire();   // every CTA of the cluster has started: rank 0's shared memory exists
    const uint32_t dst = map_to_rank(mine, 0);
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        st_cluster_f32(dst + (((e >> 1) * 8 * (8 * NB)) + nb * 8 + (e & 1)) * 4, total[nb][e]);
    cluster_arrive_release();
    cluster_wait_acquire();
  } else {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) sts32f(mine + (((e >> 1) * 8 * (8 * NB)) + nb * 8 + (e & 1)) * 4, total[nb][e]);
    __syncthreads();
  }
  if (rank != 0) return;
  const float* red = reinterpret_cast<const float*>(smem + a.red_offset);
  const int cta_rows = a.WR * 16;
  const int row_base = blockIdx.y * cta_rows;
  for (int o = tid; o < cta_rows * a.batch; o += blockDim.x) {
    const int n = o / cta_rows, rr = o % cta_rows;
    const int r = row_base + rr;
    if (r >= a.N) continue;
    float sum = 0.f;
    for (int p = 0; p < T; ++p) sum += red[((p * a.WR) * 16 + rr) * (8 * NB) + n];
    a.Y[static_cast<long long>(n) * a.N + r] = __float2half_rn(sum);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
struct Plan {
  int WR, WK, S;
};

int env_int(const char* name, int dflt) {
#ifdef VQ_TUNING
  if (const char* e = getenv(name)) return atoi(e);
#else
  (void)name;
#endif
  return dflt;
}

// Choose the CTA shape and the K split.  Targets: about 16 resident warps per SM, at least two
// steps per warp, many more CTAs than SMs for large layers (the hardware balances them).
Plan make_plan(int N, int n_steps, int sms) {
  const int row_tiles = (N + 15) / 16;
  const long long want_warps = static_cast<long long>(sms) * 16;
  int T = static_cast<int>((want_warps + row_tiles - 1) / row_tiles);
  int max_T = n_steps / 2;
  if (max_T < 1) max_T = 1;
  if (T > max_T) T = max_T;
  if (T > 64) T = 64;
  // round down to a power of two
  int p = 1;
  while (2 * p <= T) p *= 2;
  T = p;
  Plan pl;
  pl.WK = T < 8 ? T : 8;
  pl.S = T / pl.WK;
  pl.WR = 8 / pl.WK;
  if (T == 1) pl.WR = 4;   // large layers: 64-row CTAs
  pl.WK = env_int("VQ_WK", pl.WK);
  pl.WR = env_int("VQ_WR", pl.WR);
  pl.S = env_int("VQ_S", pl.S);
  return pl;
}

template <class P, int NB>
vq_status launch(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, cudaStream_t s) {
  if (g.K % P::STEP_COLS || g.Bc % P::STEP_COLS) return VQ_ERR_UNSUPPORTED;
  // per device, once: SM count and the opt-in to large dynamic shared memory
  static int sms_of[kMaxDevices] = {};
  auto kern = rowcb_kernel<P, NB>;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (sms_of[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return VQ_ERR_CUDA;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return VQ_ERR_CUDA;
    sms_of[dev] = n;
  }
  const int sms = sms_of[dev];
  RowArgs a;
  a.idx = p.idx;
  a.cb = static_cast<const uint8_t*>(p.cb);
  a.scale = p.scale;
  a.X = X;
  a.Y = Y;
  a.stride = g.stride;
  a.N = g.N;
  a.K = g.K;
  a.batch = batch;
  a.n_steps = g.K / P::STEP_COLS;
  a.steps_per_block = g.Bc / P::STEP_COLS;
  a.blocks_per_row = g.blocks_per_row;
  Plan pl = make_plan(g.N, a.n_steps, sms);
  // activations of a CTA's column range must fit in shared memory: split K further if not
  size_t x_bytes, red_bytes, tbl_bytes;
  for (;;) {
    const int T = pl.S * pl.WK;
    int cta_steps = 0;
    for (int r = 0; r < pl.S; ++r) {
      const int c = a.n_steps * ((r + 1) * pl.WK) / T - a.n_steps * (r * pl.WK) / T;
      if (c > cta_steps) cta_steps = c;
    }
    x_bytes = static_cast<size_t>(cta_steps) * P::STEP_COLS * 2 * batch;
    red_bytes = T > 1 ? static_cast<size_t>(T) * pl.WR * 16 * 8 * NB * sizeof(float) : 0;
    tbl_bytes = static_cast<size_t>(P::TABLE_BYTES_PER_WARP) * pl.WR * pl.WK;
    if (x_bytes + red_bytes + tbl_bytes <= 160 * 1024) break;
    if (pl.S >= 8 || pl.S * 2 * pl.WK > a.n_steps) return VQ_ERR_UNSUPPORTED;
    pl.S *= 2;
  }
  if (pl.S * pl.WK > a.n_steps) return VQ_ERR_UNSUPPORTED;
  a.WR = pl.WR;
  a.WK = pl.WK;
  a.x_offset = static_cast<int>(tbl_bytes);
  a.red_offset = static_cast<int>(tbl_bytes + (x_bytes + 15) / 16 * 16);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.S, (g.N + 16 * pl.WR - 1) / (16 * pl.WR), 1);
  cfg.blockDim = dim3(32 * pl.WR * pl.WK, 1, 1);
  cfg.dynamicSmemBytes = a.red_offset + red_bytes + 4096;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (pl.S > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = pl.S;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  if (env_int("VQ_PDL", 1)) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  if (cudaLaunchKernelEx(&cfg, kern, a) != cudaSuccess) return VQ_ERR_CUDA;
  return check_launch();
}

}  // namespace

// Per-row codebook families (block_rows == 1, 4-bit indices).
vq_status launch_gemm_rowcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                            cudaStream_t s) {
  if (g.Br != 1 || g.b != 4) return VQ_ERR_UNSUPPORTED;
  const bool nb1 = batch <= 8;
  if (g.cb_int8) {
    const int use_lds = env_int("VQ_I8_LDS", 0);
    if (g.d == 1) return nb1 ? launch<PrmtI8<1>, 1>(g, p, X, Y, batch, s) : launch<PrmtI8<1>, 2>(g, p, X, Y, batch, s);
    if (g.d == 2) {
      if (use_lds) return nb1 ? launch<LdsTbl<true>, 1>(g, p, X, Y, batch, s) : launch<LdsTbl<true>, 2>(g, p, X, Y, batch, s);
      return nb1 ? launch<PrmtI8<2>, 1>(g, p, X, Y, batch, s) : launch<PrmtI8<2>, 2>(g, p, X, Y, batch, s);
    }
    return VQ_ERR_UNSUPPORTED;
  }
  if (g.d == 2) return nb1 ? launch<LdsTbl<false>, 1>(g, p, X, Y, batch, s) : launch<LdsTbl<false>, 2>(g, p, X, Y, batch, s);
  return VQ_ERR_UNSUPPORTED;
}

}  // namespace vq
