// Tuned skinny-GEMM kernels for formats whose codebooks belong to ONE row (block_rows == 1) and
// are indexed by 4-bit indices: the layouts of the mobile LUT decode (16-entry int8 codebook + fp16 scale per
// row segment) and the 16-entry fp16 2-D codebooks.
//
// Work decomposition.  A CTA owns WR tiles of 16 rows and a column range; warp (wr, wk) walks part
// wk of that range for tile wr in steps of STEP_COLS columns.  Lane (g = lane/4, t = lane%4)
// streams, with one 128-bit load per row and step, the 32 indices of rows g and g+8 that cover
// its quarter of the step, a few steps ahead of their use.  The indices are expanded to fp16
// weights in registers and fed, as the A fragment, to mma.sync m16n8k16; the activations are the
// B fragment (batch row = g), staged once per CTA in shared memory in the order the lanes
// consume them and read only by the lanes whose batch row exists; accumulation is fp32.
// Two ways of expanding an index:
//   * PrmtI8 (1-D int8 codebooks): the row's 16 entries live in 4 registers and are looked up
//     with byte permutes - the register-file analogue of the paper's LUT instruction (Sec. 3.2:
//     index -> 8-bit value).  The bytes become fp16 by the 0x6400 exponent trick, exactly.
//   * LdsTbl (2-D codebooks, fp16 or int8): the rows' entries are expanded once per block into
//     lane-private fp16 tables in shared memory (bank = lane: conflict-free for any index
//     pattern) and gathered with ld.shared; index bits and the lane's address bits are merged by
//     one logic operation.
// int8 codebooks: the block scale multiplies the block's fp32 partial sum (Sec. 3.1 scale factor).
// Partial sums of the K parts (warps of the CTA, CTAs of a thread block cluster) meet in the
// shared memory of cluster rank 0 and are added in a fixed order.
#include <cstdio>
#include <cstdlib>

#include "vq_common.cuh"
#include "vq_device.cuh"

#ifndef VQ_ROW_MIN_CTAS
#define VQ_ROW_MIN_CTAS 1   // resident 256-thread CTAs per SM the register budget allows
#endif
#ifndef VQ_ROW_PREFETCH
#define VQ_ROW_PREFETCH 2   // steps of the index stream a lane keeps in flight
#endif

namespace vq {
namespace {

using namespace dev;

struct RowArgs {
  const uint8_t* idx;
  const uint8_t* cb;
  const __half* scale;
  const __half* X;
  __half* Y;
  int* error_flag;      // device counter of waits that ran out
  long long stride;     // bytes between index rows
  int N, K, batch;
  int n_steps;          // K / STEP_COLS
  int steps_per_block;  // block_cols / STEP_COLS
  int blocks_per_row;   // K / block_cols
  int Br;               // rows that share a codebook block (1 for per-row codebooks)
  int WR, WK;           // warps of a CTA: row tiles x K parts
  // dynamic shared memory, from its first 4096-byte boundary: warp-private tables, then the
  // activations (x_offset), then the reduction buffer (red_offset)
  int x_offset;
  int red_offset;
  int bar_offset;   // receive barrier of the reduction (8 bytes), behind the reduction buffer
};

constexpr int kWaitTries = 1 << 18;            // mbarrier polls before rank 0 gives up and flags an error
constexpr uint32_t kMagic = 0x64646464u;      // high byte of fp16 1024.0
constexpr uint32_t kBias2 = 0x64806480u;      // fp16 pair (1152, 1152) = 1024 + 128

// (1024 + u) - 1152 = u - 128, exact in fp16
__device__ __forceinline__ uint32_t sub_bias(uint32_t h) {
  uint32_t r;
  asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(h), "r"(kBias2));
  return r;
}

// ---------------------------------------------------------------------------------------------
// PrmtI8: 16 int8 entries of 1 dim per (row, block); register LUT.
// ---------------------------------------------------------------------------------------------
struct PrmtI8 {
  static constexpr int D = 1;
  static constexpr int STEP_COLS = 128;       // 4 lanes x 32 indices
  static constexpr int WORD_CHUNKS = 1;       // 8-column activation chunks per index word
  static constexpr bool SCALED = true;
  static constexpr int TABLE_BYTES_PER_WARP = 0;
  static constexpr int CB_ROW_BYTES = 16;
  static __device__ __forceinline__ uint4 permute_x(uint4 in) { return in; }   // natural column order

  struct State {
    uint32_t T[2][4];   // [row g / g+8][entries 4q..4q+3], biased by +128
    const uint8_t* cb_row[2];
    const __half* sc_row[2];
    float sc[2];

    __device__ __forceinline__ void init(const RowArgs& a, int, int rl, int rh, int, uint32_t) {
      cb_row[0] = a.cb + static_cast<long long>(rl / a.Br) * a.blocks_per_row * CB_ROW_BYTES;
      cb_row[1] = a.cb + static_cast<long long>(rh / a.Br) * a.blocks_per_row * CB_ROW_BYTES;
      sc_row[0] = a.scale + static_cast<long long>(rl / a.Br) * a.blocks_per_row;
      sc_row[1] = a.scale + static_cast<long long>(rh / a.Br) * a.blocks_per_row;
    }

    uint4 raw[2];     // requested entries of the next block
    float sc_raw[2];

    // Request the entries and the scale of block blk (global loads, not waited for here) ...
    __device__ __forceinline__ void fetch(int blk) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        raw[h] = ldg128_nc(cb_row[h] + static_cast<long long>(blk) * CB_ROW_BYTES);
        sc_raw[h] = __half2float(__ldg(sc_row[h] + blk));
      }
    }
    // ... and make them the current look-up table.
    __device__ __forceinline__ void install() {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        T[h][0] = raw[h].x ^ 0x80808080u; T[h][1] = raw[h].y ^ 0x80808080u;
        T[h][2] = raw[h].z ^ 0x80808080u; T[h][3] = raw[h].w ^ 0x80808080u;
        sc[h] = sc_raw[h];
      }
    }

    // One index word of each row (8 indices = 8 columns) -> A fragments of 2 mma steps.
    // a[c][q][.]: chunk c of the word, mma q of the chunk, registers a0..a3.
    __device__ __forceinline__ void decode(uint32_t wl, uint32_t wh, uint32_t (&a)[1][2][4]) const {
      const uint32_t w[2] = {wl, wh};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        // byte permute: selector nibble = entry mod 8 (bit 3 would mean "replicate sign"), looked
        // up in entries 0..7 and 8..15; a second permute picks per index by the index's bit 3
        const uint32_t sel = w[h] & 0x77777777u;
        const uint32_t pick = ((w[h] >> 1) & 0x44444444u) | 0x32103210u;
        const uint32_t rL = prmt(prmt(T[h][0], T[h][1], sel), prmt(T[h][2], T[h][3], sel), pick);
        const uint32_t rH = prmt(prmt(T[h][0], T[h][1], sel >> 16), prmt(T[h][2], T[h][3], sel >> 16), pick >> 16);
        a[0][0][h] = sub_bias(prmt(rL, kMagic, 0x4140));       // columns 0,1
        a[0][0][h + 2] = sub_bias(prmt(rL, kMagic, 0x4342));   // columns 2,3
        a[0][1][h] = sub_bias(prmt(rH, kMagic, 0x4140));       // columns 4,5
        a[0][1][h + 2] = sub_bias(prmt(rH, kMagic, 0x4342));   // columns 6,7
      }
    }
  };
};

// ---------------------------------------------------------------------------------------------
// LdsTbl<INT8>: 16 entries of 2 dims per (row, block), fp16 or int8; lane-private fp16 tables in
// shared memory, 4096-byte aligned per warp: word (half, entry, lane) at half*2048 + entry*128 +
// lane*4, so the entry index occupies address bits 7..10 and never carries.
// ---------------------------------------------------------------------------------------------
template <bool INT8>
struct LdsTbl {
  static constexpr int D = 2;
  static constexpr int STEP_COLS = 256;
  static constexpr int WORD_CHUNKS = 2;
  static constexpr bool SCALED = INT8;
  static constexpr int TABLE_BYTES_PER_WARP = 4096;
  static constexpr int CB_ROW_BYTES = INT8 ? 32 : 64;
  static __device__ __forceinline__ uint4 permute_x(uint4 in) { return in; }   // natural column order

  struct State {
    const uint8_t* cb_row[2];
    const __half* sc_row[2];
    float sc[2];
    uint32_t tbl;   // shared address of this lane's column of the table
    uint32_t fill;  // shared address this lane writes when building the table

    // The table is BUILT with a different lane mapping than it is read with: lane l fetches
    // entries 4*(l/8)..+3 of rows l%8 and l%8+8, so that the 8 lanes of a quarter warp write 8
    // different 16-byte bank groups (conflict-free 128-bit stores).
    __device__ __forceinline__ void init(const RowArgs& a, int row0, int rl, int rh, int lane, uint32_t warp_tbl) {
      const int gb = lane & 7, tb = lane >> 3;
      const int b_lo = min(row0 + gb, a.N - 1), b_hi = min(row0 + gb + 8, a.N - 1);
      cb_row[0] = a.cb + static_cast<long long>(b_lo / a.Br) * a.blocks_per_row * CB_ROW_BYTES + tb * (CB_ROW_BYTES / 4);
      cb_row[1] = a.cb + static_cast<long long>(b_hi / a.Br) * a.blocks_per_row * CB_ROW_BYTES + tb * (CB_ROW_BYTES / 4);
      if constexpr (INT8) {
        sc_row[0] = a.scale + static_cast<long long>(rl / a.Br) * a.blocks_per_row;
        sc_row[1] = a.scale + static_cast<long long>(rh / a.Br) * a.blocks_per_row;
      }
      tbl = warp_tbl + lane * 4;
      fill = warp_tbl + (4 * tb) * 128 + gb * 16;   // entries 4tb..4tb+3, the 4 copies of row gb
    }

    uint32_t raw[2][4];   // requested entries of the next block (int8: still packed)
    float sc_raw[2];

    // Request this lane's share of the entries (and the scales) of block blk; not waited for here.
    __device__ __forceinline__ void fetch(int blk) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint8_t* p = cb_row[h] + static_cast<long long>(blk) * CB_ROW_BYTES;
        if constexpr (INT8) {
          const uint2 v = ldg64_nc(p);   // 4 entries x (c0, c1)
          raw[h][0] = v.x; raw[h][1] = v.y; raw[h][2] = raw[h][3] = 0u;
          sc_raw[h] = __half2float(__ldg(sc_row[h] + blk));
        } else {
          const uint4 v = ldg128_nc(p);
          raw[h][0] = v.x; raw[h][1] = v.y; raw[h][2] = v.z; raw[h][3] = v.w;
        }
      }
    }

    // Build the table from the requested entries: each is written 4 times (one copy per lane of the
    // row's quad).
    __device__ __forceinline__ void install() {
      uint32_t e[2][4];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if constexpr (INT8) {
          e[h][0] = sub_bias(prmt(raw[h][0] ^ 0x80808080u, kMagic, 0x4140));
          e[h][1] = sub_bias(prmt(raw[h][0] ^ 0x80808080u, kMagic, 0x4342));
          e[h][2] = sub_bias(prmt(raw[h][1] ^ 0x80808080u, kMagic, 0x4140));
          e[h][3] = sub_bias(prmt(raw[h][1] ^ 0x80808080u, kMagic, 0x4342));
          sc[h] = sc_raw[h];
        } else {
#pragma unroll
          for (int i = 0; i < 4; ++i) e[h][i] = raw[h][i];
        }
      }
      __syncwarp();   // every lane is done with the previous block's table
#pragma unroll
      for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int i = 0; i < 4; ++i) sts128(fill + h * 2048 + i * 128, make_uint4(e[h][i], e[h][i], e[h][i], e[h][i]));
      __syncwarp();
      fence_value(tbl);   // gathers of the new block stay behind the rewrite
    }

    template <int I, int HALF>
    __device__ __forceinline__ uint32_t gather(uint32_t w) const {
      constexpr int p = 4 * I;
      const uint32_t x = p < 7 ? w << (7 - p) : w >> (p - 7);
      return lds32_off<HALF * 2048>((x & 0x780u) | tbl);
    }

    __device__ __forceinline__ void decode(uint32_t wl, uint32_t wh, uint32_t (&a)[2][2][4]) const {
      // chunk c = indices 4c..4c+3; mma q of the chunk = indices 4c+2q, 4c+2q+1
      a[0][0][0] = gather<0, 0>(wl); a[0][0][1] = gather<0, 1>(wh); a[0][0][2] = gather<1, 0>(wl); a[0][0][3] = gather<1, 1>(wh);
      a[0][1][0] = gather<2, 0>(wl); a[0][1][1] = gather<2, 1>(wh); a[0][1][2] = gather<3, 0>(wl); a[0][1][3] = gather<3, 1>(wh);
      a[1][0][0] = gather<4, 0>(wl); a[1][0][1] = gather<4, 1>(wh); a[1][0][2] = gather<5, 0>(wl); a[1][0][3] = gather<5, 1>(wh);
      a[1][1][0] = gather<6, 0>(wl); a[1][1][1] = gather<6, 1>(wh); a[1][1][2] = gather<7, 0>(wl); a[1][1][3] = gather<7, 1>(wh);
    }
  };
};

// ---------------------------------------------------------------------------------------------
// Int4G128: the uniform INT4 group-128 yard-stick run through the same skeleton (paper Sec. 2.1
// symmetric uniform quantiser x ~ s*x_int; Sec. 5: uniform 4-bit weights with a scale per 128 columns).  No table: a nibble q becomes the
// fp16 value q - 8 by the exponent trick, (1024 + q) - 1032; a "block" is one 128-column group whose
// fp16 scale multiplies the group's fp32 partial sum.  The two nibbles that share a mask
// (columns c and c+4 of an 8-column word) land in one fp16 pair, so the activations are staged in
// the matching order.
// ---------------------------------------------------------------------------------------------
struct Int4G128 {
  static constexpr int D = 1;
  static constexpr int STEP_COLS = 128;
  static constexpr int WORD_CHUNKS = 1;
  static constexpr bool SCALED = true;
  static constexpr int TABLE_BYTES_PER_WARP = 0;
  // (x0x1, x2x3, x4x5, x6x7) -> (x0x4, x1x5, x2x6, x3x7)
  static __device__ __forceinline__ uint4 permute_x(uint4 in) {
    return make_uint4(prmt(in.x, in.z, 0x5410), prmt(in.x, in.z, 0x7632), prmt(in.y, in.w, 0x5410), prmt(in.y, in.w, 0x7632));
  }

  struct State {
    const __half* sc_row[2];
    float sc[2], sc_next[2];
    int n_blocks;

    __device__ __forceinline__ void init(const RowArgs& a, int, int rl, int rh, int, uint32_t) {
      sc_row[0] = a.scale + static_cast<long long>(rl) * a.blocks_per_row;
      sc_row[1] = a.scale + static_cast<long long>(rh) * a.blocks_per_row;
      n_blocks = a.blocks_per_row;
    }

    __device__ __forceinline__ void fetch(int blk) {
#pragma unroll
      for (int h = 0; h < 2; ++h) sc_next[h] = __half2float(__ldg(sc_row[h] + blk));
    }
    __device__ __forceinline__ void install() {
      sc[0] = sc_next[0];
      sc[1] = sc_next[1];
    }

    __device__ __forceinline__ void decode(uint32_t wl, uint32_t wh, uint32_t (&a)[1][2][4]) const {
      constexpr uint32_t kBias1032 = 0x64086408u;   // fp16 pair (1032, 1032) = 1024 + 8
      const uint32_t w[2] = {wl, wh};
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        uint32_t p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t m = ((w[h] >> (4 * i)) & 0x000F000Fu) | 0x64006400u;   // nibbles i and i+4
          asm("sub.f16x2 %0, %1, %2;" : "=r"(p[i]) : "r"(m), "r"(kBias1032));
        }
        a[0][0][h] = p[0];       // columns 0,4
        a[0][0][h + 2] = p[1];   // columns 1,5
        a[0][1][h] = p[2];       // columns 2,6
        a[0][1][h + 2] = p[3];   // columns 3,7
      }
    }
  };
};

// ---------------------------------------------------------------------------------------------
// The kernel.  Grid (S, ceil(N / (16*WR))), cluster (S, 1, 1); CTA = WR*WK warps.
// Activations in shared memory: 16-byte chunk (step, chunk c of the lane's columns, batch row m,
// lane quarter t) at index ((step*CHUNKS + c)*batch + m)*4 + t, so that the lanes of a warp that
// read (those with g < batch) touch consecutive chunks.
// ---------------------------------------------------------------------------------------------
// XS: the activations are not staged for the CTA's whole column range but streamed in windows of
// kWindow steps per column part (two buffers, cp.async one window ahead, a barrier among the warps
// of the part at every window): the shared memory they take no longer grows with K, which at batch
// 16 is what limits the CTAs per SM (used for the two-tile batch variant).
#ifndef VQ_ROW_WINDOW
#define VQ_ROW_WINDOW 8
#endif
constexpr int kWindow = VQ_ROW_WINDOW;   // steps per window; a multiple of the index prefetch depth

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void part_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <class P, int NB, bool XS>
__global__ void __launch_bounds__(256, VQ_ROW_MIN_CTAS) rowcb_kernel(const RowArgs a) {
  static_assert(kWindow % VQ_ROW_PREFETCH == 0, "windows hold whole prefetch groups");
  constexpr int PF = VQ_ROW_PREFETCH;
  constexpr int WC = P::WORD_CHUNKS;
  constexpr int CHUNKS = 4 * WC;                 // chunks of a lane per step
  constexpr int LANE_COLS = P::STEP_COLS / 4;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // the tables' address bits 7..11 must be free for the entry index and the row half
  const uint32_t smem_base = (smem_u32(smem_raw) + 4095u) & ~4095u;
  unsigned char* smem = smem_raw + (smem_base - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int S = gridDim.x, rank = blockIdx.x;
  // Receive barrier of the K-part reduction in cluster rank 0: every warp of the cluster sends its
  // 16 rows x batch partial sums there by asynchronous remote stores that count on this barrier.
  // Initialised before the start-up arrive, so that it is visible to every CTA whose start-up wait
  // (in front of the first remote store) has returned.
  const uint32_t red_bar = smem_base + a.bar_offset;
  if (S > 1) {
    if (tid == 0) {
      mbar_init(red_bar, 1);
      mbar_init_fence();
      mbar_arrive_expect_tx(red_bar, static_cast<uint32_t>(S * (blockDim.x / 32) * 16 * a.batch * 4));
    }
    __syncwarp();
    cluster_arrive_release();
  }
  pdl_launch_dependents();

  const int wr = warp % a.WR, wk = warp / a.WR;
  const int T = S * a.WK;
  const int part = rank * a.WK + wk;
  const int cta_s0 = a.n_steps * (rank * a.WK) / T;
  const int cta_s1 = a.n_steps * ((rank + 1) * a.WK) / T;
  const int s0 = a.n_steps * part / T, s1 = a.n_steps * (part + 1) / T;

  const int row0 = (blockIdx.y * a.WR + wr) * 16;
  const int r_lo = row0 + g, r_hi = r_lo + 8;
  const int rl = min(r_lo, a.N - 1), rh = min(r_hi, a.N - 1);   // tail rows load a valid row, store nothing
  const uint8_t* pl = a.idx + rl * a.stride + t * 16 + static_cast<long long>(s0) * 64;
  const uint8_t* ph = a.idx + rh * a.stride + t * 16 + static_cast<long long>(s0) * 64;

  typename P::State st;
  st.init(a, row0, rl, rh, lane, smem_base + warp * P::TABLE_BYTES_PER_WARP);

  // Indices of the first PF steps and the first block's tables: weights do not depend on the
  // previous kernel of the stream, so they are requested before the dependency wait.
  uint4 ql[PF], qh[PF];
#pragma unroll
  for (int u = 0; u < PF; ++u) {
    ql[u] = qh[u] = make_uint4(0, 0, 0, 0);
    if (s0 + u < s1) {
      ql[u] = ldg128_stream(pl + u * 64);
      qh[u] = ldg128_stream(ph + u * 64);
    }
  }
  if (s0 < s1) st.fetch(s0 / a.steps_per_block);

  // ---- activations of the CTA's column range ----
  pdl_wait();   // the activations (and Y) belong to the previous kernel until here
  // XS: window k of this column part = steps s0 + k*kWindow ..; buffer k & 1 of the part's pair
  const uint32_t win_bytes = kWindow * CHUNKS * a.batch * 64;
  const uint32_t part_x = smem_base + a.x_offset + wk * 2 * win_bytes;
  auto issue_window = [&](int k) {
    const int w0 = s0 + k * kWindow;
    const int steps = min(kWindow, s1 - w0);
    if (steps > 0) {
      const int per_row = steps * (P::STEP_COLS / 8);   // 16-byte pieces per batch row
      const int lt = wr * 32 + lane, nthreads = a.WR * 32;
      for (int o = lt; o < per_row * a.batch; o += nthreads) {
        const int m = o / per_row, c8 = o - m * per_row;
        const int col = c8 * 8;
        const int step = col / P::STEP_COLS, within = col % P::STEP_COLS;
        const int tt = within / LANE_COLS, chunk = (within % LANE_COLS) / 8;
        cp_async16(part_x + (k & 1) * win_bytes + (((step * CHUNKS + chunk) * a.batch + m) * 4 + tt) * 16,
                   a.X + static_cast<long long>(m) * a.K + static_cast<long long>(w0) * P::STEP_COLS + col);
      }
    }
    cp_async_commit();
  };
  if constexpr (XS) {
    issue_window(0);
  } else {
    const int col0 = cta_s0 * P::STEP_COLS;
    const int n8 = (cta_s1 - cta_s0) * (P::STEP_COLS / 8);
    uint4* xs = reinterpret_cast<uint4*>(smem + a.x_offset);
    for (int m = 0; m < a.batch; ++m) {
      const uint4* src = reinterpret_cast<const uint4*>(a.X + static_cast<long long>(m) * a.K + col0);
      for (int c8 = tid; c8 < n8; c8 += blockDim.x) {
        const int col = c8 * 8;
        const int step = col / P::STEP_COLS, within = col % P::STEP_COLS;
        const int tt = within / LANE_COLS, chunk = (within % LANE_COLS) / 8;
        xs[((step * CHUNKS + chunk) * a.batch + m) * 4 + tt] = P::permute_x(__ldg(src + c8));
      }
    }
  }
  if (s0 < s1) st.install();   // the first block's entries were requested ahead of the activations
  __syncthreads();
  // every CTA of the cluster started long ago; the wait that proves it (needed before the first
  // remote store) hides here behind the first index loads
  if (S > 1) cluster_wait_acquire();

  float acc[NB][4], total[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[nb][e] = total[nb][e] = 0.f;

  // B fragments: two register sets used alternately; lanes without a batch row keep zeros
  bool on[NB];
  uint32_t xaddr[NB];
  uint4 xb[2][NB][WC];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    on[nb] = nb * 8 + g < a.batch;
    xaddr[nb] = XS ? 0u : smem_base + a.x_offset + (((s0 - cta_s0) * CHUNKS * a.batch + nb * 8 + g) * 4 + t) * 16;
#pragma unroll
    for (int c = 0; c < WC; ++c) xb[0][nb][c] = xb[1][nb][c] = make_uint4(0, 0, 0, 0);
  }
  const uint32_t xstride = a.batch * 64;   // bytes between consecutive chunks

  int in_blk = s0 % a.steps_per_block, blk = s0 / a.steps_per_block;
  for (int sb = s0; sb < s1; sb += PF) {
#pragma unroll
    for (int u = 0; u < PF; ++u) {
      const int s = sb + u;
      if (s >= s1) break;
      if constexpr (XS) {
        if ((s - s0) % kWindow == 0) {
          const int k = (s - s0) / kWindow;
          part_barrier(1 + wk, 32 * a.WR);   // every warp of the part has left window k - 1
          issue_window(k + 1);               // ... whose buffer takes window k + 1
          cp_async_wait<1>();                // this thread's pieces of window k have landed
          part_barrier(1 + wk, 32 * a.WR);   // ... and everybody else's
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) xaddr[nb] = part_x + (k & 1) * win_bytes + ((nb * 8 + g) * 4 + t) * 16;
        }
      }
      const uint4 cl = ql[u], ch = qh[u];
      if (s + PF < s1) {
        ql[u] = ldg128_stream(pl + PF * 64);
        qh[u] = ldg128_stream(ph + PF * 64);
      }
      pl += 64;
      ph += 64;
      // last step of a codebook block: request the next block's entries one step ahead
      if (in_blk + 1 == a.steps_per_block && s + 1 < s1) st.fetch(blk + 1);
      const uint32_t wl[4] = {cl.x, cl.y, cl.z, cl.w}, wh[4] = {ch.x, ch.y, ch.z, ch.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int c = 0; c < WC; ++c) lds128_if(xb[j & 1][nb][c], xaddr[nb] + (j * WC + c) * xstride, on[nb]);
        uint32_t af[WC][2][4];
        st.decode(wl[j], wh[j], af);
#pragma unroll
        for (int c = 0; c < WC; ++c) {
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            const uint4 b = xb[j & 1][nb][c];
            mma16816(acc[nb], af[c][0][0], af[c][0][1], af[c][0][2], af[c][0][3], b.x, b.y);
            mma16816(acc[nb], af[c][1][0], af[c][1][1], af[c][1][2], af[c][1][3], b.z, b.w);
          }
        }
      }
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) xaddr[nb] += CHUNKS * xstride;
      if (++in_blk == a.steps_per_block || s + 1 == s1) {
        // end of a codebook block: apply its scale to the block's partial sums
        if constexpr (P::SCALED) {
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
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
        if (s + 1 < s1) st.install();
      }
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
  // red[K part][tile wr][row 0..15][batch row 0..8*NB-1] in the shared memory of cluster rank 0
  constexpr int NBT = 8 * NB;
  const uint32_t red_local = smem_base + a.red_offset;
  const uint32_t mine = red_local + (((part * a.WR + wr) * 16 + g) * NBT + 2 * t) * 4;
  if (S > 1) {
    const uint32_t dst = map_to_rank(mine, 0), dst_bar = map_to_rank(red_bar, 0);
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (nb * 8 + 2 * t + (e & 1) < a.batch)   // only existing batch rows travel
          st_async_f32(dst + ((e >> 1) * 8 * NBT + nb * 8 + (e & 1)) * 4, total[nb][e], dst_bar);
    // nobody writes into the other ranks' shared memory: they are done; rank 0 waits for the values
    if (rank != 0) return;
    if (!mbar_wait(red_bar, 0, kWaitTries) && tid == 0) atomicAdd(a.error_flag, 1);
  } else {
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (nb * 8 + 2 * t + (e & 1) < a.batch) sts32f(mine + ((e >> 1) * 8 * NBT + nb * 8 + (e & 1)) * 4, total[nb][e]);
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
    for (int p = 0; p < T; ++p) sum += red[(p * cta_rows + rr) * NBT + n];
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

// Choose the CTA shape (WR row tiles x WK column parts, at most 8 warps) and the cluster size S.
// Model fitted to sweeps on B200: time ~ waves x (steps per warp + a fixed per-CTA overhead of
// about 3 steps, 4 with a cluster, + the CTA's activation staging), where a wave is as many CTAs as are co-resident (registers
// allow about 16 warps per SM, 8 for the two-tile batch variant).  One wave of 8-warp CTAs with
// as many column parts per CTA as possible wins; ties go to more column parts, then fewer CTAs
// per cluster.  Shapes whose tables, activations and reduction buffer exceed smem_budget bytes of
// shared memory are left out; {0,0,0} if none fits.
Plan make_plan(int N, int n_steps, int step_cols, int batch, int sms, int tbl_per_warp, int nb, size_t smem_budget,
               bool streamed) {
  const int row_tiles = (N + 15) / 16;
  const int warps_per_sm = nb == 1 ? 16 : 8;
  Plan best = {0, 0, 0};
  double best_cost = -1.0;
  for (int S = 1; S <= 8; S *= 2)
    for (int WK = 8; WK >= 1; WK /= 2)
      for (int WR = 1; WR * WK <= 8; WR *= 2) {
        const int T = S * WK;
        if (T > n_steps || (T > 1 && 2 * T > n_steps)) continue;   // at least two steps per warp
        const int W = WR * WK;
        const double cta_steps = static_cast<double>(n_steps) / S;
        const double x_need = streamed ? 2.0 * kWindow * WK * step_cols * 2.0 * batch : (cta_steps + 1.0) * step_cols * 2.0 * batch;
        const double smem_need = x_need + static_cast<double>(tbl_per_warp) * W +
                                 (T > 1 ? T * WR * 16.0 * 8.0 * nb * 4.0 : 0.0) + 4096.0 + 16.0;
        if (smem_need > static_cast<double>(smem_budget)) continue;
        int per_sm = warps_per_sm / W;
        const int by_smem = static_cast<int>(227.0 * 1024.0 / (smem_need + 1024.0));
        if (per_sm > by_smem) per_sm = by_smem;
        if (per_sm < 1) per_sm = 1;
        const long long ctas = static_cast<long long>((row_tiles + WR - 1) / WR) * S;
        const long long slots = static_cast<long long>(per_sm) * sms;
        // more CTAs than fit at once: between the work-conserving ratio and whole waves
        const double ratio = static_cast<double>(ctas) / static_cast<double>(slots);
        const double whole = static_cast<double>((ctas + slots - 1) / slots);
        // (measured at batch 1 and 2; with more batch rows the staging of a late CTA is not hidden)
        const double waves = batch <= 2 ? 0.5 * (ratio < 1.0 ? 2.0 : ratio + whole) : whole;
        const double steps = static_cast<double>(n_steps) / T;
        // every CTA stages the activations of its whole column range: about a tenth of a step of
        // work per staged step, shared by its warps
        const double stage = batch <= 2 ? 0.1 * cta_steps / W : 0.0;
        // few resident warps hide latency badly
        const double resident = static_cast<double>(ctas < slots ? ctas : slots) * W / sms;
        const double slow = resident >= 8.0 ? 1.0 : 8.0 / (resident < 1.0 ? 1.0 : resident);
        const double cost = waves * (steps * slow + (S > 1 ? 4.0 : 3.0) + stage);
        if (best_cost < 0.0 || cost < best_cost) {
          best_cost = cost;
          best = {WR, WK, S};
        }
      }
  best.WR = env_int("VQ_WR", best.WR);
  best.WK = env_int("VQ_WK", best.WK);
  best.S = env_int("VQ_S", best.S);
  return best;
}

template <class P, int NB, bool XS = false>
vq_status launch(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, cudaStream_t s) {
  if (g.K % P::STEP_COLS || g.Bc % P::STEP_COLS) return VQ_ERR_UNSUPPORTED;
  // per device, once: SM count and the opt-in to large dynamic shared memory
  static int attr_set[kMaxDevices] = {};
  auto kern = rowcb_kernel<P, NB, XS>;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (!__atomic_load_n(&attr_set[dev], __ATOMIC_ACQUIRE)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024) != cudaSuccess) return VQ_ERR_CUDA;
    __atomic_store_n(&attr_set[dev], 1, __ATOMIC_RELEASE);
  }
  RowArgs a;
  a.idx = p.idx;
  a.cb = static_cast<const uint8_t*>(p.cb);
  a.scale = p.scale;
  a.X = X;
  a.Y = Y;
  if (device_error_counter(&a.error_flag) != VQ_OK) return VQ_ERR_CUDA;
  a.stride = g.stride;
  a.N = g.N;
  a.K = g.K;
  a.batch = batch;
  a.n_steps = g.K / P::STEP_COLS;
  a.steps_per_block = g.Bc / P::STEP_COLS;
  a.blocks_per_row = g.blocks_per_row;
  a.Br = g.Br;
  constexpr size_t kSmemBudget = 200 * 1024;
  const Plan pl = make_plan(g.N, a.n_steps, P::STEP_COLS, batch, sms, P::TABLE_BYTES_PER_WARP, NB, kSmemBudget, XS);
  const int T = pl.S * pl.WK;
  if (pl.WR < 1 || pl.WK < 1 || pl.WR * pl.WK > 8 || pl.S < 1 || pl.S > 8 || T > a.n_steps) return VQ_ERR_UNSUPPORTED;
  a.WR = pl.WR;
  a.WK = pl.WK;
  int cta_steps = 0;   // longest column range of a CTA of the cluster
  for (int r = 0; r < pl.S; ++r) {
    const int c = a.n_steps * ((r + 1) * pl.WK) / T - a.n_steps * (r * pl.WK) / T;
    if (c > cta_steps) cta_steps = c;
  }
  const size_t tbl_bytes = static_cast<size_t>(P::TABLE_BYTES_PER_WARP) * pl.WR * pl.WK;
  const size_t x_bytes = XS ? static_cast<size_t>(2 * kWindow) * pl.WK * P::STEP_COLS * 2 * batch
                            : static_cast<size_t>(cta_steps) * P::STEP_COLS * 2 * batch;
  const size_t red_bytes = T > 1 ? static_cast<size_t>(T) * pl.WR * 16 * 8 * NB * sizeof(float) : 0;
  if (tbl_bytes + x_bytes + 16 + red_bytes + 16 + 4096 > 208 * 1024) return VQ_ERR_UNSUPPORTED;
  a.x_offset = static_cast<int>(tbl_bytes);
  a.red_offset = static_cast<int>(tbl_bytes + (x_bytes + 15) / 16 * 16);
  a.bar_offset = a.red_offset + static_cast<int>(red_bytes);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.S, (g.N + 16 * pl.WR - 1) / (16 * pl.WR), 1);
  cfg.blockDim = dim3(32 * pl.WR * pl.WK, 1, 1);
  cfg.dynamicSmemBytes = a.red_offset + red_bytes + 16 + 4096;   // + barrier, + room to align the tables
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
#ifdef VQ_TUNING
  {
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, a);
    if (e != cudaSuccess) {
      fprintf(stderr, "rowcb launch failed: %s (grid %d,%d block %d smem %zu S %d WR %d WK %d)\n", cudaGetErrorString(e),
              cfg.gridDim.x, cfg.gridDim.y, cfg.blockDim.x, cfg.dynamicSmemBytes, pl.S, pl.WR, pl.WK);
      return VQ_ERR_CUDA;
    }
    return check_launch();
  }
#endif
  if (cudaLaunchKernelEx(&cfg, kern, a) != cudaSuccess) return VQ_ERR_CUDA;
  return check_launch();
}

}  // namespace

// 4-bit families whose codebooks are looked up per row: block_rows == 1, or a few rows that share
// a block (every lane then simply takes the entries of its own rows' block).
vq_status launch_gemm_rowcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                            cudaStream_t s) {
  if (g.b != 4) return VQ_ERR_UNSUPPORTED;
  // batch 1-8: activations staged once for the CTA's column range; batch 9-16 (two batch tiles):
  // streamed in windows (measured: 316 against 465 us on the 70B-shaped set at batch 16, but
  // 197 against 165 us at batch 4 and 232 against 212 us at batch 8, where staging still fits)
  auto pick = [&](auto policy) {
    using P = decltype(policy);
    return batch <= 8 ? launch<P, 1, false>(g, p, X, Y, batch, s) : launch<P, 2, true>(g, p, X, Y, batch, s);
  };
  if (g.cb_int8 && g.d == 1) return pick(PrmtI8{});
  if (g.cb_int8 && g.d == 2) return pick(LdsTbl<true>{});
  if (!g.cb_int8 && g.d == 2) return pick(LdsTbl<false>{});
  return VQ_ERR_UNSUPPORTED;
}

// Uniform INT4 group-128 yard-stick through the row-kernel skeleton; UNSUPPORTED if K is not a
// multiple of 128.
vq_status launch_int4g128_rowcb(int N, int K, const uint8_t* q, const __half* scale, const __half* X, __half* Y, int batch,
                                cudaStream_t s) {
  if (K % 128) return VQ_ERR_UNSUPPORTED;
  Geometry g = {};
  g.N = N; g.K = K; g.d = 1; g.b = 4; g.Br = 1; g.Bc = 128;
  g.cb_int8 = 1; g.cb_int4 = 0; g.entries = 16; g.J = K; g.blocks_per_row = K / 128; g.stride = K / 2;
  LayerPtrs p;
  p.idx = q;
  p.cb = nullptr;
  p.scale = scale;
  return batch <= 8 ? launch<Int4G128, 1>(g, p, X, Y, batch, s) : launch<Int4G128, 2>(g, p, X, Y, batch, s);
}

}  // namespace vq
