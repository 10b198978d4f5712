// Tuned skinny-GEMM kernels for formats whose codebook is shared by a tall block of rows
// (block_rows a multiple of the CTA's rows): the 2-D 5- and 6-bit and the 4-D 8-bit families, with
// fp16 codebooks or int8 codebooks (whose entries enter the tables as fp16(scale * c)).
//
// A CTA owns one block-row slab (128 or 256 rows: every warp 32 of them) and a range of 256-column
// chunks; a thread block cluster of S CTAs splits K.  Per chunk and warp the packed indices of 32
// rows arrive as ONE tiled TMA box (32 rows x 96 or 64 bytes) in a warp-private ring of shared
// memory, a few chunks ahead, completion counted on an mbarrier; lane (g = lane/4, t = lane%4)
// reads its own 64 columns of rows g, g+8, g+16, g+24 from the box (conflict-free), looks every
// index up in a lane-private copy of the chunk's codebook ([entry][lane] words: bank = lane, so
// the gather is conflict-free for any index pattern; index bits and lane bits of the address are
// merged by one logic operation) and feeds the fp16 pairs, untouched, into mma.sync m16n8k16 as
// the A fragment.  The activations of the CTA's column range are staged once in shared memory in
// the order the lanes consume them (B fragment, batch row = g); accumulation is fp32.  Codebook
// tables are double buffered for 2-D formats (the next one is replicated while the current chunk
// is computed, its entries fetched from global memory two tables ahead); the 32 KB tables of the
// 4-D format use one buffer rewritten between two block-wide barriers, and blocks of 32 or 64 rows
// one table per warp.  Partial sums of the K parts travel as asynchronous remote stores, counted
// on an mbarrier, to the cluster rank that owns the rows, are added in rank order, rounded once to
// fp16 and stored.
// Paper: Sec. 3.2 (packed indices -> LUT -> mat-vec), App. A (Q is a look-up of C); the tiling,
// the replication and the reduction are this library's.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <utility>

#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

using namespace dev;

#ifndef VQ_BLOCK_STAGES
#define VQ_BLOCK_STAGES 3   // chunks of the index stream a warp keeps in flight
#endif
constexpr int kStages = VQ_BLOCK_STAGES;
// Warp-private tables take 32 KB of a CTA's shared memory: two ring stages keep three CTAs on an SM.
#ifndef VQ_BLOCK_STAGES_D4
#define VQ_BLOCK_STAGES_D4 2
#endif
#ifndef VQ_BLOCK_TB_D4
#define VQ_BLOCK_TB_D4 1
#endif
template <int D, bool PRIV>
constexpr int kStagesOf = PRIV ? 2 : (D == 4 ? VQ_BLOCK_STAGES_D4 : kStages);
// Table buffers of the shared-table mode: 2 = the next table is replicated during the current one's
// math; 1 = it replaces the current one between two block-wide barriers (saves TABLE_BYTES).
template <int D>
constexpr int kTableBuffers = D == 4 ? VQ_BLOCK_TB_D4 : 2;
constexpr int kWaitTries = 1 << 18;   // mbarrier polls before a warp gives up and flags an error

struct BlockArgs {
  const void* cb;
  const __half* scale;   // one per block for int8 codebooks, else null
  const __half* gscale;  // int4 codebooks (Sec. 4.2): one per row and group of 128 columns, [N][K/128]; else null
  const __half* X;
  __half* Y;
  int* error_flag;       // device counter of waits that ran out
  int N, K, batch;
  int n_chunks;          // K / 256
  int blocks_per_row;    // K / block_cols
  int Br, Bc;
  // byte offsets from the tables' boundary (the first TABLE_BYTES boundary that leaves front_bytes of
  // dynamic shared memory in front of it): parts that fit lie in front of the tables (negative
  // offsets), in bytes that alignment would otherwise waste; the rest follows the tables
  int compact_off, ring_off, bar_off, x_off, recv_off;
  int front_bytes, after_bytes;
};

// Layers of one call (same format and K, their own rows): row tiles [tile0, next tile0) of the grid
// belong to layer i.
struct BlockGroup {
  const void* cb[kMaxSegments];
  const __half* scale[kMaxSegments];
  __half* Y[kMaxSegments];
  int N[kMaxSegments];
  int tile0[kMaxSegments];
  int n_seg;
};
struct BlockMaps {
  CUtensorMap m[kMaxSegments];   // the layers' index streams
};

// ---- format policies -----------------------------------------------------------------------
template <int D, int B>
struct Policy;

// 2-D, B-bit indices (B = 5, 6): 256 columns = 128 indices = 16*B bytes per row; a lane owns 32
// indices = B words of them
template <int B>
struct PolicyD2 {
  static constexpr int LANE_WORDS = B, ENTRIES = 1 << B, SEG = 16 * B;
  static constexpr int WARPS = 4;                           // CTA = 128 rows
  static constexpr int TABLE_BYTES = ENTRIES * 128;          // [entry][lane] words
  static constexpr int COMPACT_BYTES = ENTRIES * 8;          // [entry][half] words
  static constexpr uint32_t MASK = static_cast<uint32_t>(ENTRIES - 1) << 7;   // index bits at address bits 7..

  template <int I>   // (index I of the lane's 32) * 128
  static __device__ __forceinline__ uint32_t entry_off(const uint32_t (&w)[LANE_WORDS]) {
    constexpr int p = B * I;
    if constexpr (p < 7) {
      return (w[0] << (7 - p)) & MASK;
    } else {
      constexpr int q = p - 7, wi = q >> 5, s = q & 31;
      if constexpr (s == 0) return w[wi] & MASK;
      else if constexpr (s + 7 + B > 32) return __funnelshift_r(w[wi], w[wi + 1], s) & MASK;
      else return (w[wi] >> s) & MASK;
    }
  }
};
template <>
struct Policy<2, 6> : PolicyD2<6> {};
template <>
struct Policy<2, 5> : PolicyD2<5> {};

// 4-D, 8-bit indices: 256 columns = 64 indices = 64 bytes per row; a lane owns 16 of them
template <>
struct Policy<4, 8> {
  static constexpr int LANE_WORDS = 4, ENTRIES = 256, SEG = 64;
  static constexpr int WARPS = 8;                           // CTA = 256 rows
  static constexpr int TABLE_BYTES = ENTRIES * 128;          // [entry][lane%16] 8-byte entries
  static constexpr int COMPACT_BYTES = ENTRIES * 8;
  static constexpr uint32_t MASK = 0x7F80u;

  template <int I>
  static __device__ __forceinline__ uint32_t entry_off(const uint32_t (&w)[LANE_WORDS]) {
    constexpr int wi = I >> 2, p = 8 * (I & 3);
    if constexpr (p < 7) return (w[wi] << (7 - p)) & MASK;
    else return (w[wi] >> (p - 7)) & MASK;
  }
};

template <int D, int B>
struct Tile {
  using P = Policy<D, B>;
  static constexpr int CTA_ROWS = 32 * P::WARPS;
  static constexpr int THREADS = 32 * P::WARPS;
  static constexpr int STAGE_BYTES = 32 * P::SEG;            // one TMA box
};

__device__ __forceinline__ uint32_t lds32_ordered(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ uint2 lds64_ordered(uint32_t addr) {   // ring reads: stay behind the barrier wait
  uint2 v;
  asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
  return v;
}

// A fragments of NSTEPS mma steps (each step = 4 columns per lane) of one 16-row tile; wa / wb are
// the lane's index words of rows g and g+8 of the tile, tbl the lane's table address.
template <int D, int B, int STEP0, int NSTEPS>
__device__ __forceinline__ void gather_steps(uint32_t (&a)[NSTEPS][4], const uint32_t (&wa)[Policy<D, B>::LANE_WORDS],
                                             const uint32_t (&wb)[Policy<D, B>::LANE_WORDS], uint32_t tbl) {
  using P = Policy<D, B>;
  if constexpr (D == 2) {
    [&]<int... S>(std::integer_sequence<int, S...>) {
      ((a[S][0] = lds32(P::template entry_off<2 * (STEP0 + S)>(wa) | tbl),
        a[S][1] = lds32(P::template entry_off<2 * (STEP0 + S)>(wb) | tbl),
        a[S][2] = lds32(P::template entry_off<2 * (STEP0 + S) + 1>(wa) | tbl),
        a[S][3] = lds32(P::template entry_off<2 * (STEP0 + S) + 1>(wb) | tbl)), ...);
    }(std::make_integer_sequence<int, NSTEPS>{});
  } else {
    [&]<int... S>(std::integer_sequence<int, S...>) {
      (([&] {
         const uint2 u = lds64(P::template entry_off<STEP0 + S>(wa) | tbl);
         const uint2 v = lds64(P::template entry_off<STEP0 + S>(wb) | tbl);
         a[S][0] = u.x; a[S][2] = u.y; a[S][1] = v.x; a[S][3] = v.y;
       }()), ...);
    }(std::make_integer_sequence<int, NSTEPS>{});
  }
}

// Both 16-row tiles of a warp for NSTEPS steps: their accumulator chains are independent, so the
// look-ups are issued together and the mmas alternate.
// I4 (int4 codebooks): the table holds the signed 4-bit entries as fp16; sc[q] is the fp16 scale (twice)
// of row 8q + g of the warp's rows for the lane's group of 128 columns, and every looked-up pair is
// multiplied by it: fp16(scale * c), the value vq_decode_weights writes (one rounding of an exact product).
__device__ __forceinline__ uint32_t mul_f16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
template <int D, int B, int NB, int STEP0, int NSTEPS, bool I4 = false>
__device__ __forceinline__ void chunk_steps(float (&acc)[2][NB][4], const uint32_t (&w)[4][Policy<D, B>::LANE_WORDS],
                                            const uint32_t (&xr)[NB][32], uint32_t tbl, const uint32_t (&sc)[4]) {
  uint32_t a0[NSTEPS][4], a1[NSTEPS][4];
  gather_steps<D, B, STEP0, NSTEPS>(a0, w[0], w[1], tbl);
  gather_steps<D, B, STEP0, NSTEPS>(a1, w[2], w[3], tbl);
  if constexpr (I4) {
#pragma unroll
    for (int s = 0; s < NSTEPS; ++s) {
      a0[s][0] = mul_f16x2(a0[s][0], sc[0]); a0[s][1] = mul_f16x2(a0[s][1], sc[1]);
      a0[s][2] = mul_f16x2(a0[s][2], sc[0]); a0[s][3] = mul_f16x2(a0[s][3], sc[1]);
      a1[s][0] = mul_f16x2(a1[s][0], sc[2]); a1[s][1] = mul_f16x2(a1[s][1], sc[3]);
      a1[s][2] = mul_f16x2(a1[s][2], sc[2]); a1[s][3] = mul_f16x2(a1[s][3], sc[3]);
    }
  }
#pragma unroll
  for (int s = 0; s < NSTEPS; ++s)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      mma16816(acc[0][nb], a0[s][0], a0[s][1], a0[s][2], a0[s][3], xr[nb][2 * (STEP0 + s)], xr[nb][2 * (STEP0 + s) + 1]);
      mma16816(acc[1][nb], a1[s][0], a1[s][1], a1[s][2], a1[s][3], xr[nb][2 * (STEP0 + s)], xr[nb][2 * (STEP0 + s) + 1]);
    }
}

// Compiler-level ordering point: everything that produced the accumulators (the mmas, hence the
// gathers that feed them) is emitted before whatever follows.
template <int NB>
__device__ __forceinline__ void fence_acc(float (&acc)[2][NB][4]) {
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) asm volatile("" : "+f"(acc[mt][nb][e])::"memory");
}

// Fetch this thread's share of the codebook entries of table k (global memory -> register).
// 2-D: thread (e = tid%64, h = tid/64) takes entry e of the block under columns h*128.. of the
// chunk; 4-D: thread tid takes entry tid of the block the table's chunks lie in.
template <int D, int B>
__device__ __forceinline__ uint2 fetch_entry(const BlockArgs& a, long long blk_row, int chunk, int tid) {
  using P = Policy<D, B>;
  uint2 v = make_uint2(0u, 0u);
  // int8 codebooks: the table holds fp16(scale * c), the value vq_decode_weights writes for the weight
  auto pair = [](float s, int lo, int hi) {
    const __half2 hv = __halves2half2(__float2half_rn(s * static_cast<float>(lo)), __float2half_rn(s * static_cast<float>(hi)));
    return *reinterpret_cast<const uint32_t*>(&hv);
  };
  if constexpr (D == 2) {
    const int e = tid % P::ENTRIES, h = tid / P::ENTRIES;
    if (h >= 2) return v;
    const long long blk = blk_row + (chunk * 256 + h * 128) / a.Bc;
    if (a.gscale != nullptr) {   // int4 entries: one byte per 2-D entry, low nibble = first value; exact in fp16
      const uint32_t byte = __ldg(static_cast<const uint8_t*>(a.cb) + blk * P::ENTRIES + e);
      v.x = pair(1.f, (static_cast<int>(byte & 15u) ^ 8) - 8, (static_cast<int>(byte >> 4) ^ 8) - 8);
    } else if (a.scale == nullptr) {
      v.x = __ldg(static_cast<const uint32_t*>(a.cb) + blk * P::ENTRIES + e);
    } else {
      const uint16_t raw = __ldg(static_cast<const uint16_t*>(a.cb) + blk * P::ENTRIES + e);
      v.x = pair(__half2float(__ldg(a.scale + blk)), static_cast<int8_t>(raw & 0xff), static_cast<int8_t>(raw >> 8));
    }
  } else {
    const long long blk = blk_row + (chunk * 256) / a.Bc;
    if (a.scale == nullptr) {
      v = __ldg(static_cast<const uint2*>(a.cb) + blk * P::ENTRIES + tid);
    } else {
      const uint32_t raw = __ldg(static_cast<const uint32_t*>(a.cb) + blk * P::ENTRIES + tid);
      const float s = __half2float(__ldg(a.scale + blk));
      v.x = pair(s, static_cast<int8_t>(raw & 0xff), static_cast<int8_t>((raw >> 8) & 0xff));
      v.y = pair(s, static_cast<int8_t>((raw >> 16) & 0xff), static_cast<int8_t>(raw >> 24));
    }
  }
  return v;
}

template <int D, int B>
__device__ __forceinline__ void store_compact(unsigned char* compact, uint2 v, int tid) {
  if constexpr (D == 2) {
    constexpr int E = Policy<D, B>::ENTRIES;
    if (tid / E < 2) reinterpret_cast<uint32_t*>(compact)[2 * (tid % E) + tid / E] = v.x;   // [entry][half]
  }
  else reinterpret_cast<uint2*>(compact)[tid] = v;
}

// Replicate a compact codebook into the lane-private layout with 128-bit stores (the 8 lanes of a
// quarter warp write 8 different 16-byte bank groups).
template <int D, int B>
__device__ __forceinline__ void replicate(uint32_t table, const unsigned char* compact, int tid) {
  using P = Policy<D, B>;
  constexpr int THREADS = Tile<D, B>::THREADS;
#pragma unroll
  for (int j = 0; j < P::ENTRIES * 8 / THREADS; ++j) {
    const int item = tid + j * THREADS;   // (entry, 16-byte group)
    const int e = item >> 3, u = item & 7;
    const uint2 c = reinterpret_cast<const uint2*>(compact)[e];
    // 2-D: lanes 4u..4u+3 = columns 0-127 (two lanes, half 0) and 128-255 (half 1) of the chunk
    const uint4 v = D == 2 ? make_uint4(c.x, c.x, c.y, c.y) : make_uint4(c.x, c.y, c.x, c.y);
    sts128(table + e * 128 + u * 16, v);
  }
}

// ---- warp-private tables (2-D formats whose block is 32 or 64 rows tall: every warp's 32 rows have
// their own codebooks).  Lane l takes entries l*EPL .. +EPL-1 (EPL = ENTRIES / 32) of the two blocks
// under the chunk's column halves: requested by load_private(), converted and written by
// write_private() with the same rotation of the 16-byte groups as replicate().
template <int B>
struct PrivateRegs {
  static constexpr int EPL = (1 << B) / 32;
  uint32_t raw[2][EPL];   // fp16 codebooks: the entries; int8: EPL entries of 2 bytes in raw[h][0]
  float scale[2];
};
template <int B>
__device__ __forceinline__ void load_private(PrivateRegs<B>& r, const BlockArgs& a, long long blk_row, int chunk, int lane) {
  constexpr int E = 1 << B, EPL = PrivateRegs<B>::EPL;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const long long blk = blk_row + (chunk * 256 + h * 128) / a.Bc;
    if (a.gscale != nullptr) {   // int4 entries: EPL bytes
      const uint8_t* src = static_cast<const uint8_t*>(a.cb) + blk * E + lane * EPL;
      if constexpr (EPL == 2) r.raw[h][0] = __ldg(reinterpret_cast<const uint16_t*>(src));
      else r.raw[h][0] = __ldg(src);
      r.scale[h] = 1.f;
    } else if (a.scale == nullptr) {
      const uint32_t* src = static_cast<const uint32_t*>(a.cb) + blk * E + lane * EPL;
      if constexpr (EPL == 2) {
        const uint2 q = ldg64_nc(src);
        r.raw[h][0] = q.x;
        r.raw[h][1] = q.y;
      } else {
        r.raw[h][0] = __ldg(src);
      }
      r.scale[h] = 1.f;
    } else {
      const uint16_t* src = static_cast<const uint16_t*>(a.cb) + blk * E + lane * EPL;
      if constexpr (EPL == 2) r.raw[h][0] = __ldg(reinterpret_cast<const uint32_t*>(src));
      else r.raw[h][0] = __ldg(src);
      r.scale[h] = __half2float(__ldg(a.scale + blk));
    }
  }
}
template <int B>
__device__ __forceinline__ void write_private(uint32_t table, const PrivateRegs<B>& r, int mode, int lane) {   // mode 0 fp16, 1 int8, 2 int4
  constexpr int EPL = PrivateRegs<B>::EPL;
#pragma unroll
  for (int i = 0; i < EPL; ++i) {
    uint32_t e[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (mode == 0) {
        e[h] = r.raw[h][i];
      } else if (mode == 2) {
        const uint32_t byte = (r.raw[h][0] >> (8 * i)) & 0xffu;
        const __half2 hv = __halves2half2(__int2half_rn((static_cast<int>(byte & 15u) ^ 8) - 8), __int2half_rn((static_cast<int>(byte >> 4) ^ 8) - 8));
        e[h] = *reinterpret_cast<const uint32_t*>(&hv);
      } else {
        const uint32_t two = r.raw[h][0] >> (16 * i);
        const __half2 hv = __halves2half2(__float2half_rn(r.scale[h] * static_cast<float>(static_cast<int8_t>(two & 0xff))),
                                          __float2half_rn(r.scale[h] * static_cast<float>(static_cast<int8_t>((two >> 8) & 0xff))));
        e[h] = *reinterpret_cast<const uint32_t*>(&hv);
      }
    }
    const uint4 v = make_uint4(e[0], e[0], e[1], e[1]);
    const uint32_t row = table + (lane * EPL + i) * 128;
#pragma unroll
    for (int j = 0; j < 8; ++j) sts128(row + ((j + lane) & 7) * 16, v);
  }
}

// Grid (S, N / CTA_ROWS), cluster (S, 1, 1).  Dynamic shared memory from its first TABLE_BYTES
// boundary: two tables, two compact codebooks, the warps' index rings, their barriers, the
// activations, the receive buffer of the reduction.
// PRIV: every warp keeps its own pair of tables (block rows a multiple of 32, 2-D only).
// I4: int4 codebooks with a scale per row and group of 128 columns (2-D only; a lane's 64 columns of a
// chunk lie inside one group).
template <int D, int B, int NB, bool PRIV, bool I4>
__global__ void __launch_bounds__(Tile<D, B>::THREADS)
blockcb_kernel(const __grid_constant__ BlockMaps maps, const BlockArgs a_in, const BlockGroup grp) {
  static_assert(!PRIV || D == 2, "warp-private tables exist for 2-D codebooks only");
  static_assert(!I4 || D == 2, "int4 codebooks are served for 2-D formats only");
  constexpr int ST = kStagesOf<D, PRIV>;   // ring stages per warp
  using P = Policy<D, B>;
  using T = Tile<D, B>;
  constexpr int LW = P::LANE_WORDS;
  constexpr int NBT = 8 * NB;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const uint32_t raw_u32 = smem_u32(smem_raw);
  const uint32_t base = (raw_u32 + a_in.front_bytes + P::TABLE_BYTES - 1) & ~static_cast<uint32_t>(P::TABLE_BYTES - 1);
  unsigned char* smem = smem_raw + (base - raw_u32);
  {   // the host sized the launch for dynamic shared memory that starts 1024 bytes into the CTA's window
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (base - raw_u32 + static_cast<uint32_t>(a_in.after_bytes) > dyn) {   // (the same for every thread of the cluster)
      if (threadIdx.x == 0) atomicAdd(a_in.error_flag, 1);
      return;
    }
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int S = gridDim.x, rank = blockIdx.x;
  // the layer of this row tile
  int sgi = 0;
#pragma unroll
  for (int i = 1; i < kMaxSegments; ++i)
    if (i < grp.n_seg && static_cast<int>(blockIdx.y) >= grp.tile0[i]) sgi = i;
  BlockArgs a = a_in;
  a.cb = grp.cb[sgi];
  a.scale = I4 ? nullptr : grp.scale[sgi];
  a.gscale = I4 ? grp.scale[sgi] : nullptr;
  a.Y = grp.Y[sgi];
  a.N = grp.N[sgi];
  const CUtensorMap* tm = &maps.m[sgi];
  // Receive barrier of the K-part reduction: S * rpo * batch values of 4 bytes arrive through
  // asynchronous remote stores.  Initialised before the start-up arrive so that every CTA of the
  // cluster sees it once its start-up wait (in front of the first remote store) returns.
  const uint32_t recv_bar = base + a.bar_off + P::WARPS * ST * 8;
  if (S > 1) {
    if (tid == 0) {
      mbar_init(recv_bar, 1);
      mbar_init_fence();
      mbar_arrive_expect_tx(recv_bar, static_cast<uint32_t>(T::CTA_ROWS * a.batch * 4));
    }
    __syncwarp();
    cluster_arrive_release();
  }
  pdl_launch_dependents();

  const int c0 = a.n_chunks * rank / S, c1 = a.n_chunks * (rank + 1) / S, n = c1 - c0;
  const int row0 = (static_cast<int>(blockIdx.y) - grp.tile0[sgi]) * T::CTA_ROWS;
  // first block of the block row the CTA's (PRIV: the warp's) rows lie in
  const long long blk_row = static_cast<long long>((row0 + (PRIV ? 32 * warp : 0)) / a.Br) * a.blocks_per_row;
  const int cpt = D == 2 ? 1 : a.Bc / 256;   // chunks that share one table
  const int t0 = c0 / cpt, nt = n > 0 ? (c1 - 1) / cpt - t0 + 1 : 0;

  // ---- index ring: warp-private stages, one TMA box each ----
  const uint32_t bars = base + a.bar_off + warp * ST * 8;
  const uint32_t ring = base + a.ring_off + warp * ST * T::STAGE_BYTES;
  if (lane == 0) {
    for (int s = 0; s < ST; ++s) mbar_init(bars + 8 * s, 1);
    mbar_init_fence();
  }
  __syncwarp();
  auto issue = [&](int i) {   // lane 0 only
    const int st = i % ST;
    mbar_arrive_expect_tx(bars + 8 * st, T::STAGE_BYTES);
    tma_box_2d(ring + st * T::STAGE_BYTES, tm, (c0 + i) * P::SEG, row0 + 32 * warp, bars + 8 * st);
  };
  if (lane == 0)
    for (int i = 0; i < ST && i < n; ++i) issue(i);

  // ---- first two codebook tables and the activations: all global loads are requested before any
  // of them is waited for ----
  unsigned char* compact = smem + a.compact_off;
  uint2 cb0 = make_uint2(0u, 0u), cb1 = cb0;
  PrivateRegs<PRIV ? B : 5> mine;   // PRIV: this warp's entries of the table that is written next
  const uint32_t my_tables = base + (PRIV ? warp * P::TABLE_BYTES : 0);   // PRIV: one table per warp
  if constexpr (PRIV) {
    if (n > 0) load_private<B>(mine, a, blk_row, c0, lane);
  } else {
    if (nt > 0) cb0 = fetch_entry<D, B>(a, blk_row, t0 * cpt, tid);
    if (nt > 1) cb1 = fetch_entry<D, B>(a, blk_row, (t0 + 1) * cpt, tid);
  }

  // Activations of the CTA's column range: chunk i, 16-byte piece j of a lane's 64 columns, batch
  // row m, lane quarter tt at ((i*8 + j)*batch + m)*4 + tt.
  pdl_wait();   // the activations (and Y) belong to the previous kernel until here
  {
    uint4* xs = reinterpret_cast<uint4*>(smem + a.x_off);
    const int n16 = n * 32;   // 16-byte pieces per batch row
    const int total = n16 * a.batch;
    constexpr int kInReg = 4;   // pieces a thread keeps in registers: enough for the usual ranges
    uint4 xv[kInReg];
#pragma unroll
    for (int u = 0; u < kInReg; ++u) {
      const int item = tid + u * T::THREADS;
      xv[u] = make_uint4(0u, 0u, 0u, 0u);
      if (item < total) {
        const int m = item / n16, q = item - m * n16;
        xv[u] = __ldg(reinterpret_cast<const uint4*>(a.X + static_cast<long long>(m) * a.K + c0 * 256) + q);
      }
    }
    if constexpr (PRIV) {
      if (n > 0) write_private<B>(my_tables, mine, I4 ? 2 : a.scale != nullptr ? 1 : 0, lane);
      if (n > 1) load_private<B>(mine, a, blk_row, c0 + 1, lane);
    } else {
      if (nt > 0) store_compact<D, B>(compact, cb0, tid);
      if (nt > 1) store_compact<D, B>(compact + P::COMPACT_BYTES, cb1, tid);
    }
    auto put = [&](int item, uint4 v) {
      const int m = item / n16, q = item - m * n16;
      const int i = q >> 5, tt = (q >> 3) & 3, j = q & 7;
      xs[((i * 8 + j) * a.batch + m) * 4 + tt] = v;
    };
#pragma unroll
    for (int u = 0; u < kInReg; ++u) {
      const int item = tid + u * T::THREADS;
      if (item < total) put(item, xv[u]);
    }
    for (int item = tid + kInReg * T::THREADS; item < total; item += T::THREADS) {
      const int m = item / n16, q = item - m * n16;
      put(item, __ldg(reinterpret_cast<const uint4*>(a.X + static_cast<long long>(m) * a.K + c0 * 256) + q));
    }
  }
  __syncthreads();
  if constexpr (!PRIV)
    if (nt > 0) replicate<D, B>(base, compact, tid);
  // every CTA of the cluster has started long ago; the wait that proves it (needed before the first
  // remote store) costs a few hundred ns and hides here behind the first index box
  if (S > 1) cluster_wait_acquire();
  __syncthreads();

  float acc[2][NB][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nb][e] = 0.f;
  uint32_t xr[NB][32];
  bool on[NB];
  uint32_t xaddr[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    on[nb] = nb * 8 + g < a.batch;
    xaddr[nb] = base + a.x_off + ((nb * 8 + g) * 4 + t) * 16;
#pragma unroll
    for (int i = 0; i < 32; ++i) xr[nb][i] = 0u;
  }
  const uint32_t xstride = a.batch * 64;
  const uint32_t lane_off = D == 2 ? lane * 4 : (lane & 15) * 8;
  const uint32_t row_off = t * (LW * 4) + g * P::SEG;
  // int4 codebooks: the scales of the lane's four rows (8q + g of the warp's 32) for its group of 128
  // columns (lanes t < 2: the chunk's first group, t >= 2: the second), requested one chunk ahead
  uint32_t sc[4] = {0u, 0u, 0u, 0u}, sc_next[4] = {0u, 0u, 0u, 0u};
  auto load_scales = [&](int chunk, uint32_t (&o)[4]) {
    const unsigned short* base_sc = reinterpret_cast<const unsigned short*>(a.gscale) + chunk * 2 + (t >> 1);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      o[q] = __ldg(base_sc + static_cast<long long>(row0 + 32 * warp + 8 * q + g) * (a.K / 128)) * 0x10001u;
  };
  if constexpr (I4) {
    if (n > 0) load_scales(c0, sc_next);
  }

  for (int i = 0; i < n; ++i) {
    const int c = c0 + i;
    const int k = c / cpt - t0;
    const bool first_of_table = i == 0 || (c - 1) / cpt - t0 != k;
    const bool last_of_table = i == n - 1 || (c + 1) / cpt - t0 != k;
    // codebook two tables ahead: request now, park in shared memory after the chunk's math
    const bool fetch2 = !PRIV && first_of_table && k + 2 < nt;
    uint2 vnext = make_uint2(0u, 0u);
    if constexpr (!PRIV) {
      if (fetch2) vnext = fetch_entry<D, B>(a, blk_row, (t0 + k + 2) * cpt, tid);
      if (kTableBuffers<D> == 2 && first_of_table && k + 1 < nt)
        replicate<D, B>(base + ((k + 1) & 1) * P::TABLE_BYTES, compact + ((k + 1) & 1) * P::COMPACT_BYTES, tid);
    }

    if constexpr (I4) {
#pragma unroll
      for (int q = 0; q < 4; ++q) sc[q] = sc_next[q];
      if (i + 1 < n) load_scales(c + 1, sc_next);
    }
    // ---- this warp's indices of the chunk ----
    const int st = i % ST;
    if (!mbar_wait(bars + 8 * st, (i / ST) & 1, kWaitTries) && lane == 0) atomicAdd(a.error_flag, 1);
    uint32_t w[4][LW];
    const uint32_t src = ring + st * T::STAGE_BYTES + row_off;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if constexpr (D == 2 && LW == 6) {
#pragma unroll
        for (int h = 0; h < 3; ++h) {
          const uint2 v = lds64_ordered(src + q * 8 * P::SEG + 8 * h);
          w[q][2 * h] = v.x;
          w[q][2 * h + 1] = v.y;
        }
      } else if constexpr (D == 2) {   // odd word counts: 32-bit reads, conflict-free for odd B
#pragma unroll
        for (int h = 0; h < LW; ++h) w[q][h] = lds32_ordered(src + q * 8 * P::SEG + 4 * h);
      } else {
        const uint4 v = lds128(src + q * 8 * P::SEG);
        w[q][0] = v.x; w[q][1] = v.y; w[q][2] = v.z; w[q][3] = v.w;
      }
    }
    __syncwarp();   // every lane has read the stage: refill it
    if (lane == 0 && i + ST < n) {
      fence_proxy_async();
      issue(i + ST);
    }

    // ---- activations of the lane's 64 columns -> B fragments ----
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        uint4 v = make_uint4(xr[nb][4 * j], xr[nb][4 * j + 1], xr[nb][4 * j + 2], xr[nb][4 * j + 3]);
        lds128_if(v, xaddr[nb] + (i * 8 + j) * xstride, on[nb]);
        xr[nb][4 * j] = v.x; xr[nb][4 * j + 1] = v.y; xr[nb][4 * j + 2] = v.z; xr[nb][4 * j + 3] = v.w;
      }

    // ---- look up + multiply-accumulate ----
    uint32_t tbl = (my_tables + (PRIV || kTableBuffers<D> == 1 ? 0 : (k & 1) * P::TABLE_BYTES)) | lane_off;
    if constexpr (!PRIV && kTableBuffers<D> == 1) fence_value(tbl);
    if constexpr (PRIV) fence_value(tbl);   // the gathers stay behind the warp's own table writes
    chunk_steps<D, B, NB, 0, 4, I4>(acc, w, xr, tbl, sc);
    chunk_steps<D, B, NB, 4, 4, I4>(acc, w, xr, tbl, sc);
    chunk_steps<D, B, NB, 8, 4, I4>(acc, w, xr, tbl, sc);
    chunk_steps<D, B, NB, 12, 4, I4>(acc, w, xr, tbl, sc);

    if constexpr (PRIV) {
      // the warp's table for the next chunk replaces the one it has just finished with (only this
      // warp reads it); the entries of the chunk after it are requested at once
      if (i + 1 < n) {
        fence_acc(acc);   // this chunk's gathers are emitted before the writes
        __syncwarp();     // ... by every lane of the warp
        write_private<B>(my_tables, mine, I4 ? 2 : a.scale != nullptr ? 1 : 0, lane);
        if (i + 2 < n) load_private<B>(mine, a, blk_row, c + 2, lane);
        __syncwarp();
      }
    } else {
      if (fetch2) store_compact<D, B>(compact + (k & 1) * P::COMPACT_BYTES, vnext, tid);
      if (last_of_table && i != n - 1) {
        if constexpr (kTableBuffers<D> == 1) {
          fence_acc(acc);
          __syncthreads();   // every warp has left table k
          replicate<D, B>(base, compact + ((k + 1) & 1) * P::COMPACT_BYTES, tid);
        }
        __syncthreads();   // table k is done with, table k+1 complete
      }
    }
  }

  // ---- combine the K parts ----
  // acc[mt][nb][e]: row 32*warp + 16*mt + g + 8*(e/2) of the slab, batch row nb*8 + 2t + (e&1)
  if (S == 1) {
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = row0 + 32 * warp + 16 * mt + g + 8 * (e >> 1), nn = nb * 8 + 2 * t + (e & 1);
          if (nn < a.batch) a.Y[static_cast<long long>(nn) * a.N + r] = __float2half_rn(acc[mt][nb][e]);
        }
    return;
  }
  // Rows [q*rpo, (q+1)*rpo) of the slab are summed by cluster rank q, which receives one value per
  // (source rank, row, batch row): recv[src][row % rpo][n].  rpo is a multiple of 16.
  const int rpo = T::CTA_ROWS / S;
  const uint32_t recv_u32 = base + a.recv_off;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt) {
    const int r16 = 32 * warp + 16 * mt;             // first row of the 16-row tile
    const int owner = r16 / rpo, slot = r16 % rpo + g;
    const uint32_t dst = map_to_rank(recv_u32 + ((rank * rpo + slot) * NBT + 2 * t) * 4, owner);
    const uint32_t dst_bar = map_to_rank(recv_bar, owner);
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (nb * 8 + 2 * t + (e & 1) < a.batch)
          st_async_f32(dst + ((e >> 1) * 8 * NBT + nb * 8 + (e & 1)) * 4, acc[mt][nb][e], dst_bar);
  }
  // every value this CTA sums has been counted on its barrier; nobody writes here afterwards, so the
  // CTA may leave without a cluster barrier
  if (!mbar_wait(recv_bar, 0, kWaitTries) && tid == 0) atomicAdd(a.error_flag, 1);
  const float* recv = reinterpret_cast<const float*>(smem + a.recv_off);
  for (int o = tid; o < rpo * a.batch; o += T::THREADS) {
    const int nn = o / rpo, slot = o % rpo;
    float sum = 0.f;
    for (int q = 0; q < S; ++q) sum += recv[(q * rpo + slot) * NBT + nn];
    a.Y[static_cast<long long>(nn) * a.N + row0 + rank * rpo + slot] = __float2half_rn(sum);
  }
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
int env_int(const char* name, int dflt) {
#ifdef VQ_TUNING
  if (const char* e = getenv(name)) return atoi(e);
#else
  (void)name;
#endif
  return dflt;
}

size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

template <int D, int B, int NB, bool PRIV = false>
vq_status launch(const StreamCall& call, cudaStream_t s) {
  const Geometry& g = call.g;
  const __half* X = call.X;
  const int batch = call.batch;
  using P = Policy<D, B>;
  using T = Tile<D, B>;
  auto kern = blockcb_kernel<D, B, NB, PRIV, false>;
  if constexpr (D == 2) {
    if (call.g.cb_int4) kern = blockcb_kernel<D, B, NB, PRIV, true>;
  } else {
    if (call.g.cb_int4) return VQ_ERR_UNSUPPORTED;
  }
  static int attr_set[kMaxDevices][2] = {};   // [device][fp16 / int8 kernel, int4 kernel]
  const int which = call.g.cb_int4 ? 1 : 0;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  if (!__atomic_load_n(&attr_set[dev][which], __ATOMIC_ACQUIRE)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess) return VQ_ERR_CUDA;
    __atomic_store_n(&attr_set[dev][which], 1, __ATOMIC_RELEASE);
  }
  int* error_flag = nullptr;
  if (device_error_counter(&error_flag) != VQ_OK) return VQ_ERR_CUDA;

  BlockArgs a;
  a.cb = nullptr;      // (per layer: the kernel takes them from the group)
  a.scale = nullptr;
  a.gscale = nullptr;
  a.X = X;
  a.Y = nullptr;
  a.error_flag = error_flag;
  a.N = 0;
  a.K = g.K;
  a.batch = batch;
  a.n_chunks = g.K / 256;
  a.blocks_per_row = g.blocks_per_row;
  a.Br = g.Br;
  a.Bc = g.Bc;
  BlockGroup grp = {};
  BlockMaps maps;
  grp.n_seg = call.n_seg;
  int row_blocks = 0;
  for (int i = 0; i < call.n_seg; ++i) {
    if (call.N[i] <= 0 || call.N[i] % T::CTA_ROWS) return VQ_ERR_UNSUPPORTED;
    grp.cb[i] = call.cb[i];
    grp.scale[i] = (g.cb_int8 || g.cb_int4) ? call.scale[i] : nullptr;   // per block (int8) or per row and 128 columns (int4)
    grp.Y[i] = call.Y[i];
    grp.N[i] = call.N[i];
    grp.tile0[i] = row_blocks;
    row_blocks += call.N[i] / T::CTA_ROWS;
    // index stream as a 2-D byte tensor: rows of `stride` bytes; one box = 32 rows x SEG bytes
    if (encode_index_map(&maps.m[i], call.idx[i], g.stride, call.N[i], P::SEG, 32) != VQ_OK) return VQ_ERR_CUDA;
  }
  for (int i = call.n_seg; i < kMaxSegments; ++i) maps.m[i] = maps.m[0];

  // Shared memory of a CTA whose column range is `chunks` long.
  // The tables start on a TABLE_BYTES boundary of the CTA's shared-memory window (their address bits
  // merge with the index bits); dynamic shared memory starts 1024 bytes into the window (the first 1024
  // are the system's; the kernel checks what it gets).  Parts that fit into the bytes in front of that
  // boundary go there, largest first (`compact`); the others follow the tables.
  auto smem_for = [&](int chunks, BlockArgs* out, bool use_front) {
    constexpr int ST = kStagesOf<D, PRIV>;
    const size_t tables = (PRIV ? P::WARPS : kTableBuffers<D>) * static_cast<size_t>(P::TABLE_BYTES);
    struct Part { size_t bytes, align; long long off; };
    Part ring = {static_cast<size_t>(P::WARPS) * ST * T::STAGE_BYTES, 128, 0};
    Part x = {static_cast<size_t>(chunks) * 512 * batch, 16, 0};
    Part recv = {static_cast<size_t>(T::CTA_ROWS) * 8 * NB * sizeof(float), 16, 0};
    Part compact = {2 * static_cast<size_t>(P::COMPACT_BYTES), 16, 0};
    Part bars = {static_cast<size_t>(P::WARPS) * ST * 8 + 8, 8, 0};   // rings + receive barrier
    Part* order[5] = {&ring, &x, &recv, &compact, &bars};
    for (int i = 0; i < 5; ++i)   // largest first
      for (int j = i + 1; j < 5; ++j)
        if (order[j]->bytes > order[i]->bytes) { Part* t = order[i]; order[i] = order[j]; order[j] = t; }
    const size_t room = use_front ? P::TABLE_BYTES - 1024 : 0;
    size_t front = 0, after = tables;
    bool in_front[5];
    for (int i = 0; i < 5; ++i) {
      const size_t at = round_up(front, order[i]->align);
      in_front[i] = room > 0 && at + order[i]->bytes <= room;
      if (in_front[i]) {
        order[i]->off = static_cast<long long>(at);
        front = at + order[i]->bytes;
      } else {
        const size_t pos = round_up(after, order[i]->align);
        order[i]->off = static_cast<long long>(pos);
        after = pos + order[i]->bytes;
      }
    }
    front = round_up(front, 128);   // the front region ends at the tables' boundary
    for (int i = 0; i < 5; ++i)
      if (in_front[i]) order[i]->off -= static_cast<long long>(front);
    const size_t lead = round_up(1024 + front, P::TABLE_BYTES) - 1024;
    if (out) {
      out->compact_off = static_cast<int>(compact.off); out->ring_off = static_cast<int>(ring.off);
      out->bar_off = static_cast<int>(bars.off); out->x_off = static_cast<int>(x.off); out->recv_off = static_cast<int>(recv.off);
      out->front_bytes = static_cast<int>(front);
      out->after_bytes = static_cast<int>(after);
    }
    return lead + after;
  };
  // K split: waves of co-resident CTAs times (chunks per CTA + fixed overhead, in chunk times); ties
  // go to the larger split.
  auto plan = [&](bool compact, double* cost_out) {
    int best = 0;
    double best_cost = -1.0;
    for (int S = 1; S <= 8; S *= 2) {
      if (S > a.n_chunks) break;
      const int chunks = (a.n_chunks + S - 1) / S;
      const size_t smem = smem_for(chunks, nullptr, compact);
      if (smem > 220 * 1024) continue;
      const int per_sm = static_cast<int>((228 * 1024) / (smem + 1024));
      const long long ctas = static_cast<long long>(row_blocks) * S;
      const long long slots = static_cast<long long>(per_sm < 1 ? 1 : per_sm) * sms;
      const double waves = static_cast<double>((ctas + slots - 1) / slots);
      const double cost = waves * (chunks + (S > 1 ? 2.0 : 1.5));
      if (best_cost < 0.0 || cost <= best_cost) {
        best_cost = cost;
        best = S;
      }
    }
    *cost_out = best_cost;
    return best;
  };
  // The compact layout lets more CTAs share an SM.  It is taken from batch 3 on, where the staged
  // activations make a CTA large (4-D format at batch 8: one 128 KB CTA per SM becomes two of 96 KB, 106 ->
  // 88 us per 13B-shaped layer set; 2-D 6-bit 32 x 256 blocks at batch 8: 94 -> 87 us).  At batch 1-2 the
  // grids are less than a wave and the plain layout stays: once an extra CTA fits, such a grid spreads
  // unevenly over the SMs (224 CTAs on 148 SMs: 37 against 31 us alone, 67 against 63 us per layer set).
  double cost = -1.0;
  bool compact = batch > 2;
  int best = plan(compact, &cost);
  compact = env_int("VQ_COMPACT", compact ? 1 : 0) != 0;
  best = env_int("VQ_SPLIT", best);
  if (best < 1 || best > 8 || (best & (best - 1)) || best > a.n_chunks) return VQ_ERR_UNSUPPORTED;
  const size_t smem_bytes = smem_for((a.n_chunks + best - 1) / best, &a, compact);
  if (smem_bytes > 220 * 1024) return VQ_ERR_UNSUPPORTED;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(best, row_blocks, 1);
  cfg.blockDim = dim3(T::THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (best > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = best;
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
  if (env_int("VQ_VERBOSE", 0))
    fprintf(stderr, "blockcb launch: split %d row tiles %d smem %zu front %d after %d\n", best, row_blocks, smem_bytes, a.front_bytes, a.after_bytes);
#endif
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, maps, a, grp);
  if (e != cudaSuccess) {
#ifdef VQ_TUNING
    fprintf(stderr, "blockcb launch failed: %s (S %d smem %zu)\n", cudaGetErrorString(e), best, smem_bytes);
#endif
    return VQ_ERR_CUDA;
  }
  return check_launch();
}

}  // namespace

// Shared-codebook families: fp16 or int8 codebooks, block rows a multiple of the CTA's rows, block columns
// a multiple of 128 (2-D) / 256 (4-D), K a multiple of the 256-column chunk.  One launch serves every
// layer of the call (same format and K; rows per layer in call.N).
bool blockcb_covers(const Geometry& g) {
  if (g.K % 256) return false;
  if (g.cb_int4 && g.d != 2) return false;   // int4 codebooks: the 2-D policies only
  if (g.d == 2 && (g.b == 6 || g.b == 5)) return g.Bc % 128 == 0 && (g.Br % 128 == 0 || (g.Br % 32 == 0 && 128 % g.Br == 0));
  if (g.d == 4 && g.b == 8) return g.Br % Tile<4, 8>::CTA_ROWS == 0 && g.Bc % 256 == 0;
  return false;
}

vq_status launch_gemm_blockcb_group(const StreamCall& call, cudaStream_t s) {
  const Geometry& g = call.g;
  const int batch = call.batch;
  if (g.K % 256) return VQ_ERR_UNSUPPORTED;
  if (g.d == 2 && (g.b == 6 || g.b == 5)) {
    if (g.Bc % 128) return VQ_ERR_UNSUPPORTED;
    // blocks of 128 rows or more: one pair of tables per CTA; 32 or 64 rows (the CTA's 128 rows must
    // consist of whole blocks): a pair per warp
    const bool shared_tables = g.Br % 128 == 0;
    if (!shared_tables && (g.Br % 32 || 128 % g.Br)) return VQ_ERR_UNSUPPORTED;
    for (int i = 0; i < call.n_seg; ++i)
      if (call.N[i] % 128) return VQ_ERR_UNSUPPORTED;
    if (g.b == 6) {
      if (shared_tables) return batch <= 8 ? launch<2, 6, 1>(call, s) : launch<2, 6, 2>(call, s);
      return batch <= 8 ? launch<2, 6, 1, true>(call, s) : launch<2, 6, 2, true>(call, s);
    }
    if (shared_tables) return batch <= 8 ? launch<2, 5, 1>(call, s) : launch<2, 5, 2>(call, s);
    return batch <= 8 ? launch<2, 5, 1, true>(call, s) : launch<2, 5, 2, true>(call, s);
  }
  if (g.d == 4 && g.b == 8) {
    if (g.Br % Tile<4, 8>::CTA_ROWS || g.Bc % 256) return VQ_ERR_UNSUPPORTED;
    return batch <= 8 ? launch<4, 8, 1>(call, s) : launch<4, 8, 2>(call, s);
  }
  return VQ_ERR_UNSUPPORTED;
}

vq_status launch_gemm_blockcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s) {
  StreamCall call = {};
  call.g = g;
  call.n_seg = 1;
  call.idx[0] = p.idx;
  call.cb[0] = p.cb;
  call.scale[0] = p.scale;
  call.Y[0] = Y;
  call.N[0] = g.N;
  call.X = X;
  call.batch = batch;
  return launch_gemm_blockcb_group(call, s);
}

}  // namespace vq
