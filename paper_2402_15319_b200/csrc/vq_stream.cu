// Persistent, warp-specialised skinny-GEMM kernel for the VQ-decode linear layer (paper Sec. 3.2:
// packed indices -> look-up table -> mat-vec; App. A: the weight matrix is a look-up of the
// codebook).  The tiling, the pipeline and the reduction are this library's.
//
// Work.  The rows of every layer of a call ("segment": layers that share the activations, e.g. the
// q/k/v or gate/up projections) are cut into slabs of 16*R*WR rows (R row tiles of 16 rows per consumer
// warp, WR row groups per CTA), a row's index stream into WK column parts of S chunks of CHUNK_BYTES.
// A slab takes S pipeline stages; in stage s consumer warp (wr, wk) multiplies its 16*R rows by chunk
// wk*S + s.  The grid is persistent: 1, 2 or 3 CTAs per SM (the kernel is compiled per occupancy, which
// bounds its registers), each with a static share computed from its index alone.  Every CTA takes q =
// slabs / P whole slabs; the stages of the slabs left over form one sequence that is cut into equal
// contiguous pieces, one per CTA, and a CTA walks its piece FIRST, so that the slabs shared with other
// CTAs are summed while everyone still computes whole slabs.
//
// Roles.  Warps 0..W-1 consume (W = WR*WK); warp W (one thread) produces; warp W+1 writes results; warp
// W+2 exists for shared-codebook policies only and builds every stage's look-up tables.
//
// Pipeline.  The producer thread walks the CTA's stages D deep ahead of the consumers with two tiled TMA
// loads per stage, both counted on the stage's "full" mbarrier: a box {CHUNK_BYTES, slab rows, WK parts}
// of the index stream and a box of the activations of the same columns, laid out so that the B
// fragments of mma.sync m16n8k16 (batch row = lane / 4) are read without bank conflicts.  Index boxes
// are issued before the programmatic-dependency wait (weights must be complete before the call is
// enqueued), activation boxes after it.  Consumers wait on "full", expand indices to fp16 weights (A
// fragments; the R row tiles share one activation fragment), run the tensor-core steps with fp32
// accumulation, and release the stage through its "empty" mbarrier.
//
// Reduction.  At the end of a slab the consumers hand their fp32 sums to the results warp through a
// double-buffered shared-memory area; it adds the WK column parts in part order.  A slab whose stages all
// belong to one CTA is rounded to fp16 and stored.  A left-over slab spans several CTAs: each writes
// its partial sums into the workspace and, when its piece is done, draws a ticket from the slab's
// counter; the CTA that draws the last ticket adds the partial sums in CTA order (fixed order: results
// do not depend on timing), stores the outputs and resets the counter to 0.
//
// Shared memory.  Dynamic shared memory starts 1024 bytes into the CTA's window; the hand-over buffers
// and the barriers fill the bytes up to the tables' 4096-byte boundary, tables and stages follow.  The
// kernel checks the size it was given against what the host planned and leaves if they disagree.
//
// Every wait is bounded; a wait that runs out increments a device counter, and the warp stops
// waiting for anything else but still arrives on every barrier it owes, so that the kernel ends.
#include <cstdio>
#include <cstdlib>

#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

using namespace dev;

// Index-word steps of the decode loops that are emitted back to back (8 = the whole chunk; measured
// on B200: 1, 2, 4, 8 steps give 32.3 / 31.4 / 30.7 / 30.0 us on a 28672 x 8192 layer).
#ifndef VQ_UNROLL_D2
#define VQ_UNROLL_D2 8
#endif
#ifndef VQ_UNROLL_D1
#define VQ_UNROLL_D1 8
#endif
constexpr int kUnrollD2 = VQ_UNROLL_D2, kUnrollD1 = VQ_UNROLL_D1;
constexpr int kWaitTries = 1 << 18;   // polls (with a sleep of 40-500 ns in between) before a wait gives up

struct Segment {
  const void* cb;
  const __half* scale;
  __half* Y;
  int N;
  int slab0;   // first slab of the segment in the call's slab sequence
};

struct StreamArgs {
  Segment seg[kMaxSegments];
  int n_seg;
  float* ws_part;     // [CTA][2][16*WR * batch] partial sums
  int* ws_ticket;     // [slab], zero between calls
  int* error_flag;
  int K, batch;
  int S;                 // stages per slab
  int WR, WK, D;
  int q;                 // whole slabs per CTA
  int tail_units;        // stages of the left-over slabs
  int tail_ctas;         // CTAs that share them (each at least one stage)
  int blocks_per_row;
  int cpb_shift;         // row policies: log2 of the chunks that share one codebook block
  int br_shift;          // log2 of the rows that share one codebook block
  int sr_shift;          // log2 of the rows of a slab (16*WR)
  // byte offsets from the tables' boundary (the first BASE_ALIGN boundary that leaves front_bytes of
  // dynamic shared memory in front of it): the slab hand-over buffers and the barriers lie in front
  // (negative offsets), tables and stages behind
  int red_off, bar_off, stage_off;
  int front_bytes, after_bytes;
  int stage_bytes;       // a stage: WK index boxes, then WK activation boxes
  int x_off;             // activations inside a stage
  int idx_part_bytes, x_part_bytes;
  int tbl_off, tbl_part_bytes;   // block policies: the stage's look-up tables
  int Br, Bc, cb_int8;
  uint32_t tx_bytes;     // bytes the two loads of a stage bring
};

struct Maps {
  CUtensorMap idx[kMaxSegments];
  CUtensorMap x;
};

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait for phase `parity` that sleeps `ns` nanoseconds between polls, so that a waiting warp
// leaves the issue slots of its scheduler to the warps that compute.  Returns false if the phase
// did not complete within the attempts.
__device__ __forceinline__ bool mbar_wait_idle(uint32_t bar, uint32_t parity, int max_tries, unsigned ns) {
#pragma unroll 1
  for (int i = 0; i < max_tries; ++i) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    __nanosleep(ns);
  }
  return false;
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ float ldcg_f32(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void tma_box_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
               ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_box_4d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
               ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}
template <int NB>
__device__ __forceinline__ void fence_acc(float (&acc)[NB][4]) {
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int e = 0; e < 4; ++e) asm volatile("" : "+f"(acc[nb][e])::"memory");
}

constexpr uint32_t kMagic = 0x64646464u;      // high byte of fp16 1024.0
constexpr uint32_t kBias2 = 0x64806480u;      // fp16 pair (1152, 1152) = 1024 + 128
// (1024 + u) - 1152 = u - 128, exact in fp16
__device__ __forceinline__ uint32_t mul_f16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ uint32_t sub_bias(uint32_t h) {
  uint32_t r;
  asm("sub.f16x2 %0, %1, %2;" : "=r"(r) : "r"(h), "r"(kBias2));
  return r;
}

// The CTA's walk over its stages: first its piece of the left-over stages (so that the slabs shared
// with other CTAs are summed while the whole slabs are still being computed), then its q whole slabs.
struct Walk {
  int n;           // stages of this CTA
  int n_tail;      // of which in left-over slabs (they come first)
  int t0, t1;      // its piece of the left-over sequence
  int slab, s;     // current stage
  int k;
  int whole0;      // first whole slab of this CTA
  int tail_slab0;  // first left-over slab of the call

  __device__ __forceinline__ void init(const StreamArgs& a, int c, int P) {
    t0 = t1 = 0;
    if (c < a.tail_ctas) {   // (the host keeps tail_units * tail_ctas below 2^31: 32-bit arithmetic)
      t0 = static_cast<int>(static_cast<unsigned>(a.tail_units) * static_cast<unsigned>(c) / static_cast<unsigned>(a.tail_ctas));
      t1 = static_cast<int>(static_cast<unsigned>(a.tail_units) * static_cast<unsigned>(c + 1) / static_cast<unsigned>(a.tail_ctas));
    }
    n_tail = t1 - t0;
    n = n_tail + a.q * a.S;
    whole0 = c * a.q;
    tail_slab0 = a.q * P;
    k = 0;
    if (n_tail > 0) {
      slab = tail_slab0 + t0 / a.S;
      s = t0 % a.S;
    } else {
      slab = whole0;
      s = 0;
    }
  }
  __device__ __forceinline__ void next(const StreamArgs& a) {
    ++k;
    if (k == n_tail) {
      slab = whole0;
      s = 0;
    } else if (++s == a.S) {
      s = 0;
      ++slab;
    }
  }
  // last stage of its slab that this CTA works on
  __device__ __forceinline__ bool slab_end(const StreamArgs& a) const { return s == a.S - 1 || k == n_tail - 1; }
  // does this CTA hold every stage of the current slab?
  __device__ __forceinline__ bool complete(const StreamArgs& a) const {
    if (k >= n_tail) return true;
    const int first_u = (slab - tail_slab0) * a.S;
    return first_u >= t0 && first_u + a.S <= t1;
  }
};

// What a consumer warp knows about the stage it works on.
struct Where {
  int seg;       // segment of the slab
  int row0;      // first of the warp's 16 rows inside the segment
  int ch;        // chunk of the row
  int key;       // identifies (slab, codebook block): equal keys share a table
};

// =============================================================================================
// Row policies: codebooks that belong to one row (or a few rows), 4-bit indices.  Chunk = 128 bytes
// of a row, boxes land with the 128-byte swizzle (16-byte piece p of box row r at p ^ (r & 7)), lane
// (g, t) reads index word 4w + t of rows g and g+8 for w = 0..7: conflict-free 32-bit reads.
// The activations of the 16*d columns that index word 4w + t covers are X_ROW_BYTES / 4 bytes at
// t * X_ROW_BYTES / 4 of row (w, batch row) of the stage's activation box.
// =============================================================================================

// Index words of rows g and g+8: idx = address of the warp's box rows + g*128 + t*4.
__device__ __forceinline__ void load_words(const unsigned char* idx, int ww, uint32_t sw, uint32_t& wl, uint32_t& wh) {
  const unsigned char* p = idx + ((16u * ww) ^ sw);
  wl = *reinterpret_cast<const uint32_t*>(p);
  wh = *reinterpret_cast<const uint32_t*>(p + 1024);
}

// ---- 2-D codebooks of 16 entries (fp16, or int8 + block scale): lane-private fp16 tables in shared
// memory, word (entry, row half, lane) at entry*256 + half*128 + lane*4 from a 4096-byte boundary:
// the entry index sits in address bits 8..11 and merges with the lane's address by one logic op.
template <bool INT8>
struct RowD2B4 {
  static constexpr int CHUNK_BYTES = 128, CHUNK_COLS = 512, X_ROW_BYTES = 128, X_ROWS = 8, LANE_BYTES = 4;
  static constexpr bool X_SWIZZLE = true, IDX_SWIZZLE = true, X_BATCH_INNER = true;
  static constexpr int TILE_TABLE_BYTES = 4096;   // per 16-row tile
  static constexpr int STAGE_TABLE_BYTES = 0, BASE_ALIGN = 4096;
  static constexpr int CB_ROW_BYTES = INT8 ? 32 : 64;
  static constexpr int RAW = INT8 ? 2 : 4;

  template <int NB, int R>
  struct State {
    float acc[R][NB][4];
    uint32_t sc_raw[R][2];      // the block scale of the rows this lane FILLS, twice (an fp16 pair)
    uint32_t raw[R][2][RAW];
    uint32_t tbl, fill, pat;
    int cur_key, pend_key;

    __device__ __forceinline__ void probe_fill(const uint32_t*) {}
    __device__ __forceinline__ void init(uint32_t warp_tbl, int lane) {
      tbl = warp_tbl + lane * 4;
      pat = ((warp_tbl >> 12) & 0xFu) * 0x10101010u;   // address bits 12..15 of the tables, in every byte's high half
      fill = warp_tbl + (4 * (lane >> 3)) * 256 + (lane & 7) * 16;   // entries 4tb..4tb+3, the quad of row gb
      cur_key = pend_key = -1;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[r][nb][e] = 0.f;
    }

    // Request the entries (and scales) of the block of `w`; lane l takes entries 4*(l/8)..+3 of rows
    // l%8 and l%8+8 of every tile (the mapping the table is WRITTEN with) and those rows' scales.
    __device__ __forceinline__ void fetch(const StreamArgs& a, const Where& w, int lane) {
      const Segment& sg = a.seg[w.seg];
      const int blk = w.ch >> a.cpb_shift;
      const int gb = lane & 7, tb = lane >> 3;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int rb = min(w.row0 + 16 * r + gb + 8 * h, sg.N - 1);
          const uint8_t* p = static_cast<const uint8_t*>(sg.cb) +
                             (static_cast<long long>(rb >> a.br_shift) * a.blocks_per_row + blk) * CB_ROW_BYTES + tb * (CB_ROW_BYTES / 4);
          if constexpr (INT8) {
            const uint2 v = ldg64_nc(p);
            raw[r][h][0] = v.x; raw[r][h][1] = v.y;
            const uint32_t s16 = __ldg(reinterpret_cast<const unsigned short*>(sg.scale) + static_cast<long long>(rb >> a.br_shift) * a.blocks_per_row + blk);
            sc_raw[r][h] = s16 * 0x10001u;
          } else {
            const uint4 v = ldg128_nc(p);
            raw[r][h][0] = v.x; raw[r][h][1] = v.y; raw[r][h][2] = v.z; raw[r][h][3] = v.w;
          }
        }
      pend_key = w.key;
    }

    __device__ __forceinline__ void install() {
      __syncwarp();   // every lane is done with the previous tables
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t e[4];
          if constexpr (INT8) {   // the table holds fp16(scale * c), the values vq_decode_weights writes
            e[0] = mul_f16x2(sub_bias(prmt(raw[r][h][0] ^ 0x80808080u, kMagic, 0x4140)), sc_raw[r][h]);
            e[1] = mul_f16x2(sub_bias(prmt(raw[r][h][0] ^ 0x80808080u, kMagic, 0x4342)), sc_raw[r][h]);
            e[2] = mul_f16x2(sub_bias(prmt(raw[r][h][1] ^ 0x80808080u, kMagic, 0x4140)), sc_raw[r][h]);
            e[3] = mul_f16x2(sub_bias(prmt(raw[r][h][1] ^ 0x80808080u, kMagic, 0x4342)), sc_raw[r][h]);
          } else {
#pragma unroll
            for (int i = 0; i < 4; ++i) e[i] = raw[r][h][i];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) sts128(fill + r * TILE_TABLE_BYTES + i * 256 + h * 128, make_uint4(e[i], e[i], e[i], e[i]));
        }
      __syncwarp();
      fence_value(tbl);   // gathers of the new block stay behind the rewrite
    }

    // Hand the slab's sums over (the scales are already inside the tables: one accumulator runs
    // across the blocks of a row).
    __device__ __forceinline__ void flush(float (&total)[R][NB][4]) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            total[r][nb][e] = acc[r][nb][e];
            acc[r][nb][e] = 0.f;
          }
    }

    __device__ __forceinline__ void prefetch(const StreamArgs& a, const Where& next, int lane) {
      if (next.key != cur_key && next.key != pend_key) fetch(a, next, lane);
    }

    // Make the block of `w` the current one (its tables must be complete before the stage's look-ups).
    __device__ __forceinline__ void begin(const StreamArgs& a, const Where& w, int lane, float (&total)[R][NB][4]) {
      if (w.key != cur_key) {
        if (pend_key != w.key) fetch(a, w, lane);
        install();
        cur_key = w.key;
      }
    }

    // Index I of a word whose even indices lie one per byte in `we` and odd ones in `wo`, each byte already
    // carrying address bits 12..15 in its high half: one byte permute puts the byte into bits 8..15 of the
    // lane's table address (a shift and a logic op per look-up otherwise; the integer pipe issues half as
    // many instructions per clock as the four schedulers can).
    template <int I, int OFF>
    __device__ __forceinline__ uint32_t gather(uint32_t we, uint32_t wo) const {
      constexpr uint32_t sel = 0x3200u | ((4u + I / 2) << 4);
      return lds32_off<OFF>(prmt(tbl, (I & 1) ? wo : we, sel));
    }

    template <int RR>
    __device__ __forceinline__ void tile_step(const unsigned char* idx, int ww, uint32_t sw, const uint4 (&b)[NB][2]) {
      uint32_t wl, wh;
      load_words(idx + RR * 2048, ww, sw, wl, wh);
      constexpr int T0 = RR * TILE_TABLE_BYTES, T1 = T0 + 128;
      const uint32_t le = (wl & 0x0F0F0F0Fu) | pat, lo = ((wl >> 4) & 0x0F0F0F0Fu) | pat;
      const uint32_t he = (wh & 0x0F0F0F0Fu) | pat, ho = ((wh >> 4) & 0x0F0F0F0Fu) | pat;
      uint32_t af[4][4];
      af[0][0] = gather<0, T0>(le, lo); af[0][1] = gather<0, T1>(he, ho); af[0][2] = gather<1, T0>(le, lo); af[0][3] = gather<1, T1>(he, ho);
      af[1][0] = gather<2, T0>(le, lo); af[1][1] = gather<2, T1>(he, ho); af[1][2] = gather<3, T0>(le, lo); af[1][3] = gather<3, T1>(he, ho);
      af[2][0] = gather<4, T0>(le, lo); af[2][1] = gather<4, T1>(he, ho); af[2][2] = gather<5, T0>(le, lo); af[2][3] = gather<5, T1>(he, ho);
      af[3][0] = gather<6, T0>(le, lo); af[3][1] = gather<6, T1>(he, ho); af[3][2] = gather<7, T0>(le, lo); af[3][3] = gather<7, T1>(he, ho);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        mma16816(acc[RR][nb], af[0][0], af[0][1], af[0][2], af[0][3], b[nb][0].x, b[nb][0].y);
        mma16816(acc[RR][nb], af[1][0], af[1][1], af[1][2], af[1][3], b[nb][0].z, b[nb][0].w);
        mma16816(acc[RR][nb], af[2][0], af[2][1], af[2][2], af[2][3], b[nb][1].x, b[nb][1].y);
        mma16816(acc[RR][nb], af[3][0], af[3][1], af[3][2], af[3][3], b[nb][1].z, b[nb][1].w);
      }
    }

    // idx: the warp's box rows + g*128 + t*4 (tile r 2048 bytes further); xpart: the part's activation
    // box [w][batch row][128 bytes]; xm[nb]: the lane's batch rows.
    __device__ __forceinline__ void compute(const unsigned char* idx, const unsigned char* xpart, const int (&xm)[NB], int batch,
                                            uint32_t, int lane, float (&)[R][NB][4]) {
      const unsigned char* xrow[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) xrow[nb] = xpart + xm[nb] * X_ROW_BYTES;
      const uint32_t xstep = batch * X_ROW_BYTES;
      const uint32_t sw = static_cast<uint32_t>(lane >> 2) << 4;
      const uint32_t t32 = static_cast<uint32_t>(lane & 3) << 5;
      uint4 b[NB][2];
#pragma unroll kUnrollD2
      for (int ww = 0; ww < 8; ++ww) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          // 32 bytes at t*32 of the 128-byte row; the box is swizzled: piece p of row r at p ^ (r & 7)
          const unsigned char* r = xrow[nb] + ww * xstep;
          const uint32_t ph = (static_cast<uint32_t>(reinterpret_cast<uintptr_t>(r)) >> 3) & 0x70u;
          b[nb][0] = *reinterpret_cast<const uint4*>(r + (t32 ^ ph));
          b[nb][1] = *reinterpret_cast<const uint4*>(r + ((t32 + 16u) ^ ph));
        }
        tile_step<0>(idx, ww, sw, b);
        if constexpr (R > 1) tile_step<1>(idx, ww, sw, b);
        if constexpr (R > 2) tile_step<2>(idx, ww, sw, b);
        if constexpr (R > 3) tile_step<3>(idx, ww, sw, b);
      }
    }
  };
};

// ---- 1-D int8 codebooks of 16 entries + block scale: the row's entries live in 4 registers and
// are looked up with byte permutes, the register-file analogue of the paper's LUT instruction
// (Sec. 3.2: index -> 8-bit value); bytes become fp16 by the 0x6400 exponent trick, exactly.
struct RowD1B4I8 {
  static constexpr int CHUNK_BYTES = 128, CHUNK_COLS = 256, X_ROW_BYTES = 64, X_ROWS = 8, LANE_BYTES = 4;
  static constexpr bool X_SWIZZLE = false, IDX_SWIZZLE = true, X_BATCH_INNER = true;
  static constexpr int TILE_TABLE_BYTES = 0;
  static constexpr int STAGE_TABLE_BYTES = 0, BASE_ALIGN = 4096;

  template <int NB, int R>
  struct State {
    float acc[R][NB][4];
    float sc[R][2], sc_raw[R][2];
    uint32_t T[R][2][4];
    uint4 raw[R][2];
    int cur_key, pend_key;

    // (decode-loop probe) register tables from arbitrary values: w must not be a compile-time constant
    __device__ __forceinline__ void probe_fill(const uint32_t* w) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int i = 0; i < 4; ++i) T[r][h][i] = w[r * 8 + h * 4 + i];
    }
    __device__ __forceinline__ void init(uint32_t, int) {
      cur_key = pend_key = -1;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        sc[r][0] = sc[r][1] = 1.f;
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[r][nb][e] = 0.f;
      }
    }
    __device__ __forceinline__ void fetch(const StreamArgs& a, const Where& w, int lane) {
      const Segment& sg = a.seg[w.seg];
      const int blk = w.ch >> a.cpb_shift;
      const int g = lane >> 2;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int rr = min(w.row0 + 16 * r + g + 8 * h, sg.N - 1);
          const long long b = static_cast<long long>(rr >> a.br_shift) * a.blocks_per_row + blk;
          raw[r][h] = ldg128_nc(static_cast<const uint8_t*>(sg.cb) + b * 16);
          sc_raw[r][h] = __half2float(__ldg(sg.scale + b));
        }
      pend_key = w.key;
    }
    __device__ __forceinline__ void install() {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          T[r][h][0] = raw[r][h].x ^ 0x80808080u; T[r][h][1] = raw[r][h].y ^ 0x80808080u;
          T[r][h][2] = raw[r][h].z ^ 0x80808080u; T[r][h][3] = raw[r][h].w ^ 0x80808080u;
          sc[r][h] = sc_raw[r][h];
        }
    }
    __device__ __forceinline__ void flush(float (&total)[R][NB][4]) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) {
          total[r][nb][0] = fmaf(sc[r][0], acc[r][nb][0], total[r][nb][0]);
          total[r][nb][1] = fmaf(sc[r][0], acc[r][nb][1], total[r][nb][1]);
          total[r][nb][2] = fmaf(sc[r][1], acc[r][nb][2], total[r][nb][2]);
          total[r][nb][3] = fmaf(sc[r][1], acc[r][nb][3], total[r][nb][3]);
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[r][nb][e] = 0.f;
        }
    }
    __device__ __forceinline__ void prefetch(const StreamArgs& a, const Where& next, int lane) {
      if (next.key != cur_key && next.key != pend_key) fetch(a, next, lane);
    }
    __device__ __forceinline__ void begin(const StreamArgs& a, const Where& w, int lane, float (&total)[R][NB][4]) {
      if (w.key != cur_key) {
        flush(total);
        if (pend_key != w.key) fetch(a, w, lane);
        install();
        cur_key = w.key;
      }
    }
    __device__ __forceinline__ void compute(const unsigned char* idx, const unsigned char* xpart, const int (&xm)[NB], int batch,
                                            uint32_t, int lane, float (&)[R][NB][4]) {
      const unsigned char* xrow[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) xrow[nb] = xpart + xm[nb] * X_ROW_BYTES;
      const uint32_t xstep = batch * X_ROW_BYTES;
      const uint32_t sw = static_cast<uint32_t>(lane >> 2) << 4;
      const uint32_t t16 = static_cast<uint32_t>(lane & 3) << 4;
      uint4 b[NB];
#pragma unroll kUnrollD1
      for (int ww = 0; ww < 8; ++ww) {
#pragma unroll
        for (int nb = 0; nb < NB; ++nb) b[nb] = *reinterpret_cast<const uint4*>(xrow[nb] + ww * xstep + t16);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          uint32_t wd[2];
          load_words(idx + r * 2048, ww, sw, wd[0], wd[1]);
          uint32_t af[2][4];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            // selector nibble = entry mod 8 (bit 3 would mean "replicate sign"), looked up in entries
            // 0..7 and 8..15; a second permute picks per index by the index's bit 3
            const uint32_t sel = wd[h] & 0x77777777u;
            const uint32_t pick = ((wd[h] >> 1) & 0x44444444u) | 0x32103210u;
            const uint32_t rL = prmt(prmt(T[r][h][0], T[r][h][1], sel), prmt(T[r][h][2], T[r][h][3], sel), pick);
            const uint32_t rH = prmt(prmt(T[r][h][0], T[r][h][1], sel >> 16), prmt(T[r][h][2], T[r][h][3], sel >> 16), pick >> 16);
            af[0][h] = sub_bias(prmt(rL, kMagic, 0x4140));       // columns 0,1
            af[0][h + 2] = sub_bias(prmt(rL, kMagic, 0x4342));   // columns 2,3
            af[1][h] = sub_bias(prmt(rH, kMagic, 0x4140));       // columns 4,5
            af[1][h + 2] = sub_bias(prmt(rH, kMagic, 0x4342));   // columns 6,7
          }
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            mma16816(acc[r][nb], af[0][0], af[0][1], af[0][2], af[0][3], b[nb].x, b[nb].y);
            mma16816(acc[r][nb], af[1][0], af[1][1], af[1][2], af[1][3], b[nb].z, b[nb].w);
          }
        }
      }
    }
  };
};

// ---- uniform INT4 with an fp16 scale per 128 columns (paper Sec. 2.1 symmetric uniform quantiser;
// Sec. 5, the uniform 4-bit group-128 rows of the tables), the bandwidth yard-stick: no table.  Nibble i
// of an index word is column i of the lane's 8 columns.  Masking the word with 0x000F000F leaves nibbles
// 0 and 4 in the two halves of a register, 0x00F000F0 nibbles 1 and 5 (times 16); merged with the fp16
// exponent of 1024 they are the pairs (1024 + q0, 1024 + q4) and (1024 + 16 q1, 1024 + 16 q5), and one
// fused multiply-add by (1, -1032) or (1/16, -72) makes them (q - 8), exactly.  The tensor-core step sums
// over its 16 columns in any order, so the activations are paired the same way (one byte permute per
// pair, shared by the row tiles): five integer-pipe operations per 8 weights instead of eight.
struct RowInt4G128 {
  static constexpr int CHUNK_BYTES = 128, CHUNK_COLS = 256, X_ROW_BYTES = 64, X_ROWS = 8, LANE_BYTES = 4;
  static constexpr bool X_SWIZZLE = false, IDX_SWIZZLE = true, X_BATCH_INNER = true;
  static constexpr int TILE_TABLE_BYTES = 0;
  static constexpr int STAGE_TABLE_BYTES = 0, BASE_ALIGN = 4096;

  template <int NB, int R>
  struct State {
    uint32_t sc_cur[R][2], sc_next[R][2];   // two fp16 scales (the chunk's two groups) per row
    int cur_key, pend_key;

    __device__ __forceinline__ void probe_fill(const uint32_t*) {}
    __device__ __forceinline__ void init(uint32_t, int) { cur_key = pend_key = -1; }
    __device__ __forceinline__ void fetch(const StreamArgs& a, const Where& w, int lane) {
      const Segment& sg = a.seg[w.seg];
      const int g = lane >> 2;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int rr = min(w.row0 + 16 * r + g + 8 * h, sg.N - 1);
          sc_next[r][h] = __ldg(reinterpret_cast<const uint32_t*>(sg.scale + static_cast<long long>(rr) * (a.K / 128) + 2 * w.ch));
        }
      pend_key = w.key;
    }
    __device__ __forceinline__ void flush(float (&)[R][NB][4]) {}
    __device__ __forceinline__ void prefetch(const StreamArgs& a, const Where& next, int lane) {
      if (next.key != cur_key && next.key != pend_key) fetch(a, next, lane);
    }
    __device__ __forceinline__ void begin(const StreamArgs& a, const Where& w, int lane, float (&)[R][NB][4]) {
      if (w.key != cur_key) {
        if (pend_key != w.key) fetch(a, w, lane);
#pragma unroll
        for (int r = 0; r < R; ++r) {
          sc_cur[r][0] = sc_next[r][0];
          sc_cur[r][1] = sc_next[r][1];
        }
        cur_key = w.key;
      }
    }
    __device__ __forceinline__ void compute(const unsigned char* idx, const unsigned char* xpart, const int (&xm)[NB], int batch,
                                            uint32_t, int lane, float (&total)[R][NB][4]) {
      const unsigned char* xrow[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) xrow[nb] = xpart + xm[nb] * X_ROW_BYTES;
      const uint32_t xstep = batch * X_ROW_BYTES;
      constexpr uint32_t kOne = 0x3C003C00u, kLoAdd = 0xE408E408u;         // (1, 1), (-1032, -1032)
      constexpr uint32_t kSixteenth = 0x2C002C00u, kHiAdd = 0xD480D480u;   // (1/16, 1/16), (-72, -72)
      const uint32_t sw = static_cast<uint32_t>(lane >> 2) << 4;
      const uint32_t t16 = static_cast<uint32_t>(lane & 3) << 4;
      uint4 b[NB];
#pragma unroll 1
      for (int grp = 0; grp < 2; ++grp) {
        float acc[R][NB][4];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
          for (int nb = 0; nb < NB; ++nb)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[r][nb][e] = 0.f;
#pragma unroll kUnrollD1
        for (int w4 = 0; w4 < 4; ++w4) {
          const int ww = 4 * grp + w4;
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            // the lane's 8 activations x0..x7, paired as the nibbles pair below: (x0,x4) (x1,x5) (x2,x6) (x3,x7);
            // one permute per pair, shared by every row tile
            const uint4 v = *reinterpret_cast<const uint4*>(xrow[nb] + ww * xstep + t16);
            b[nb] = make_uint4(prmt(v.x, v.z, 0x5410u), prmt(v.x, v.z, 0x7632u), prmt(v.y, v.w, 0x5410u), prmt(v.y, v.w, 0x7632u));
          }
#pragma unroll
          for (int r = 0; r < R; ++r) {
            uint32_t wd[2];
            load_words(idx + r * 2048, ww, sw, wd[0], wd[1]);
            // nibbles n0..n7 of a word are columns 0..7: one logic op takes (n0, n4) or (16 n1, 16 n5) into
            // the mantissas of the pair (1024, 1024); the word shifted by 8 gives (n2, n6) and (16 n3, 16 n7)
            uint32_t q[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const uint32_t w0 = wd[h], w8 = wd[h] >> 8;
              const uint32_t m0 = (w0 & 0x000F000Fu) | 0x64006400u, m1 = (w0 & 0x00F000F0u) | 0x64006400u;
              const uint32_t m2 = (w8 & 0x000F000Fu) | 0x64006400u, m3 = (w8 & 0x00F000F0u) | 0x64006400u;
              asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(q[h][0]) : "r"(m0), "r"(kOne), "r"(kLoAdd));
              asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(q[h][1]) : "r"(m1), "r"(kSixteenth), "r"(kHiAdd));
              asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(q[h][2]) : "r"(m2), "r"(kOne), "r"(kLoAdd));
              asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(q[h][3]) : "r"(m3), "r"(kSixteenth), "r"(kHiAdd));
            }
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) {
              mma16816(acc[r][nb], q[0][0], q[1][0], q[0][1], q[1][1], b[nb].x, b[nb].y);   // columns 0,4 | 1,5
              mma16816(acc[r][nb], q[0][2], q[1][2], q[0][3], q[1][3], b[nb].z, b[nb].w);   // columns 2,6 | 3,7
            }
          }
        }
        // the group's scale multiplies its fp32 partial sums
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const float s0 = __half2float(__ushort_as_half(static_cast<unsigned short>(grp ? sc_cur[r][0] >> 16 : sc_cur[r][0] & 0xffffu)));
          const float s1 = __half2float(__ushort_as_half(static_cast<unsigned short>(grp ? sc_cur[r][1] >> 16 : sc_cur[r][1] & 0xffffu)));
#pragma unroll
          for (int nb = 0; nb < NB; ++nb) {
            total[r][nb][0] = fmaf(s0, acc[r][nb][0], total[r][nb][0]);
            total[r][nb][1] = fmaf(s0, acc[r][nb][1], total[r][nb][1]);
            total[r][nb][2] = fmaf(s1, acc[r][nb][2], total[r][nb][2]);
            total[r][nb][3] = fmaf(s1, acc[r][nb][3], total[r][nb][3]);
          }
        }
      }
    }
  };
};

// =============================================================================================
// Block policy: 2-D codebooks of 64 entries (6-bit indices) shared by a tall block of rows (fp16, or
// int8 whose entries enter the tables as fp16(scale * c)).  Chunk = 96 bytes of a row = 128 indices
// = 256 columns; lane (g, t) owns the 32 indices (24 bytes, read as three 64-bit words: conflict-free
// with rows 96 bytes apart) of columns 64t .. 64t+63 of rows g and g+8.  A helper warp replicates the
// chunk's codebooks into a lane-private table of the stage, word (entry, lane) at entry*128 + lane*4:
// lanes t < 2 see the block under columns 0..127 of the chunk, lanes t >= 2 the block under columns
// 128..255.  The activations of the chunk lie as [batch row][t][128 bytes] (128-byte swizzle).
// =============================================================================================
struct BlkD2B6 {
  static constexpr int CHUNK_BYTES = 96, CHUNK_COLS = 256, X_ROW_BYTES = 128, X_ROWS = 4, LANE_BYTES = 24;
  static constexpr bool X_SWIZZLE = true, IDX_SWIZZLE = false, X_BATCH_INNER = false;
  static constexpr int TILE_TABLE_BYTES = 0;
  static constexpr int STAGE_TABLE_BYTES = 8192, BASE_ALIGN = 8192;
  static constexpr uint32_t MASK = 63u << 7;

  template <int I>   // (index I of the lane's 32) * 128
  static __device__ __forceinline__ uint32_t entry_off(const uint32_t (&w)[6]) {
    constexpr int p = 6 * I;
    if constexpr (p < 7) {
      return (w[0] << (7 - p)) & MASK;
    } else {
      constexpr int q = p - 7, wi = q >> 5, sft = q & 31;
      if constexpr (sft == 0) return w[wi] & MASK;
      else if constexpr (sft + 13 > 32) return __funnelshift_r(w[wi], w[wi + 1], sft) & MASK;
      else return (w[wi] >> sft) & MASK;
    }
  }

  // The helper warp's share of one part's table: lane l converts entries 2l, 2l+1 of the two blocks
  // under the chunk (requested one stage ahead by load()) and writes each 8 times with 128-bit stores
  // whose 16-byte groups are rotated by the lane (the 8 lanes of a quarter warp hit 8 different groups).
  struct Builder {
    uint32_t raw[2][2];   // [block A / B][entry 2l, 2l+1] (int8: both entries in raw[.][0])
    float sc[2];
    __device__ __forceinline__ void load(const StreamArgs& a, const Segment& sg, int row0, int ch, int lane) {
      const long long brow = static_cast<long long>(row0 >> a.br_shift) * a.blocks_per_row;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const long long blk = brow + (ch * CHUNK_COLS + h * 128) / a.Bc;
        if (a.cb_int8) {
          raw[h][0] = __ldg(reinterpret_cast<const uint32_t*>(static_cast<const uint16_t*>(sg.cb) + blk * 64 + 2 * lane));
          raw[h][1] = 0u;
          sc[h] = __half2float(__ldg(sg.scale + blk));
        } else {
          const uint2 v = ldg64_nc(static_cast<const uint32_t*>(sg.cb) + blk * 64 + 2 * lane);
          raw[h][0] = v.x;
          raw[h][1] = v.y;
          sc[h] = 1.f;
        }
      }
    }
    __device__ __forceinline__ void store(const StreamArgs& a, uint32_t table, int lane) const {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        uint32_t e[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (a.cb_int8) {
            const uint32_t two = raw[h][0] >> (16 * i);
            const __half2 hv = __halves2half2(__float2half_rn(sc[h] * static_cast<float>(static_cast<int8_t>(two & 0xff))),
                                              __float2half_rn(sc[h] * static_cast<float>(static_cast<int8_t>((two >> 8) & 0xff))));
            e[h] = *reinterpret_cast<const uint32_t*>(&hv);
          } else {
            e[h] = raw[h][i];
          }
        }
        const uint4 v = make_uint4(e[0], e[0], e[1], e[1]);
        const uint32_t row = table + (2 * lane + i) * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) sts128(row + ((j + lane) & 7) * 16, v);
      }
    }
  };

  template <int NB, int R>
  struct State {
    float acc[R][NB][4];
    __device__ __forceinline__ void probe_fill(const uint32_t*) {}
    __device__ __forceinline__ void init(uint32_t, int) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[r][nb][e] = 0.f;
    }
    __device__ __forceinline__ void prefetch(const StreamArgs&, const Where&, int) {}
    __device__ __forceinline__ void begin(const StreamArgs&, const Where&, int, float (&)[R][NB][4]) {}
    __device__ __forceinline__ void settle() {
#pragma unroll
      for (int r = 0; r < R; ++r) fence_acc(acc[r]);
    }
    __device__ __forceinline__ void flush(float (&total)[R][NB][4]) {
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            total[r][nb][e] += acc[r][nb][e];
            acc[r][nb][e] = 0.f;
          }
    }

    template <int J, int RR>
    __device__ __forceinline__ void piece_step(const uint32_t (&wl)[6], const uint32_t (&wh)[6], uint32_t tbl, const uint4 (&b)[NB]) {
      // indices 4J .. 4J+3 of rows g and g+8: two tensor-core steps
      uint32_t af[2][4];
      af[0][0] = lds32(entry_off<4 * J>(wl) | tbl);     af[0][1] = lds32(entry_off<4 * J>(wh) | tbl);
      af[0][2] = lds32(entry_off<4 * J + 1>(wl) | tbl); af[0][3] = lds32(entry_off<4 * J + 1>(wh) | tbl);
      af[1][0] = lds32(entry_off<4 * J + 2>(wl) | tbl); af[1][1] = lds32(entry_off<4 * J + 2>(wh) | tbl);
      af[1][2] = lds32(entry_off<4 * J + 3>(wl) | tbl); af[1][3] = lds32(entry_off<4 * J + 3>(wh) | tbl);
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        mma16816(acc[RR][nb], af[0][0], af[0][1], af[0][2], af[0][3], b[nb].x, b[nb].y);
        mma16816(acc[RR][nb], af[1][0], af[1][1], af[1][2], af[1][3], b[nb].z, b[nb].w);
      }
    }

    template <int J>
    __device__ __forceinline__ void piece(const uint32_t (&w)[R][2][6], uint32_t tbl, const unsigned char* const (&xrow)[NB],
                                          const uint32_t (&ph)[NB]) {
      uint4 b[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) b[nb] = *reinterpret_cast<const uint4*>(xrow[nb] + ((16u * J) ^ ph[nb]));
      piece_step<J, 0>(w[0][0], w[0][1], tbl, b);
      if constexpr (R > 1) piece_step<J, 1>(w[1][0], w[1][1], tbl, b);
      if constexpr (R > 2) piece_step<J, 2>(w[2][0], w[2][1], tbl, b);
      if constexpr (R > 3) piece_step<J, 3>(w[3][0], w[3][1], tbl, b);
    }

    // idx: the warp's box rows + g*96 + t*24 (tile r 16 rows further); xpart: [batch row][t][128 bytes];
    // table: shared address of the part's table.
    __device__ __forceinline__ void compute(const unsigned char* idx, const unsigned char* xpart, const int (&xm)[NB], int,
                                            uint32_t table, int lane, float (&)[R][NB][4]) {
      uint32_t w[R][2][6];
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int q = 0; q < 3; ++q) {
            const uint2 v = *reinterpret_cast<const uint2*>(idx + (r * 16 + h * 8) * CHUNK_BYTES + 8 * q);
            w[r][h][2 * q] = v.x;
            w[r][h][2 * q + 1] = v.y;
          }
      const unsigned char* xrow[NB];
      uint32_t ph[NB];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        xrow[nb] = xpart + (xm[nb] * 4 + (lane & 3)) * X_ROW_BYTES;
        ph[nb] = (static_cast<uint32_t>(reinterpret_cast<uintptr_t>(xrow[nb])) >> 3) & 0x70u;
      }
      const uint32_t tbl = table + lane * 4;
      piece<0>(w, tbl, xrow, ph); piece<1>(w, tbl, xrow, ph); piece<2>(w, tbl, xrow, ph); piece<3>(w, tbl, xrow, ph);
      piece<4>(w, tbl, xrow, ph); piece<5>(w, tbl, xrow, ph); piece<6>(w, tbl, xrow, ph); piece<7>(w, tbl, xrow, ph);
    }
  };
};

// =============================================================================================
// The kernel.  Grid (P), block (W + 2) warps: warps 0..W-1 consume (warp = wk*WR + wr), warp W produces
// (one thread), warp W+1 writes the results.  CW = the most consumer warps a launch may use (4: two
// CTAs per SM, 8: one), which fixes the registers a thread may take.
// =============================================================================================
// CPS = CTAs per SM the kernel is compiled for (it bounds the registers of a thread).
template <class P, int NB, int R, int CW, int CPS>
__global__ void __launch_bounds__((CW + (P::STAGE_TABLE_BYTES ? 3 : 2)) * 32, CPS)
stream_kernel(const __grid_constant__ Maps maps, const StreamArgs a) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + a.front_bytes + (P::BASE_ALIGN - 1)) & ~static_cast<uint32_t>(P::BASE_ALIGN - 1);
  unsigned char* smem = smem_raw + (sbase - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  {   // the host sized the launch for dynamic shared memory that starts 1024 bytes into the CTA's window
    uint32_t dyn;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    if (sbase - smem_u32(smem_raw) + static_cast<uint32_t>(a.after_bytes) > dyn) {   // (the same for every thread)
      if (tid == 0) atomicAdd(a.error_flag, 1);
      return;
    }
  }
  const int W = a.WR * a.WK;
  const int D = a.D;
  // barriers: full[D], empty[D] (pipeline stages); out_full[2], out_empty[2] (results of a slab)
  const uint32_t full0 = sbase + a.bar_off, empty0 = full0 + 8 * D;
  const uint32_t out_full0 = empty0 + 8 * D, out_empty0 = out_full0 + 16;
  constexpr int NBT = 8 * NB;
  const int red_floats = W * R * 16 * a.batch;   // one buffer of the slab's partial sums: [wk][16*R*WR rows][batch]

  if (tid == 0) {
    for (int i = 0; i < D; ++i) {
      mbar_init(full0 + 8 * i, P::STAGE_TABLE_BYTES ? 2 : 1);   // the producer's arrival (+ the table builder's)
      mbar_init(empty0 + 8 * i, W);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(out_full0 + 8 * i, W);
      mbar_init(out_empty0 + 8 * i, 1);
    }
    mbar_init_fence();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int c = blockIdx.x, Pn = gridDim.x;
  const int slab_rows = 16 * R * a.WR;
  Walk wk_;
  wk_.init(a, c, Pn);

  auto segment_of = [&](int slab) {
    int sgi = 0;
#pragma unroll
    for (int i = 1; i < kMaxSegments; ++i)
      if (i < a.n_seg && slab >= a.seg[i].slab0) sgi = i;
    return sgi;
  };

  // ------------------------------------------------------------------------------------------
  // producer: one thread
  // ------------------------------------------------------------------------------------------
  if (warp == W) {
    if (lane != 0) return;
    prefetch_tensormap(&maps.x);
    for (int i = 0; i < a.n_seg; ++i) prefetch_tensormap(&maps.idx[i]);
    bool waited = false;
    for (; wk_.k < wk_.n; wk_.next(a)) {
      const int k = wk_.k, slot = k % D;
      const uint32_t full = full0 + 8 * slot;
      if (k >= D && !mbar_wait_idle(empty0 + 8 * slot, ((k / D) & 1) ^ 1, kWaitTries, 200)) {
        atomicAdd(a.error_flag, 1);
        break;
      }
      const int sg = segment_of(wk_.slab);
      const int row0 = (wk_.slab - a.seg[sg].slab0) * slab_rows;
      const uint32_t stage = sbase + a.stage_off + slot * a.stage_bytes;
      mbar_arrive_expect_tx(full, a.tx_bytes);
      // indices: {CHUNK_BYTES, slab rows, WK parts} at (byte s*CHUNK_BYTES of a part, row, part 0)
      tma_box_3d(stage, &maps.idx[sg], wk_.s * P::CHUNK_BYTES, row0, 0, full);
      if (!waited) {   // the activations belong to the previous kernel of the stream until here
        pdl_wait();
        waited = true;
      }
      // activations of the stage's columns: box rows s*X_ROWS .. of every part
      if constexpr (P::X_BATCH_INNER) tma_box_4d(stage + a.x_off, &maps.x, 0, 0, wk_.s * P::X_ROWS, 0, full);
      else tma_box_4d(stage + a.x_off, &maps.x, 0, wk_.s * P::X_ROWS, 0, 0, full);
    }
    return;
  }

  // ------------------------------------------------------------------------------------------
  // table builder (formats whose codebook is shared by a block of rows): one warp replicates the
  // codebooks under every stage's chunks into the stage's lane-private tables, one stage ahead of
  // its global loads
  // ------------------------------------------------------------------------------------------
  if constexpr (P::STAGE_TABLE_BYTES > 0) {
    if (warp == W + 2) {
      typename P::Builder cur[2], nxt[2];   // at most two column parts per stage
      auto request = [&](typename P::Builder (&b)[2], const Walk& w) {
        const int sg = segment_of(w.slab);
        const int row0 = (w.slab - a.seg[sg].slab0) * slab_rows;
        for (int p = 0; p < a.WK && p < 2; ++p) b[p].load(a, a.seg[sg], row0, p * a.S + w.s, lane);
      };
      if (wk_.n > 0) request(cur, wk_);
      for (; wk_.k < wk_.n;) {
        const int k = wk_.k, slot = k % D;
        wk_.next(a);
        if (wk_.k < wk_.n) request(nxt, wk_);
        if (k >= D && !mbar_wait_idle(empty0 + 8 * slot, ((k / D) & 1) ^ 1, kWaitTries, 200)) {
          if (lane == 0) atomicAdd(a.error_flag, 1);
          break;
        }
        const uint32_t tables = sbase + a.stage_off + slot * a.stage_bytes + a.tbl_off;
        for (int p = 0; p < a.WK && p < 2; ++p) cur[p].store(a, tables + p * a.tbl_part_bytes, lane);
        __syncwarp();
        if (lane == 0) mbar_arrive(full0 + 8 * slot);
        cur[0] = nxt[0];
        cur[1] = nxt[1];
      }
      return;
    }
  }

  // ------------------------------------------------------------------------------------------
  // results: one warp takes the slabs' partial sums from the consumers, adds the WK column parts in
  // part order and stores the outputs (or, for a slab shared with other CTAs, this CTA's share)
  // ------------------------------------------------------------------------------------------
  if (warp == W + 1) {
    pdl_wait();   // outputs and workspace belong to earlier kernels of the stream until here
    int ev = 0;                                   // slabs handed over so far
    int n_partial = 0, partial_a = 0, partial_b = 0;
    bool dead = false;
    for (; wk_.k < wk_.n; wk_.next(a)) {
      if (!wk_.slab_end(a)) continue;
      const int buf = ev & 1;
      if (!dead && !mbar_wait_idle(out_full0 + 8 * buf, (ev >> 1) & 1, kWaitTries, 500)) {
        if (lane == 0) atomicAdd(a.error_flag, 1);
        dead = true;
      }
      dead = __any_sync(0xffffffffu, dead);
      const int slab = wk_.slab;
      const bool complete = wk_.complete(a);
      const Segment& sg = a.seg[segment_of(slab)];
      const int srow0 = (slab - sg.slab0) * slab_rows;
      const int n_out = slab_rows * a.batch;
      const float* red = reinterpret_cast<const float*>(smem + a.red_off) + buf * red_floats;
      // this CTA's share of a left-over slab goes to the workspace: slot 0 if the CTA's piece begins
      // inside this slab, else slot 1
      float* part = nullptr;
      if (!complete) {
        const int my_slot = (wk_.tail_slab0 + wk_.t0 / a.S == slab) ? 0 : 1;
        part = a.ws_part + (static_cast<long long>(c) * 2 + my_slot) * n_out;
        if (n_partial == 0) partial_a = slab;
        else partial_b = slab;
        ++n_partial;
      }
      if (!dead) {
        for (int o = lane; o < n_out; o += 32) {
          const int n = o >> a.sr_shift, rr = o & (slab_rows - 1);
          float sum = 0.f;
          for (int p = 0; p < a.WK; ++p) sum += red[(p * slab_rows + rr) * a.batch + n];
          if (complete) {
            if (srow0 + rr < sg.N) sg.Y[static_cast<long long>(n) * sg.N + srow0 + rr] = __float2half_rn(sum);
          } else {
            part[o] = sum;
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(out_empty0 + 8 * buf);   // the buffer may be refilled
      ++ev;

      // ---- the CTA's piece of the left-over stages is done: tickets, and the sums of the slabs
      // this CTA completes (the consumers are already at work on the whole slabs) ----
      if (wk_.k == wk_.n_tail - 1 && n_partial > 0) {
        if (n_partial > 2) n_partial = 2;   // (cannot happen: a piece is shorter than a slab)
        const long long T = a.tail_units;
        const int Pt = a.tail_ctas;
        int last_mask = 0;
        if (lane == 0) {
          __threadfence();            // this warp's partial sums are visible to the GPU before a ticket is drawn
          for (int i = 0; i < n_partial; ++i) {
            const int ps = i == 0 ? partial_a : partial_b;
            const int first_u = (ps - wk_.tail_slab0) * a.S, last_u = first_u + a.S - 1;
            const int c_first = static_cast<int>((static_cast<long long>(first_u + 1) * Pt - 1) / T);
            const int c_last = static_cast<int>((static_cast<long long>(last_u + 1) * Pt - 1) / T);
            const int ticket = atomicAdd(a.ws_ticket + ps, 1);
            if (ticket == c_last - c_first) {
              a.ws_ticket[ps] = 0;   // nobody else touches the counter in this call
              last_mask |= 1 << i;
            }
          }
          if (last_mask) __threadfence();   // the other CTAs' partial sums are visible after the tickets
        }
        last_mask = __shfl_sync(0xffffffffu, last_mask, 0);
        for (int i = 0; i < n_partial; ++i) {
          if (!(last_mask >> i & 1)) continue;
          const int ps = i == 0 ? partial_a : partial_b;
          const Segment& sp = a.seg[segment_of(ps)];
          const int prow0 = (ps - sp.slab0) * slab_rows;
          const int first_u = (ps - wk_.tail_slab0) * a.S, last_u = first_u + a.S - 1;
          const int c_first = static_cast<int>((static_cast<long long>(first_u + 1) * Pt - 1) / T);
          const int c_last = static_cast<int>((static_cast<long long>(last_u + 1) * Pt - 1) / T);
          // four adjacent outputs per lane and pass; the contributors' values are requested eight at a
          // time before any is used (the loads overlap), and added in CTA order
          for (int o = 4 * lane; o < n_out; o += 128) {
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int q0 = c_first; q0 <= c_last; q0 += 8) {
              float4 v[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int qc = q0 + i;
                v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (qc <= c_last) {
                  const int q_t0 = static_cast<int>(T * qc / Pt);
                  const int q_slot = (wk_.tail_slab0 + q_t0 / a.S == ps) ? 0 : 1;
                  v[i] = __ldcg(reinterpret_cast<const float4*>(a.ws_part + (static_cast<long long>(qc) * 2 + q_slot) * n_out + o));
                }
              }
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                sum.x += v[i].x; sum.y += v[i].y; sum.z += v[i].z; sum.w += v[i].w;
              }
            }
            const float sv[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const int n = (o + j) >> a.sr_shift, rr = (o + j) & (slab_rows - 1);
              if (prow0 + rr < sp.N) sp.Y[static_cast<long long>(n) * sp.N + prow0 + rr] = __float2half_rn(sv[j]);
            }
          }
        }
      }
    }
    return;
  }
  if (warp > W + 1) return;   // (lanes of no role)

  // ------------------------------------------------------------------------------------------
  // consumers
  // ------------------------------------------------------------------------------------------
  const int g = lane >> 2, t = lane & 3;
  const int wr = warp % a.WR, wk = warp / a.WR;
  bool dead = false;

  typename P::template State<NB, R> st;
  st.init(sbase + warp * (R * P::TILE_TABLE_BYTES), lane);
  float total[R][NB][4];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) total[r][nb][e] = 0.f;
  // batch row of the lane's B fragments; lanes beyond the batch re-read the last row (their columns
  // of the result are never stored)
  int xm[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) xm[nb] = min(nb * 8 + g, a.batch - 1);

  auto where = [&](int slab, int s) {
    Where w;
    w.seg = segment_of(slab);
    w.row0 = (slab - a.seg[w.seg].slab0) * slab_rows + wr * (16 * R);
    w.ch = wk * a.S + s;
    w.key = slab * a.blocks_per_row + (w.ch >> a.cpb_shift);
    return w;
  };

  int ev = 0;
  int slot = 0;             // k % D and the parity of k / D, kept incrementally
  uint32_t phase = 0;
  Where cur = where(wk_.slab, wk_.s);
  if (wk_.n > 0) st.prefetch(a, cur, lane);
  for (; wk_.k < wk_.n;) {
    const bool slab_end = wk_.slab_end(a);
    const int slab_before = wk_.slab;
    st.begin(a, cur, lane, total);
    wk_.next(a);
    Where nxt = cur;
    if (wk_.k < wk_.n) {   // the stage after this one: request its codebook if it is another block
      if (wk_.slab == slab_before) {   // same slab: the next chunk of the same rows
        nxt.ch = cur.ch + 1;
        nxt.key = slab_before * a.blocks_per_row + (nxt.ch >> a.cpb_shift);
      } else {
        nxt = where(wk_.slab, wk_.s);
      }
      st.prefetch(a, nxt, lane);
    }
    if (!dead && !mbar_wait_idle(full0 + 8 * slot, phase, kWaitTries, 40)) {
      if (lane == 0) atomicAdd(a.error_flag, 1);
      dead = true;
    }
    dead = __any_sync(0xffffffffu, dead);   // (a vote outside the branch: the warp stays converged)
    if (!dead) {
      const unsigned char* stage = smem + a.stage_off + slot * a.stage_bytes;
      const unsigned char* idx = stage + wk * a.idx_part_bytes + (wr * (16 * R) + g) * P::CHUNK_BYTES + t * P::LANE_BYTES;
      const uint32_t table = sbase + a.stage_off + slot * a.stage_bytes + a.tbl_off + wk * a.tbl_part_bytes;
      st.compute(idx, stage + a.x_off + wk * a.x_part_bytes, xm, a.batch, table, lane, total);
      // the stage's tables may be rewritten once it is released: its look-ups are done before
      if constexpr (P::STAGE_TABLE_BYTES > 0) st.settle();
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + 8 * slot);
    if (++slot == D) {
      slot = 0;
      phase ^= 1u;
    }

    if (slab_end) {
      // ---- hand the slab's partial sums to the results warp ----
      st.flush(total);
      const int buf = ev & 1;
      if (ev >= 2 && !dead && !mbar_wait_idle(out_empty0 + 8 * buf, ((ev >> 1) & 1) ^ 1, kWaitTries, 100)) {
        if (lane == 0) atomicAdd(a.error_flag, 1);
        dead = true;
      }
      dead = __any_sync(0xffffffffu, dead);
      // total[r][nb][e]: row 16r + g + 8*(e/2) of the warp's rows, batch row nb*8 + 2t + (e&1)
      // (only batch rows that exist are kept)
      float* mine = reinterpret_cast<float*>(smem + a.red_off) + buf * red_floats + ((wk * a.WR + wr) * (16 * R) + g) * a.batch + 2 * t;
#pragma unroll
      for (int r = 0; r < R; ++r)
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (nb * 8 + 2 * t + (e & 1) < a.batch) mine[(r * 16 + (e >> 1) * 8) * a.batch + nb * 8 + (e & 1)] = total[r][nb][e];
            total[r][nb][e] = 0.f;
          }
      __syncwarp();
      if (lane == 0) mbar_arrive(out_full0 + 8 * buf);
      ++ev;
    }
    cur = nxt;
  }
}

// =============================================================================================
// host side
// =============================================================================================
int env_int(const char* name, int dflt) {
#ifdef VQ_TUNING
  if (const char* e = getenv(name)) return atoi(e);
#else
  (void)name;
#endif
  return dflt;
}

size_t round_up(size_t v, size_t al) { return (v + al - 1) / al * al; }

constexpr size_t kSmemMax = 224 * 1024;

template <class P, int NB, int R, int CW, int CPS>
vq_status launch(const StreamCall& call, int chunks_per_block, cudaStream_t s, int want_wk, int min_depth) {
  auto kern = stream_kernel<P, NB, R, CW, CPS>;
  static int attr_set[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  if (!__atomic_load_n(&attr_set[dev], __ATOMIC_ACQUIRE)) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemMax)) != cudaSuccess)
      return VQ_ERR_CUDA;
    __atomic_store_n(&attr_set[dev], 1, __ATOMIC_RELEASE);
  }
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;

  const Geometry& g = call.g;
  const int batch = call.batch;
  auto log2_exact = [](int v) {
    int l = 0;
    while ((1 << l) < v) ++l;
    return (1 << l) == v ? l : -1;
  };
  StreamArgs a = {};
  a.n_seg = call.n_seg;
  a.K = g.K;
  a.batch = batch;
  a.blocks_per_row = g.blocks_per_row;
  a.cpb_shift = log2_exact(chunks_per_block);
  a.br_shift = log2_exact(g.Br);
  if (a.cpb_shift < 0 || a.br_shift < 0) return VQ_ERR_UNSUPPORTED;
  const int n_chunks = static_cast<int>(g.stride / P::CHUNK_BYTES);
  if (device_error_counter(&a.error_flag) != VQ_OK) return VQ_ERR_CUDA;

  // ---- CTA shape: W = WR row tiles x WK column parts (WK divides the chunks of a row); D stages ----
  int W = CW;
  int ctas_per_sm = CPS;
  int WK = n_chunks % 4 == 0 ? 4 : n_chunks % 2 == 0 ? 2 : 1;
  if (P::STAGE_TABLE_BYTES) {   // shared tables: as many row tiles of the block as the CTA has warps, then column parts
    const int tiles = g.Br / (16 * R);
    WK = tiles >= CW ? 1 : (n_chunks % 2 == 0 && CW / (tiles < 1 ? 1 : tiles) >= 2 ? 2 : 1);
  }
  if (want_wk > 0 && !P::STAGE_TABLE_BYTES) WK = want_wk;
  WK = env_int("VQ_WK", WK);
  if (P::STAGE_TABLE_BYTES && WK > 2) return VQ_ERR_UNSUPPORTED;
  if (WK < 1 || n_chunks % WK || W % WK) return VQ_ERR_UNSUPPORTED;
  int WR = W / WK;
  if (P::STAGE_TABLE_BYTES && WR > g.Br / (16 * R)) WR = g.Br / (16 * R);   // a slab stays inside one block row
  WR = env_int("VQ_WR", WR);
  if (WR < 1 || WR * WK > CW || log2_exact(WR) < 0 || 16 * R * WR > kMaxSlabRows) return VQ_ERR_UNSUPPORTED;
  if (P::STAGE_TABLE_BYTES && g.Br % (16 * R * WR)) return VQ_ERR_UNSUPPORTED;   // a slab lies inside one block row
  W = WR * WK;
  a.sr_shift = 4 + log2_exact(WR * R);
  a.WR = WR;
  a.WK = WK;
  a.S = n_chunks / WK;
  const int slab_rows = 16 * R * WR;
  int slabs = 0;
  for (int i = 0; i < call.n_seg; ++i) {
    a.seg[i].cb = call.cb[i];
    a.seg[i].scale = call.scale[i];
    a.seg[i].Y = call.Y[i];
    a.seg[i].N = call.N[i];
    a.seg[i].slab0 = slabs;
    slabs += (call.N[i] + slab_rows - 1) / slab_rows;
  }
  if (static_cast<long long>(slabs) * a.S > 0x3fffffff || static_cast<long long>(slabs) * a.blocks_per_row > 0x3fffffff)
    return VQ_ERR_UNSUPPORTED;

  const size_t tbl_bytes = static_cast<size_t>(P::TILE_TABLE_BYTES) * R * W;
  const size_t red_bytes = round_up(2 * static_cast<size_t>(W) * R * 16 * batch * sizeof(float), 16);   // two buffers
  const size_t idx_part = static_cast<size_t>(slab_rows) * P::CHUNK_BYTES;       // multiple of 512
  const size_t x_part = static_cast<size_t>(P::X_ROWS) * batch * P::X_ROW_BYTES;
  const size_t x_off = round_up(idx_part * WK, 1024);
  const size_t tbl_off = round_up(x_off + x_part * WK, P::STAGE_TABLE_BYTES ? P::STAGE_TABLE_BYTES : 1024);
  const size_t stage_bytes = round_up(tbl_off + static_cast<size_t>(P::STAGE_TABLE_BYTES) * WK, P::STAGE_TABLE_BYTES ? P::STAGE_TABLE_BYTES : 1024);
  // In front of the tables: the slab hand-over buffers and the barriers.  Dynamic shared memory starts
  // 1024 bytes into the CTA's window (the first 1024 are the system's; the kernel checks what it gets), so
  // the tables' boundary lies `lead` bytes in and the front region fills bytes that alignment would waste.
  const size_t front = round_up(red_bytes + 16 * 16 + 32, 16);
  const size_t lead = round_up(1024 + front, P::BASE_ALIGN) - 1024;
  const size_t stage_off = round_up(tbl_bytes, P::STAGE_TABLE_BYTES ? P::STAGE_TABLE_BYTES : 1024);
  // shared memory of a CTA: the SM's 228 KB shared by the resident CTAs, 1 KB of each for the system
  size_t budget = (228 * 1024) / ctas_per_sm - 1024;
  if (budget > kSmemMax) budget = kSmemMax;
  const size_t kSlack = lead;
  if (budget < stage_off + kSlack + static_cast<size_t>(min_depth) * stage_bytes) {   // does not fit CPS times
    if (CW <= 4) return VQ_ERR_UNSUPPORTED;   // (a 4-warp CTA alone on an SM would leave it half empty)
    ctas_per_sm = 1;
    budget = kSmemMax;
  }
  if (budget < stage_off + kSlack + 2 * stage_bytes) return VQ_ERR_UNSUPPORTED;
  int D = static_cast<int>((budget - kSlack - stage_off) / stage_bytes);
  if (D > 8) D = 8;
  D = env_int("VQ_D", D);
  if (D < min_depth || D > 16) return VQ_ERR_UNSUPPORTED;
  const size_t smem_bytes = stage_off + static_cast<size_t>(D) * stage_bytes + kSlack;
  if (smem_bytes > kSmemMax) return VQ_ERR_UNSUPPORTED;
  a.D = D;
  a.front_bytes = static_cast<int>(front);
  a.after_bytes = static_cast<int>(stage_off + static_cast<size_t>(D) * stage_bytes);
  a.red_off = -static_cast<int>(front);
  a.bar_off = -static_cast<int>(front) + static_cast<int>(red_bytes);
  if (CPS > 2) {   // three CTAs per SM only if the device agrees that they fit
    int resident = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kern, (W + (P::STAGE_TABLE_BYTES ? 3 : 2)) * 32, smem_bytes) != cudaSuccess)
      return VQ_ERR_CUDA;
    if (resident < CPS) return VQ_ERR_UNSUPPORTED;
  }
  a.stage_off = static_cast<int>(stage_off);
  a.stage_bytes = static_cast<int>(stage_bytes);
  a.x_off = static_cast<int>(x_off);
  a.idx_part_bytes = static_cast<int>(idx_part);
  a.x_part_bytes = static_cast<int>(x_part);
  a.tbl_off = static_cast<int>(tbl_off);
  a.tbl_part_bytes = P::STAGE_TABLE_BYTES;
  a.Br = g.Br;
  a.Bc = g.Bc;
  a.cb_int8 = g.cb_int8;
  a.tx_bytes = static_cast<uint32_t>((idx_part + x_part) * WK);

  // ---- persistent CTAs: whole slabs first, the left-over stages shared evenly ----
  int Pn = env_int("VQ_P", sms * ctas_per_sm);
  if (Pn > kMaxStreamCtas) Pn = kMaxStreamCtas;
  if (Pn < 1) return VQ_ERR_UNSUPPORTED;
  a.q = slabs / Pn;
  const int left = slabs - a.q * Pn;
  const long long tail = static_cast<long long>(left) * a.S;
  a.tail_units = static_cast<int>(tail);
  a.tail_ctas = static_cast<int>(tail < Pn ? tail : Pn);
  if (tail * (a.tail_ctas + 1) >= (1LL << 31)) return VQ_ERR_UNSUPPORTED;   // the kernel splits the tail in 32-bit arithmetic
  // Left-over slabs are either cut into stages shared evenly by all CTAs (their partial sums then meet
  // through the workspace, which costs about two stage times at the end of the kernel) or handed out
  // whole, one per CTA, whichever ends earlier.
  const double t_split = static_cast<double>(slabs) * a.S / Pn + 2.0;
  const double t_whole = static_cast<double>(a.q + (left > 0 ? 1 : 0)) * a.S;
  if (env_int("VQ_NOSPLIT", t_whole <= t_split ? 1 : 0)) a.tail_ctas = left;
  if (a.q == 0) Pn = a.tail_ctas;   // fewer stages than CTAs: the others would have nothing to do
  if (Pn < 1) return VQ_ERR_UNSUPPORTED;
  // the counters take the same room whatever the slab height, so that the partial sums of one call
  // never land where another call (other batch size, other tiling) keeps its counters
  long long rows_total = 0;
  for (int i = 0; i < call.n_seg; ++i) rows_total += call.N[i];
  const size_t ticket_bytes = stream_ticket_bytes(rows_total);
  if (static_cast<size_t>(slabs) * sizeof(int) > ticket_bytes) return VQ_ERR_UNSUPPORTED;
  const size_t part_ws = static_cast<size_t>(Pn) * 2 * slab_rows * batch * sizeof(float);
  if (!call.ws || call.ws_bytes < ticket_bytes + part_ws) return VQ_ERR_WORKSPACE;
  a.ws_ticket = static_cast<int*>(call.ws);
  a.ws_part = reinterpret_cast<float*>(static_cast<char*>(call.ws) + ticket_bytes);

  // ---- tensor maps ----
  Maps maps;
  for (int i = 0; i < call.n_seg; ++i) {
    // index stream: bytes of a part, rows, parts
    const uint64_t dims[3] = {static_cast<uint64_t>(a.S) * P::CHUNK_BYTES, static_cast<uint64_t>(call.N[i]), static_cast<uint64_t>(WK)};
    const uint64_t strides[2] = {static_cast<uint64_t>(g.stride), static_cast<uint64_t>(a.S) * P::CHUNK_BYTES};
    const uint32_t box[3] = {P::CHUNK_BYTES, static_cast<uint32_t>(slab_rows), static_cast<uint32_t>(WK)};
    if (encode_tensor_map(&maps.idx[i], call.idx[i], 1, 3, dims, strides, box, P::IDX_SWIZZLE ? 2 : 0) != VQ_OK) return VQ_ERR_CUDA;
  }
  for (int i = call.n_seg; i < kMaxSegments; ++i) maps.idx[i] = maps.idx[0];
  {
    // activations: columns of a row of the box, batch rows, box rows of a part, parts
    const uint32_t row_cols = P::X_ROW_BYTES / 2;
    const uint64_t rows_per_part = static_cast<uint64_t>(a.S) * P::X_ROWS;   // box rows of X_ROW_BYTES in a part
    if (P::X_BATCH_INNER) {   // shared memory [part][box row][batch row][row bytes]
      const uint64_t dims[4] = {row_cols, static_cast<uint64_t>(batch), rows_per_part, static_cast<uint64_t>(WK)};
      const uint64_t strides[3] = {static_cast<uint64_t>(g.K) * 2, P::X_ROW_BYTES, rows_per_part * P::X_ROW_BYTES};
      const uint32_t box[4] = {row_cols, static_cast<uint32_t>(batch), P::X_ROWS, static_cast<uint32_t>(WK)};
      if (encode_tensor_map(&maps.x, call.X, 2, 4, dims, strides, box, P::X_SWIZZLE ? 2 : 0) != VQ_OK) return VQ_ERR_CUDA;
    } else {                  // shared memory [part][batch row][box row][row bytes]
      const uint64_t dims[4] = {row_cols, rows_per_part, static_cast<uint64_t>(batch), static_cast<uint64_t>(WK)};
      const uint64_t strides[3] = {P::X_ROW_BYTES, static_cast<uint64_t>(g.K) * 2, rows_per_part * P::X_ROW_BYTES};
      const uint32_t box[4] = {row_cols, P::X_ROWS, static_cast<uint32_t>(batch), static_cast<uint32_t>(WK)};
      if (encode_tensor_map(&maps.x, call.X, 2, 4, dims, strides, box, P::X_SWIZZLE ? 2 : 0) != VQ_OK) return VQ_ERR_CUDA;
    }
  }

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(Pn, 1, 1);
  cfg.blockDim = dim3((W + (P::STAGE_TABLE_BYTES ? 3 : 2)) * 32, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  int na = 0;
  if (env_int("VQ_PDL", 1)) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
#ifdef VQ_TUNING
  if (env_int("VQ_VERBOSE", 0))
    fprintf(stderr, "stream launch: CPS %d grid %d block %d depth %d smem %zu WR %d WK %d R %d\n", CPS, Pn, (int)cfg.blockDim.x, D, smem_bytes, WR, WK, R);
#endif
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, maps, a);
  if (e != cudaSuccess) {
#ifdef VQ_TUNING
    fprintf(stderr, "stream launch failed: %s (P %d WR %d WK %d D %d smem %zu)\n", cudaGetErrorString(e), Pn, WR, WK, D, smem_bytes);
#endif
    return VQ_ERR_CUDA;
  }
  return check_launch();
}

// Row tiles per consumer warp: the activation fragments of a step are loaded once and used by every
// tile, so more tiles per warp mean fewer shared-memory cycles per weight; small layers keep one
// tile so that there are enough slabs for every SM.
template <class P, int NB>
vq_status launch_tiles(const StreamCall& call, int chunks_per_block, cudaStream_t s) {
  long long rows = 0;
  for (int i = 0; i < call.n_seg; ++i) rows += call.N[i];
  // two row tiles per warp share one activation fragment (batch 9-16, two batch tiles: one row tile;
  // two were tried in the 8-warp shape, 75 against 53 us on 28672 x 8192 at batch 12)
  int R = NB == 1 && rows >= 8192 ? 2 : 1;
  // shared tables: two tiles per warp make a 4-warp CTA cover a whole 128-row block per table
  if (P::STAGE_TABLE_BYTES) R = NB == 1 && call.g.Br >= 128 ? 2 : 1;
  R = env_int("VQ_R", R);
  const int only_w = env_int("VQ_W", 0);
  // CTA shapes in order of preference: two 4-warp CTAs per SM (a CTA of the next kernel of the stream
  // can start beside one of this kernel) with as many column parts as fit, then one 8-warp CTA;
  // first with at least three pipeline stages, then with two.
  static const int kShapes[][2] = {{4, 4}, {4, 2}, {8, 4}, {8, 2}, {4, 1}, {8, 1}};
  // Three 4-warp CTAs per SM (12 consumer warps, two pipeline stages) where a CTA still gets eight
  // stages or more: measured on B200 at batch 1, 28672 x 8192 26.7 against 27.9 us with two CTAs per
  // SM, but 8192 x 8192 12.4 against 9.9 us (2.3 stages per CTA: all start-up and workspace reduction).
  if constexpr (NB == 1 && P::STAGE_TABLE_BYTES == 0) {
    int sms = 0;
    if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
    const long long stages = rows * static_cast<long long>(call.g.stride / P::CHUNK_BYTES) / (16 * R * 4);
    // (and where every CTA gets whole slabs: with fewer slabs than CTAs every output goes through the
    // workspace, 8192 x 28672: 34.1 against 30.3 us)
    if (stages >= 8LL * 3 * sms && rows / (16 * R) >= 3LL * sms && env_int("VQ_CTAS", 3) == 3 && (only_w == 0 || only_w == 4))
      for (int wk = 4; wk >= 2; wk /= 2) {
        const vq_status st = R == 2 ? launch<P, 1, 2, 4, 3>(call, chunks_per_block, s, wk, 2) : launch<P, 1, 1, 4, 3>(call, chunks_per_block, s, wk, 2);
        if (st != VQ_ERR_UNSUPPORTED) return st;
      }
  }
  // Batch 3-8: a stage's activations are as large as its indices, so one 8-warp CTA per SM with four
  // column parts and two stages comes first (28672 x 8192 at batch 8: 34.5 us against 39.5 us for two
  // 4-warp CTAs with two parts and 79 us for eight row tiles without column parts).
  // While two 4-warp CTAs with four parts still fit an SM with two stages (batch 3-4) they are faster
  // still (28672 x 8192 at batch 4: 28.8 against 32.0 us, 8192 x 8192 10.5 against 12.3).
  if constexpr (NB == 1 && P::STAGE_TABLE_BYTES == 0) {
    if (call.batch > 2 && (only_w == 0 || only_w == 4)) {
      const vq_status st = R == 2 ? launch<P, 1, 2, 4, 2>(call, chunks_per_block, s, 4, 2) : launch<P, 1, 1, 4, 2>(call, chunks_per_block, s, 4, 2);
      if (st != VQ_ERR_UNSUPPORTED) return st;
    }
    if (call.batch > 2 && (only_w == 0 || only_w == 8)) {
      const vq_status st = R == 2 ? launch<P, 1, 2, 8, 1>(call, chunks_per_block, s, 4, 2) : launch<P, 1, 1, 8, 1>(call, chunks_per_block, s, 4, 2);
      if (st != VQ_ERR_UNSUPPORTED) return st;
    }
  }
  // Batch 12-16: the same 8-warp shape with four column parts and two stages (28672 x 8192 at batch 16:
  // 53.2 us against 67.6 for two parts and three stages, 8192 x 28672 50.2 against 72.0; at batch 9 the
  // order below is the faster one, 43.4 against 47.6 us).
  if constexpr (NB == 2 && P::STAGE_TABLE_BYTES == 0) {
    if (call.batch >= 12 && (only_w == 0 || only_w == 8)) {
      const vq_status st = launch<P, 2, 1, 8, 1>(call, chunks_per_block, s, 4, 2);
      if (st != VQ_ERR_UNSUPPORTED) return st;
    }
  }
  for (int min_depth = 3; min_depth >= 2; --min_depth)
    for (const auto& sh : kShapes) {
      const int cw = sh[0], wk = sh[1];
      if (only_w && cw != only_w) continue;
      vq_status st;
      if (cw == 8) {
        st = (NB == 1 && R == 2) ? launch<P, NB, 2, 8, 1>(call, chunks_per_block, s, wk, min_depth)
                                 : launch<P, NB, 1, 8, 1>(call, chunks_per_block, s, wk, min_depth);
      } else {
        st = (NB == 1 && R == 2) ? launch<P, NB, 2, 4, 2>(call, chunks_per_block, s, wk, min_depth)
                                 : launch<P, NB, 1, 4, 2>(call, chunks_per_block, s, wk, min_depth);
      }
      if (st != VQ_ERR_UNSUPPORTED) return st;
    }
  return VQ_ERR_UNSUPPORTED;
}


// =============================================================================================
// Probes: the consumers' decode loops on a stage that stays in shared memory (no global traffic,
// no pipeline), and a plain read of a buffer.  bench.py turns their rates into the ceilings it
// prints beside the achieved numbers.
// =============================================================================================
template <class P, int NB, int R>
__global__ void __launch_bounds__(256, 1) probe_decode_kernel(int iters, int batch, long long* cycles, float* sink) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + (P::BASE_ALIGN - 1)) & ~static_cast<uint32_t>(P::BASE_ALIGN - 1);
  unsigned char* smem = smem_raw + (sbase - smem_u32(smem_raw));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, W = blockDim.x / 32;
  const int g = lane >> 2, t = lane & 3;
  // [stage table | per-warp tables | two stages of (index rows of every warp | activations)]: the passes
  // alternate between the stages as the pipeline of the real kernel does, so that no load of one pass
  // can be kept for the next
  const int tbl_words = (P::STAGE_TABLE_BYTES + W * R * P::TILE_TABLE_BYTES) / 4;
  const int idx_words = W * R * 16 * P::CHUNK_BYTES / 4;
  const int x_words = P::X_ROWS * batch * P::X_ROW_BYTES / 4;
  const int stage_words = idx_words + x_words;
  uint32_t* words = reinterpret_cast<uint32_t*>(smem);
  uint32_t seed = 1234567u + tid * 7919u + blockIdx.x;
  for (int i = tid; i < tbl_words + 2 * stage_words; i += blockDim.x) {
    seed = seed * 1664525u + 1013904223u;
    // small finite fp16 pairs for tables and activations, anything for indices
    const int j = i < tbl_words ? -1 : (i - tbl_words) % stage_words;
    words[i] = j < 0 ? (0x2C002C00u | (seed & 0x03FF03FFu)) : j < idx_words ? seed : (0x34003400u | (seed & 0x83FF83FFu));
  }
  __syncthreads();
  typename P::template State<NB, R> st;
  st.init(sbase + P::STAGE_TABLE_BYTES + warp * (R * P::TILE_TABLE_BYTES), lane);
  float total[R][NB][4];
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) total[r][nb][e] = 0.f;
  int xm[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) xm[nb] = min(nb * 8 + g, batch - 1);
  const unsigned char* idx = smem + tbl_words * 4 + (warp * R * 16 + g) * P::CHUNK_BYTES + t * P::LANE_BYTES;
  const unsigned char* xpart = smem + (tbl_words + idx_words) * 4;
  st.probe_fill(words + tbl_words + (tid * 41) % (idx_words - 64));
  const long long c0 = clock64();
  for (int it = 0; it < iters; ++it) {
    const int off = (it & 1) * stage_words * 4;
    st.compute(idx + off, xpart + off, xm, batch, sbase, lane, total);
    asm volatile("" ::: "memory");
  }
  const long long c1 = clock64();
  st.flush(total);
  float sum = 0.f;
#pragma unroll
  for (int r = 0; r < R; ++r)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) sum += total[r][nb][e];
  sink[blockIdx.x * blockDim.x + tid] = sum;
  if (tid == 0) cycles[blockIdx.x] = c1 - c0;
}

template <class P, int R>
vq_status run_probe(int warps, int batch, int iters, int sms, long long* d_cycles, float* d_sink, cudaStream_t s,
                    double* weights_per_stage) {
  auto kern = probe_decode_kernel<P, 1, R>;
  const size_t smem = P::BASE_ALIGN + P::STAGE_TABLE_BYTES + static_cast<size_t>(warps) * R * (P::TILE_TABLE_BYTES + 2 * 16 * P::CHUNK_BYTES) +
                      2 * static_cast<size_t>(P::X_ROWS) * batch * P::X_ROW_BYTES + 1024;
  if (smem > kSmemMax) return VQ_ERR_UNSUPPORTED;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemMax)) != cudaSuccess) return VQ_ERR_CUDA;
  kern<<<sms, warps * 32, smem, s>>>(iters, batch, d_cycles, d_sink);
  *weights_per_stage = static_cast<double>(warps) * R * 16 * P::CHUNK_COLS;
  return check_launch();
}

__global__ void __launch_bounds__(256) probe_read_kernel(const uint4* __restrict__ src, long long n16, uint32_t* __restrict__ out) {
  uint32_t acc = 0u;
  const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
  long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
  for (; i + 3 * stride < n16; i += 4 * stride) {   // four independent 128-bit loads in flight per thread
    const uint4 a = ldg128_stream(src + i), b = ldg128_stream(src + i + stride), c = ldg128_stream(src + i + 2 * stride),
                d = ldg128_stream(src + i + 3 * stride);
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
  }
  for (; i < n16; i += stride) {
    const uint4 a = ldg128_stream(src + i);
    acc ^= a.x ^ a.y ^ a.z ^ a.w;
  }
  if (acc == 0x9e3779b9u) out[0] = acc;   // (keeps the loads alive; practically never true)
}

}  // namespace

// Does the persistent kernel have a policy for this format (the launch may still decline a shape)?
bool stream_covers(const Geometry& g) {
  if (g.cb_int4) return false;
  if (g.b == 4 && g.Br >= 1 && g.stride % 128 == 0 && g.stride * 8 == static_cast<long long>(g.J) * 4) {
    if (g.d == 2) return g.Bc % 512 == 0;
    if (g.d == 1 && g.cb_int8) return g.Bc % 256 == 0;
  }
  return g.d == 2 && g.b == 6 && g.K % 256 == 0 && g.Bc % 128 == 0 && g.Br % 32 == 0 && g.stride * 8 == static_cast<long long>(g.J) * 6;
}

vq_status launch_gemm_stream(const StreamCall& call, cudaStream_t s) {
  const Geometry& g = call.g;
  if (call.n_seg < 1 || call.n_seg > kMaxSegments) return VQ_ERR_UNSUPPORTED;
  if (g.cb_int4) return VQ_ERR_UNSUPPORTED;
  const bool nb2 = call.batch > 8;
  if (g.b == 4 && g.Br >= 1 && g.stride % 128 == 0 && g.stride * 8 == static_cast<long long>(g.J) * 4) {
    if (g.d == 2) {
      if (g.Bc % 512) return VQ_ERR_UNSUPPORTED;
      const int cpb = g.Bc / 512;
      if (g.cb_int8) return nb2 ? launch_tiles<RowD2B4<true>, 2>(call, cpb, s) : launch_tiles<RowD2B4<true>, 1>(call, cpb, s);
      return nb2 ? launch_tiles<RowD2B4<false>, 2>(call, cpb, s) : launch_tiles<RowD2B4<false>, 1>(call, cpb, s);
    }
    if (g.d == 1 && g.cb_int8) {
      if (g.Bc % 256) return VQ_ERR_UNSUPPORTED;
      return nb2 ? launch_tiles<RowD1B4I8, 2>(call, g.Bc / 256, s) : launch_tiles<RowD1B4I8, 1>(call, g.Bc / 256, s);
    }
  }
  // 2-D 6-bit codebooks shared by blocks of at least 32 rows and 128 columns
  if (g.d == 2 && g.b == 6 && g.K % 256 == 0 && g.Bc % 128 == 0 && g.Br % 32 == 0 && g.stride * 8 == static_cast<long long>(g.J) * 6)
    return nb2 ? launch_tiles<BlkD2B6, 2>(call, 1, s) : launch_tiles<BlkD2B6, 1>(call, 1, s);
  return VQ_ERR_UNSUPPORTED;
}

// Uniform INT4 group-128 yard-stick through the same kernel; UNSUPPORTED if a row is not a whole
// number of 128-byte chunks.
vq_status launch_int4g128_stream(int N, int K, const uint8_t* q, const __half* scale, const __half* X, __half* Y, int batch,
                                 void* ws, size_t ws_bytes, cudaStream_t s) {
  if (K % 256) return VQ_ERR_UNSUPPORTED;
  StreamCall call = {};
  Geometry& g = call.g;
  g.N = N; g.K = K; g.d = 1; g.b = 4; g.Br = 1; g.Bc = 128;
  g.cb_int8 = 1; g.cb_int4 = 0; g.entries = 16; g.J = K; g.blocks_per_row = K / 256; g.stride = K / 2;
  call.n_seg = 1;
  call.idx[0] = q;
  call.cb[0] = nullptr;
  call.scale[0] = scale;
  call.Y[0] = Y;
  call.N[0] = N;
  call.X = X;
  call.batch = batch;
  call.ws = ws;
  call.ws_bytes = ws_bytes;
  return batch > 8 ? launch_tiles<RowInt4G128, 2>(call, 1, s) : launch_tiles<RowInt4G128, 1>(call, 1, s);
}

}  // namespace vq

using namespace vq;

// Decode-loop probe: `iters` passes of the inner loop of one policy over a stage that stays in shared
// memory, on every SM.  policy 0: 2-D 4-bit (two row tiles per warp), 1: 1-D 4-bit int8, 2: INT4 g128,
// 3: 2-D 6-bit shared codebooks (two row tiles per warp).  d_scratch: device memory of at least
// 8 * sms + 4 * sms * 32 * warps bytes.  Writes the average clocks of the loop and the weights one
// pass decodes per SM; synchronises the stream.
extern "C" vq_status vq_probe_decode_loop(int policy, int warps, int batch, int iters, void* d_scratch, size_t scratch_bytes,
                                          double* h_clocks, double* h_weights_per_pass, void* stream) {
  if (!d_scratch || !h_clocks || !h_weights_per_pass) return VQ_ERR_NULL;
  if (warps < 1 || warps > 8 || batch < 1 || batch > 8 || iters < 1) return VQ_ERR_SHAPE;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  const size_t need = static_cast<size_t>(sms) * 8 + static_cast<size_t>(sms) * 32 * warps * 4;
  if (scratch_bytes < need) return VQ_ERR_WORKSPACE;
  long long* d_cycles = static_cast<long long*>(d_scratch);
  float* d_sink = reinterpret_cast<float*>(static_cast<char*>(d_scratch) + static_cast<size_t>(sms) * 8);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  double wps = 0.0;
  vq_status st = VQ_ERR_UNSUPPORTED;
  if (policy == 0) st = run_probe<RowD2B4<true>, 2>(warps, batch, iters, sms, d_cycles, d_sink, s, &wps);
  else if (policy == 1) st = run_probe<RowD1B4I8, 1>(warps, batch, iters, sms, d_cycles, d_sink, s, &wps);
  else if (policy == 2) st = run_probe<RowInt4G128, 1>(warps, batch, iters, sms, d_cycles, d_sink, s, &wps);
  else if (policy == 3) st = run_probe<BlkD2B6, 2>(warps, batch, iters, sms, d_cycles, d_sink, s, &wps);
  if (st != VQ_OK) return st;
  long long h[1024];
  if (sms > 1024) return VQ_ERR_UNSUPPORTED;
  if (cudaStreamSynchronize(s) != cudaSuccess) return VQ_ERR_CUDA;
  if (cudaMemcpy(h, d_cycles, static_cast<size_t>(sms) * 8, cudaMemcpyDeviceToHost) != cudaSuccess) return VQ_ERR_CUDA;
  double sum = 0.0;
  for (int i = 0; i < sms; ++i) sum += static_cast<double>(h[i]);
  *h_clocks = sum / sms / iters;
  *h_weights_per_pass = wps;
  return VQ_OK;
}

// Read probe: every byte of d_buf once with streaming 128-bit loads (nothing is written unless a
// checksum happens to match a constant).  Enqueued on `stream`; the caller times it.
extern "C" vq_status vq_probe_read(const void* d_buf, size_t bytes, void* d_out4, void* stream) {
  if (!d_buf || !d_out4) return VQ_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(d_buf) & 15u) || bytes < 16) return VQ_ERR_ALIGN;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  probe_read_kernel<<<sms * 8, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<const uint4*>(d_buf),
                                                                            static_cast<long long>(bytes / 16),
                                                                            static_cast<uint32_t*>(d_out4));
  return check_launch();
}
