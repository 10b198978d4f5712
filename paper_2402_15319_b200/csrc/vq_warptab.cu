// warptab_kernel<EB, NB, QUAD, I4, NORM>: formats with SMALL codebook blocks (1, 2, 4, 8 rows, or any multiple of 16
// rows) and any index width the other tuned families do not take: 2-D indices of 1..8 bits, 1-D indices
// of 1..4 bits; fp16, scaled-int8 or int4 codebooks; block columns and K multiples of 64.  These are the
// remaining rows of the paper's configuration table (App. on VQ configurations: 1-D 2-bit 1x256 and
// 1x128, 2-D 2.5 bits per dimension on 2x256 and 4x256, 1-D 3-bit 32x256, 2-D 8-bit indices 256x256,
// 4-D 8-bit indices 128x256).
//
// Everything is expressed as PAIR look-ups: EB bits of the index stream select one 32-bit table word
// holding the two fp16 weights of two adjacent columns.  For d = 2 that is the codebook entry itself
// (EB = index_bits); for d = 1 two consecutive indices are looked up at once in the product table
// word[e] = (c[e mod k], c[e div k]) with EB = 2 * index_bits (the decode of Sec. 3.2 / App. A, two values
// per look-up as the paper's LUT instructions do).  Scales of int8 codebooks are folded into the table
// (w = fp16(scale * c), Sec. 3.1).  QUAD variant (d = 4, 8-bit indices): one stream byte selects four weights,
// two adjacent table words fetched by one 64-bit gather; everything else is the pair kernel at 4 stream
// bytes per lane and step.  I4 variant (INT4 codebooks, Sec. 4.2): tables hold the 4-bit entries as exact
// fp16 integers and every gathered pair is multiplied (one fp16x2 multiply, rounded once) by the fp16
// scale of its row and group of 128 columns, which gives fp16(scale * c), the value vq_decode_weights writes.
//
// Work: a CTA owns 16 output rows; its warps split K.  A warp walks its column range in steps of 64
// columns.  In a step, lane (g = lane / 4, t = lane % 4) takes 8 consecutive pairs (EB bytes of the
// stream, columns 16t .. 16t+15 of the step) of rows g and g + 8, gathers their table words and feeds
// them as A fragments to four m16n8k16 tensor-core steps whose B fragments are the activations of the
// same columns (batch rows 0..7, and 8..15 in a second accumulator when NB == 2); fp32 accumulation.
// Tables are private to the warp: one table per codebook block row that the 16 rows touch (16 / Br
// tables, one if Br >= 16), rebuilt whenever the walk enters a new block column.  The index stream
// reaches the lanes through warp-private shared-memory stages filled with 16-byte asynchronous copies,
// a chunk of 8 steps (32 * EB contiguous bytes of each of the 16 rows) at a time, kStages chunks deep:
// HBM sees row segments of 32..256 bytes instead of the 4 * EB bytes a step needs, and the copies of
// the next chunks run under the look-ups of this one.  Nothing in the loop synchronises beyond the warp.
// The warps' partial sums meet in shared memory in a fixed order (bit-identical results run to run).
#include <type_traits>

#include "vq_common.cuh"
#include "vq_device.cuh"

namespace vq {
namespace {

using namespace dev;

constexpr int kMaxWarps = 8;   // per CTA; four CTAs of that size fit an SM's registers at batch <= 8 (64 per thread), three above
constexpr int kChunkSteps = 8;   // steps per staged chunk of the index stream
constexpr int kStages = 2;
constexpr int kBuildGroup = 4;   // table words per lane whose loads are in flight together
// Bytes between the rows of a staged chunk: 32 * EB of indices + 16, an odd number of 16-byte units, so
// that the eight rows one look-up instruction reads start in different banks.
__host__ __device__ constexpr int stage_pitch(int eb) { return 32 * eb + 16; }
__host__ __device__ constexpr int stage_bytes(int eb) { return 16 * stage_pitch(eb); }
// Alignment of a warp's region: the size of one table of 2^tb words (tables start on multiples of their
// size), 16 at least.
__host__ __device__ constexpr int region_align(int tb) { return (4 << tb) < 16 ? 16 : (4 << tb); }

struct WarpTabArgs {
  // the layers of the call (same format and K, one activation tensor); tile0 = first 16-row tile of each
  const uint8_t* idx[kMaxSegments];
  const void* cb[kMaxSegments];
  const __half* scale[kMaxSegments];
  __half* Y[kMaxSegments];
  int N[kMaxSegments];
  int tile0[kMaxSegments];
  int n_seg;
  const __half* X;
  long long stride;
  int K, batch;
  int d, b, cb_int8;              // b: log2 of the entries of a block's codebook (a 4-D codebook counts as a 2-D one of 512)
  int cb_int4;                    // 4-bit entries (tables hold them as exact fp16 integers) + a scale per row and 128 columns
  int Br, br_shift;               // br_shift: log2(Br) when Br < 16
  int bsteps;                     // 64-column steps per codebook block (Bc / 64)
  int blocks_per_row;
  int steps_total, steps_per_warp;
  // block-wise normalisation (NORM kernels; single layer): 4-bit code per row and sub-row of 1 << norm_shift
  // columns, 16 binary16 scales per codebook block
  const uint8_t* norm_codes;
  const __half* norm_lut;
  int norm_shift, norm_row_bytes;
  int norm_off;                   // byte offset, in a warp's region, of its copy of the 16 scales of each of its tables
  int tbl_words;                  // words of one warp's tables
  int tbl_bytes;                  // bytes in front of the stages: tables (+ the normalisation scales), rounded up to 16
  int warp_bytes;                 // shared memory of one warp: tables, then kStages chunk stages
};

__device__ __forceinline__ uint32_t mul_f16x2(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void fence_acc4(float (&c)[4]) {
  asm volatile("" : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])::"memory");
}

// Shared-memory address of the table word of pair P of a lane's 8 pairs; (lo, hi) hold the lane's EB bytes
// from bit 0 of lo upwards.  The table starts on a multiple of its size, so base | entry * 4 == base + entry * 4
// and one logic operation masks the field and merges the base.
template <int EB, int P>
__device__ __forceinline__ uint32_t pair_address(uint32_t lo, uint32_t hi, uint32_t table) {
  constexpr int SH = P * EB;
  constexpr uint32_t M4 = ((1u << EB) - 1u) << 2;
  if constexpr (SH + EB <= 32) {
    if constexpr (SH >= 2) return ((lo >> (SH - 2)) & M4) | table;
    else return ((lo << (2 - SH)) & M4) | table;
  } else if constexpr (SH >= 32) {
    if constexpr (SH - 32 >= 2) return ((hi >> (SH - 34)) & M4) | table;
    else return ((hi << (34 - SH)) & M4) | table;
  } else {
    return (__funnelshift_r(lo, hi, SH - 2) & M4) | table;   // SH >= 25 here
  }
}

// The EB bytes of a lane at byte (base + IMM) + r of a staged row as (lo, hi), r = 0..3 being the lane's
// constant misalignment (sh = 8r): aligned 32-bit loads of the words that hold them.  two / three: whether
// the bytes reach into a second / third word (r + EB > 4 / > 8).  Every word read lies inside the row's
// slot: the last byte needed is the last one of the lane's field.
template <int EB, int IMM>
__device__ __forceinline__ void load_bits(uint32_t base, int sh, bool two, bool three, uint32_t& lo, uint32_t& hi) {
  uint32_t w0, w1 = 0, w2 = 0;
  asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(w0) : "r"(base), "n"(IMM));
  if (two) asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(w1) : "r"(base), "n"(IMM + 4));
  if constexpr (EB == 7) {
    if (three) asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(w2) : "r"(base), "n"(IMM + 8));
  }
  lo = __funnelshift_r(w0, w1, sh);
  hi = __funnelshift_r(w1, w2, sh);
}

template <int EB, int NB, bool QUAD, bool I4, bool NORM>
__global__ void __launch_bounds__(kMaxWarps * 32, NB == 1 ? 4 : 3) warptab_kernel(const WarpTabArgs a) {
  static_assert(!QUAD || EB == 4, "4-D entries: one 8-bit index per 4 columns = 4 stream bytes per lane and step");
  constexpr int TB = QUAD ? 9 : EB;   // log2 of the words of one table
  extern __shared__ __align__(16) uint8_t smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  // the layer this CTA's tile belongs to (selects, not indexed loads: the arguments stay in constant memory)
  int seg = 0;
#pragma unroll
  for (int i = 1; i < kMaxSegments; ++i)
    if (i < a.n_seg && static_cast<int>(blockIdx.x) >= a.tile0[i]) seg = i;
  auto pick = [&](const auto& arr) {
    auto v = arr[0];
#pragma unroll
    for (int i = 1; i < kMaxSegments; ++i)
      if (seg == i) v = arr[i];
    return v;
  };
  const uint8_t* const seg_idx = pick(a.idx);
  const void* const seg_cb = pick(a.cb);
  const __half* const seg_scale = pick(a.scale);
  __half* const seg_Y = pick(a.Y);
  const int seg_N = pick(a.N);
  const int row0 = (static_cast<int>(blockIdx.x) - pick(a.tile0)) * 16;
  const int rA = min(row0 + g, seg_N - 1), rB = min(row0 + g + 8, seg_N - 1);   // rows past N: computed, not written
  const int brow0 = a.Br >= 16 ? row0 / a.Br : row0 >> a.br_shift;
  const int block_rows = a.Br >= 16 ? seg_N / a.Br : seg_N >> a.br_shift;
  // warp regions start on a multiple of the table size (the host adds that much slack)
  uint8_t* mine = smem + ((0u - smem_u32(smem)) & static_cast<uint32_t>(region_align(TB) - 1)) + warp * a.warp_bytes;
  uint32_t* tbl = reinterpret_cast<uint32_t*>(mine);
  uint32_t tA = smem_u32(tbl), tB = tA;
  if (a.Br < 16) {
    tA += static_cast<uint32_t>((rA >> a.br_shift) - brow0) << (TB + 2);
    tB += static_cast<uint32_t>((rB >> a.br_shift) - brow0) << (TB + 2);
  }
  constexpr int PITCH = stage_pitch(EB);
  const uint32_t stage_s = smem_u32(mine) + a.tbl_bytes;

  float acc[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[nb][c] = 0.f;

  // One table word per (table j, pair entry e): the two fp16 weights that the EB index bits stand for.
  // Offsets into the codebook fit 32 bits (checked on the host).  The loads of kBuildGroup words per lane are
  // issued together and converted afterwards, so that a build waits for memory once per group, not once
  // per word.  (Asking L2 for the next block columns' entries at each build, prefetch.global.L2, was
  // measured and is slower on every shape: 72 against 68 us on 28672 x 8192, 22 against 11 us on 4096 x 4096
  // with 8-bit indices.)
  const uint32_t cb_shift = static_cast<uint32_t>(a.b);   // entries per block = 1 << b
  auto build = [&](int col_blk) {
#pragma unroll 1
    for (int i0 = lane; i0 < a.tbl_words; i0 += 32 * kBuildGroup) {
      uint32_t raw[kBuildGroup];
      __half sc[kBuildGroup];
#pragma unroll
      for (int k = 0; k < kBuildGroup; ++k) {
        const int i = i0 + 32 * k;
        raw[k] = 0u;
        sc[k] = __ushort_as_half(0);
        if (i - lane < a.tbl_words && i < a.tbl_words) {   // (the first test is the same for the whole warp: unused slots are jumped over)
          const uint32_t e = static_cast<uint32_t>(i) & ((1u << TB) - 1u);
          const uint32_t blk = static_cast<uint32_t>(min(brow0 + (i >> TB), block_rows - 1)) * static_cast<uint32_t>(a.blocks_per_row) +
                               static_cast<uint32_t>(col_blk);
          if (!I4 && a.cb_int8) {
            sc[k] = __ldg(seg_scale + blk);
          }
          if (I4) {   // two 4-bit values per byte, low nibble first
            const uint8_t* c = static_cast<const uint8_t*>(seg_cb);
            if (a.d == 2) {
              raw[k] = __ldg(c + (blk << cb_shift) + e);   // one byte = the entry's two values
            } else {
              const uint32_t v0 = (blk << cb_shift) + (e & ((1u << cb_shift) - 1u)), v1 = (blk << cb_shift) + (e >> cb_shift);
              const uint32_t n0 = (__ldg(c + (v0 >> 1)) >> (4 * (v0 & 1u))) & 15u, n1 = (__ldg(c + (v1 >> 1)) >> (4 * (v1 & 1u))) & 15u;
              raw[k] = n0 | (n1 << 4);
            }
          } else if (a.d == 2) {
            const uint32_t at = (blk << cb_shift) + e;   // in entries of two values
            if (a.cb_int8) {
              const uint16_t* c = static_cast<const uint16_t*>(seg_cb) + at;
              raw[k] = __ldg(c);
            } else {
              const uint32_t* c = static_cast<const uint32_t*>(seg_cb) + at;
              raw[k] = __ldg(c);
            }
          } else {   // two 1-D entries: the first column's in the low half
            const uint32_t at0 = (blk << cb_shift) + (e & ((1u << cb_shift) - 1u)), at1 = (blk << cb_shift) + (e >> cb_shift);
            if (a.cb_int8) {
              const uint8_t* c = static_cast<const uint8_t*>(seg_cb);
              raw[k] = static_cast<uint32_t>(__ldg(c + at0)) | (static_cast<uint32_t>(__ldg(c + at1)) << 8);
            } else {
              const uint16_t* c = static_cast<const uint16_t*>(seg_cb);
              raw[k] = static_cast<uint32_t>(__ldg(c + at0)) | (static_cast<uint32_t>(__ldg(c + at1)) << 16);
            }
          }
        }
      }
#pragma unroll
      for (int k = 0; k < kBuildGroup; ++k) {
        const int i = i0 + 32 * k;
        if (i - lane < a.tbl_words && i < a.tbl_words) {
          uint32_t word = raw[k];
          if (I4) {   // signed nibbles as fp16 integers (exact); the row-group scale multiplies after the look-up
            const int lo4 = static_cast<int>(raw[k] << 28) >> 28, hi4 = static_cast<int>(raw[k] << 24) >> 28;
            const __half2 hv = __floats2half2_rn(static_cast<float>(lo4), static_cast<float>(hi4));
            word = *reinterpret_cast<const uint32_t*>(&hv);
          } else if (a.cb_int8) {   // exact products of the block scale and the 8-bit entries, one rounding each
            const float f = __half2float(sc[k]);
            const __half2 hv = __floats2half2_rn(f * static_cast<float>(static_cast<int8_t>(raw[k] & 0xffu)),
                                                 f * static_cast<float>(static_cast<int8_t>((raw[k] >> 8) & 0xffu)));
            word = *reinterpret_cast<const uint32_t*>(&hv);
          }
          tbl[i] = word;
        }
      }
    }
    if constexpr (NORM) {   // the 16 scales of each table's codebook block
      __half* nl = reinterpret_cast<__half*>(mine + a.norm_off);
      for (int i = lane; i < (a.tbl_words >> TB) * 16; i += 32) {
        const uint32_t blk = static_cast<uint32_t>(min(brow0 + (i >> 4), block_rows - 1)) * static_cast<uint32_t>(a.blocks_per_row) +
                             static_cast<uint32_t>(col_blk);
        nl[i] = __ldg(a.norm_lut + blk * 16 + (i & 15));
      }
    }
  };

  // Chunk c of this warp (steps s_begin + 8c ..) into stage c % kStages: 2 * EB pieces of 16 bytes per row,
  // EB pieces per lane.  Pieces that start past the row pitch (last chunk of a row) are left out; the
  // steps that would read them lie past K and are never computed.  One commit per call, even if empty.
  const int s_begin = warp * a.steps_per_warp;
  const int s_end = min(a.steps_total, s_begin + a.steps_per_warp);
  const int n_chunks = (s_end - s_begin + kChunkSteps - 1) / kChunkSteps;
  // lane = 2 * row + y copies pieces y, y + 2, y + 4, ... of its row: a lane pair moves 32 contiguous bytes
  const int fr = lane >> 1, fy = lane & 1;
  const int off0 = s_begin * (4 * EB) + fy * 16;   // byte offset inside the row of this lane's first piece of chunk 0
  const uint8_t* src0 = seg_idx + min(row0 + fr, seg_N - 1) * a.stride + off0;
  const uint32_t dst0 = stage_s + fr * PITCH + fy * 16;
  const int row_bytes = static_cast<int>(a.stride);
  auto fetch = [&](int c) {
    if (c < n_chunks) {
      const int adv = c * (kChunkSteps * 4 * EB);
      const uint32_t dst = dst0 + (c % kStages) * stage_bytes(EB);
#pragma unroll
      for (int q = 0; q < EB; ++q)
        if (off0 + adv + 32 * q < row_bytes) cp_async16(dst + 32 * q, src0 + adv + 32 * q);
    }
    cp_async_commit();
  };

#pragma unroll
  for (int c = 0; c < kStages - 1; ++c) fetch(c);
  // the first tables, while the first chunk is on its way
  int until_rebuild;   // steps left in the current codebook block column
  {
    const int col_blk = s_begin / a.bsteps;
    until_rebuild = a.bsteps - (s_begin - col_blk * a.bsteps);
    build(col_blk);
    __syncwarp();
    fence_value(tA);
    fence_value(tB);
  }

  // Activations of one step: columns 16t .. 16t+15 of batch row g (+ 8 for the second accumulator).  Lanes
  // whose batch row does not exist read the last row instead: their accumulator columns are never written.
  const __half* xp[NB];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb)
    xp[nb] = a.X + static_cast<long long>(min(nb * 8 + g, a.batch - 1)) * a.K + s_begin * 64 + t * 16;
  uint4 xn[NB][2];   // the next step's activations, fetched one step ahead
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    xn[nb][0] = ldg128_nc(xp[nb]);
    xn[nb][1] = ldg128_nc(xp[nb] + 8);
  }

  // normalisation: code rows of rows g and g + 8, and where the scales of their tables' blocks are staged
  const uint8_t* const ncA = a.norm_codes + static_cast<long long>(rA) * a.norm_row_bytes;
  const uint8_t* const ncB = a.norm_codes + static_cast<long long>(rB) * a.norm_row_bytes;
  const uint32_t nlA = smem_u32(mine) + a.norm_off + (((tA - smem_u32(tbl)) >> (TB + 2)) << 5);
  const uint32_t nlB = smem_u32(mine) + a.norm_off + (((tB - smem_u32(tbl)) >> (TB + 2)) << 5);
  // INT4 codebooks: the scales of rows g and g + 8, one per group of 128 columns
  const __half* const scA = seg_scale + static_cast<long long>(rA) * (a.K / 128);
  const __half* const scB = seg_scale + static_cast<long long>(rB) * (a.K / 128);
  // a lane's EB bytes of a step start t * EB bytes after the step's: the same misalignment in every step
  const int bit_sh = ((t * EB) & 3) * 8;
  const bool two_words = ((t * EB) & 3) + EB > 4, three_words = ((t * EB) & 3) + EB > 8;
  static_assert(kChunkSteps == 8, "the chunk loop below is written out for 8 steps");
  for (int c = 0; c < n_chunks; ++c) {
    cp_async_wait<kStages - 2>();   // chunk c has landed (this lane's pieces; the warp barrier covers the others')
    __syncwarp();                   // ... and every lane is done reading the stage that chunk c + kStages - 1 overwrites
    fetch(c + kStages - 1);
    // this lane's first word of step 0 in rows g and g + 8 of the stage
    const uint32_t rowA_s = stage_s + (c % kStages) * stage_bytes(EB) + g * PITCH + ((t * EB) & ~3);
    const uint32_t rowB_s = rowA_s + 8 * PITCH;
    const int sc0 = s_begin + c * kChunkSteps;
    const int nst = min(kChunkSteps, s_end - sc0);
    auto step = [&](auto uc) {
      constexpr int UU = decltype(uc)::value;
      const int s = sc0 + UU;
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
      uint4 x[NB][2];
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        x[nb][0] = xn[nb][0];
        x[nb][1] = xn[nb][1];
        if (s + 1 < s_end) xp[nb] += 64;   // (the warp's last step is read twice)
        xn[nb][0] = ldg128_nc(xp[nb]);
        xn[nb][1] = ldg128_nc(xp[nb] + 8);
      }
      uint32_t loA, hiA, loB, hiB;
      load_bits<EB, UU * 4 * EB>(rowA_s, bit_sh, two_words, three_words, loA, hiA);
      load_bits<EB, UU * 4 * EB>(rowB_s, bit_sh, two_words, three_words, loB, hiB);
      uint32_t wa[8], wb[8];
      if constexpr (QUAD) {   // one byte selects four weights: a 64-bit gather fills pairs 2q and 2q + 1
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint2 va = lds64((((loA >> (8 * q)) & 0xffu) << 3) | tA);
          const uint2 vb = lds64((((loB >> (8 * q)) & 0xffu) << 3) | tB);
          wa[2 * q] = va.x; wa[2 * q + 1] = va.y;
          wb[2 * q] = vb.x; wb[2 * q + 1] = vb.y;
        }
      } else {
#define VQ_WT_PAIR(P)                                    \
  wa[P] = lds32(pair_address<EB, P>(loA, hiA, tA));     \
  wb[P] = lds32(pair_address<EB, P>(loB, hiB, tB));
        VQ_WT_PAIR(0) VQ_WT_PAIR(1) VQ_WT_PAIR(2) VQ_WT_PAIR(3)
        VQ_WT_PAIR(4) VQ_WT_PAIR(5) VQ_WT_PAIR(6) VQ_WT_PAIR(7)
#undef VQ_WT_PAIR
      }
      if constexpr (NORM) {   // every pair times the scale its sub-row's 4-bit code selects (a lane's 16 columns lie in one sub-row)
        const int j = (s * 64 + t * 16) >> a.norm_shift;
        const uint32_t cA = (static_cast<uint32_t>(__ldg(ncA + (j >> 1))) >> (4 * (j & 1))) & 15u;
        const uint32_t cB = (static_cast<uint32_t>(__ldg(ncB + (j >> 1))) >> (4 * (j & 1))) & 15u;
        uint32_t fA, fB;
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(fA) : "r"(nlA + 2 * cA) : "memory");
        asm volatile("ld.shared.u16 %0, [%1];" : "=r"(fB) : "r"(nlB + 2 * cB) : "memory");
        fA |= fA << 16;
        fB |= fB << 16;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          wa[q] = mul_f16x2(wa[q], fA);
          wb[q] = mul_f16x2(wb[q], fB);
        }
      }
      if constexpr (I4) {   // w = fp16(scale of the row's group of 128 columns * c): the value vq_decode_weights writes
        const int grp = s >> 1;   // a step's 64 columns lie inside one group
        const __half2 sA = __half2half2(__ldg(scA + grp)), sB = __half2half2(__ldg(scB + grp));
        const uint32_t uA = *reinterpret_cast<const uint32_t*>(&sA), uB = *reinterpret_cast<const uint32_t*>(&sB);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          wa[q] = mul_f16x2(wa[q], uA);
          wb[q] = mul_f16x2(wb[q], uB);
        }
      }
#pragma unroll
      for (int nb = 0; nb < NB; ++nb) {
        mma16816(acc[nb], wa[0], wb[0], wa[1], wb[1], x[nb][0].x, x[nb][0].y);
        mma16816(acc[nb], wa[2], wb[2], wa[3], wb[3], x[nb][0].z, x[nb][0].w);
        mma16816(acc[nb], wa[4], wb[4], wa[5], wb[5], x[nb][1].x, x[nb][1].y);
        mma16816(acc[nb], wa[6], wb[6], wa[7], wb[7], x[nb][1].z, x[nb][1].w);
      }
    };
    // the chunk's steps, unrolled: every shared-memory offset of a step is then an immediate
    if (0 < nst) step(std::integral_constant<int, 0>{});
    if (1 < nst) step(std::integral_constant<int, 1>{});
    if (2 < nst) step(std::integral_constant<int, 2>{});
    if (3 < nst) step(std::integral_constant<int, 3>{});
    if (4 < nst) step(std::integral_constant<int, 4>{});
    if (5 < nst) step(std::integral_constant<int, 5>{});
    if (6 < nst) step(std::integral_constant<int, 6>{});
    if (7 < nst) step(std::integral_constant<int, 7>{});
  }
  cp_async_wait<0>();
  __syncthreads();   // the reduction buffer lies over the warps' tables and stages

  // K parts of the warps meet in shared memory; thread i then owns output (batch row i / 16, row i % 16).
  float* red = reinterpret_cast<float*>(smem);   // over the warps' tables and stages, which are no longer needed
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
    if (m < a.batch && row0 + r < seg_N) seg_Y[static_cast<long long>(m) * seg_N + row0 + r] = __float2half_rn(sum);
  }
}

// 4-D entries selected by 8-bit indices: one look-up returns four weights (two table words).
bool quad_format(const Geometry& g) { return g.d == 4 && g.b == 8; }

// Stream bits per pair of columns: what a lane consumes is 8 of them = that many bytes per step.
int pair_bits(const Geometry& g) {
  if (g.d == 2) return g.b;
  if (g.d == 1 && g.b <= 4) return 2 * g.b;
  if (quad_format(g)) return 4;
  return 0;
}

// log2 of the 32-bit words of one table.
int table_bits(const Geometry& g) { return quad_format(g) ? 9 : pair_bits(g); }

int tables_per_tile(const Geometry& g) { return g.Br >= 16 ? 1 : 16 / g.Br; }

constexpr size_t kSmemLimit = 100 * 1024;   // dynamic shared memory a CTA may ask for (fewer warps per CTA beyond it)
constexpr size_t kSmemPerSm = 228 * 1024;   // shared memory of an SM; every resident CTA also costs 1 KB of it

// Picks the K split, finishes the arguments and launches.  The dynamic shared-memory limit is raised and the
// kernel's register count read once per device and instantiation.
template <int EB, int NB, bool QUAD, bool I4, bool NORM>
vq_status launch_one(WarpTabArgs a, long long tiles, int sms, cudaStream_t s) {
  constexpr int TB = QUAD ? 9 : EB;
  static int regs_of[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  int regs = __atomic_load_n(&regs_of[dev], __ATOMIC_ACQUIRE);
  if (!regs) {
    cudaFuncAttributes fa;
    if (cudaFuncSetAttribute(warptab_kernel<EB, NB, QUAD, I4, NORM>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemLimit)) !=
            cudaSuccess ||
        cudaFuncGetAttributes(&fa, warptab_kernel<EB, NB, QUAD, I4, NORM>) != cudaSuccess || fa.numRegs < 1)
      return VQ_ERR_CUDA;
    regs = fa.numRegs;
    __atomic_store_n(&regs_of[dev], regs, __ATOMIC_RELEASE);
  }
  // CTAs of w warps that one SM holds: registers (allocated per warp in units of 256), shared memory, 32 CTAs
  const int warps_by_regs = 65536 / ((regs * 32 + 255) / 256 * 256);
  auto resident = [&](int w) {
    long long c = warps_by_regs / w;
    c = c < 32 ? c : 32;
    const long long by_smem = static_cast<long long>(kSmemPerSm / (static_cast<size_t>(w) * a.warp_bytes + region_align(TB) + 1024));
    return c < by_smem ? c : by_smem;
  };
  // K split: the most warps per CTA (at most kMaxWarps, at most one per chunk of the row) with which every
  // CTA of the grid is resident at once.  A grid one CTA larger than that costs a second pass over the
  // device, which weighs more than the longer walk of fewer, longer-running warps.
  const int chunks_total = (a.steps_total + kChunkSteps - 1) / kChunkSteps;
  int wk = kMaxWarps < chunks_total ? kMaxWarps : chunks_total;
  while (wk > 1 && (static_cast<size_t>(wk) * a.warp_bytes + region_align(TB) > kSmemLimit || tiles > resident(wk) * sms)) --wk;
  a.steps_per_warp = ((a.steps_total + wk - 1) / wk + kChunkSteps - 1) / kChunkSteps * kChunkSteps;   // whole chunks
  wk = (a.steps_total + a.steps_per_warp - 1) / a.steps_per_warp;   // no warp without work
  const size_t smem_bytes = static_cast<size_t>(wk) * a.warp_bytes + region_align(TB);
  if (smem_bytes > kSmemLimit) return VQ_ERR_UNSUPPORTED;
  // A plain launch, in stream order.  (With programmatic dependent launch the next launch's CTAs take the
  // SM slots this grid leaves free and stay where they land: two such layers back to back then run with
  // 3 CTAs on some SMs and 1 on others; measured 31.5 against 23.2 us on 4096 x 14336.)
  warptab_kernel<EB, NB, QUAD, I4, NORM><<<static_cast<unsigned>(tiles), static_cast<unsigned>(wk) * 32u, smem_bytes, s>>>(a);
  return check_launch();
}

template <int EB, bool QUAD = false>
vq_status launch_eb(const WarpTabArgs& a, int nb, long long tiles, int sms, cudaStream_t s) {
  if (a.norm_codes)   // (normalisation with INT4 codebooks stays in the format-generic kernel)
    return nb == 1 ? launch_one<EB, 1, QUAD, false, true>(a, tiles, sms, s) : launch_one<EB, 2, QUAD, false, true>(a, tiles, sms, s);
  if (a.cb_int4) return nb == 1 ? launch_one<EB, 1, QUAD, true, false>(a, tiles, sms, s) : launch_one<EB, 2, QUAD, true, false>(a, tiles, sms, s);
  return nb == 1 ? launch_one<EB, 1, QUAD, false, false>(a, tiles, sms, s) : launch_one<EB, 2, QUAD, false, false>(a, tiles, sms, s);
}

}  // namespace

bool warptab_covers(const Geometry& g) {
  const int eb = pair_bits(g);
  if (eb < 1 || eb > 8) return false;
  if (g.K % 64 || g.Bc % 64) return false;
  if (!(g.Br == 1 || g.Br == 2 || g.Br == 4 || g.Br == 8 || g.Br % 16 == 0)) return false;
  if (g.stride >= (1LL << 30)) return false;   // byte offsets inside a row are 32-bit in the kernel
  return (tables_per_tile(g) << table_bits(g)) <= 1024;
}

namespace {
// norm_codes == nullptr: no normalisation.  With it: one layer, sub-rows of a power of two of at least 16 columns
// (a lane's 16 columns of a step then lie inside one sub-row), fp16 or int8 codebooks.
vq_status launch_impl(const StreamCall& call, const void* norm_codes, const void* norm_lut, int norm_block_cols, cudaStream_t s) {
  const Geometry& g = call.g;
  if (!warptab_covers(g) || call.n_seg < 1 || call.n_seg > kMaxSegments) return VQ_ERR_UNSUPPORTED;
  int norm_shift = -1;
  if (norm_codes) {
    for (int sh = 4; sh < 31; ++sh)
      if ((1 << sh) == norm_block_cols) norm_shift = sh;
    if (norm_shift < 0 || g.cb_int4 || call.n_seg != 1) return VQ_ERR_UNSUPPORTED;
  }
  const int eb = pair_bits(g);
  const int nb = call.batch <= 8 ? 1 : 2;
  WarpTabArgs a = {};
  long long tiles = 0;
  for (int i = 0; i < call.n_seg; ++i) {
    if (call.N[i] <= 0 || call.N[i] % g.Br) return VQ_ERR_UNSUPPORTED;
    // the kernel addresses codebook entries with 32-bit offsets
    if (static_cast<long long>(call.N[i] / g.Br) * g.blocks_per_row * g.entries * g.d >= (1LL << 31)) return VQ_ERR_UNSUPPORTED;
    a.idx[i] = call.idx[i];
    a.cb[i] = call.cb[i];
    a.scale[i] = call.scale[i];
    a.Y[i] = call.Y[i];
    a.N[i] = call.N[i];
    a.tile0[i] = static_cast<int>(tiles);
    tiles += (call.N[i] + 15) / 16;
  }
  if (tiles >= (1LL << 31)) return VQ_ERR_UNSUPPORTED;
  a.n_seg = call.n_seg;
  a.X = call.X;
  a.stride = g.stride;
  a.K = g.K;
  a.batch = call.batch;
  // (a 4-D codebook of 256 entries lies in memory like a 2-D one of 512: the table build treats it as such)
  a.d = quad_format(g) ? 2 : g.d;
  a.b = quad_format(g) ? 9 : g.b;
  a.cb_int8 = g.cb_int8;
  a.cb_int4 = g.cb_int4;
  a.Br = g.Br;
  a.br_shift = g.Br == 1 ? 0 : g.Br == 2 ? 1 : g.Br == 4 ? 2 : 3;
  a.bsteps = g.Bc / 64;
  a.blocks_per_row = g.blocks_per_row;
  a.steps_total = g.K / 64;
  a.tbl_words = tables_per_tile(g) << table_bits(g);
  // per warp: tables + chunk stages; the reduction buffer (nb * 512 bytes per warp) reuses that space
  a.tbl_bytes = (a.tbl_words * 4 + 15) / 16 * 16;
  if (norm_codes) {
    a.norm_codes = static_cast<const uint8_t*>(norm_codes);
    a.norm_lut = static_cast<const __half*>(norm_lut);
    a.norm_shift = norm_shift;
    a.norm_row_bytes = (g.K / norm_block_cols + 1) / 2;
    a.norm_off = a.tbl_bytes;
    a.tbl_bytes += tables_per_tile(g) * 32;   // 16 binary16 scales per table
  }
  const int tbl_align = region_align(table_bits(g));
  a.warp_bytes = (a.tbl_bytes + kStages * stage_bytes(eb) + tbl_align - 1) / tbl_align * tbl_align;
  int sms = 0;
  if (device_sms(&sms) != VQ_OK) return VQ_ERR_CUDA;
  switch (eb) {
    case 1: return launch_eb<1>(a, nb, tiles, sms, s);
    case 2: return launch_eb<2>(a, nb, tiles, sms, s);
    case 3: return launch_eb<3>(a, nb, tiles, sms, s);
    case 4: return quad_format(g) ? launch_eb<4, true>(a, nb, tiles, sms, s) : launch_eb<4>(a, nb, tiles, sms, s);
    case 5: return launch_eb<5>(a, nb, tiles, sms, s);
    case 6: return launch_eb<6>(a, nb, tiles, sms, s);
    case 7: return launch_eb<7>(a, nb, tiles, sms, s);
    default: return launch_eb<8>(a, nb, tiles, sms, s);
  }
}
}  // namespace

vq_status launch_gemm_warptab_group(const StreamCall& call, cudaStream_t s) { return launch_impl(call, nullptr, nullptr, 0, s); }

vq_status launch_gemm_warptab_norm(const Geometry& g, const LayerPtrs& p, const void* norm_codes, const void* norm_lut,
                                   int norm_block_cols, const __half* X, __half* Y, int batch, cudaStream_t s) {
  if (!norm_codes || !norm_lut) return VQ_ERR_UNSUPPORTED;
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
  return launch_impl(call, norm_codes, norm_lut, norm_block_cols, s);
}

vq_status launch_gemm_warptab(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
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
  return launch_gemm_warptab_group(call, s);
}

}  // namespace vq
