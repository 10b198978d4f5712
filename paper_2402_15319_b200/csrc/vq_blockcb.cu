// Tuned skinny-GEMM kernels for formats whose codebook is shared by a tall block of rows
// (block_rows a multiple of the CTA's rows): the 2-D 6-bit and 4-D 8-bit fp16-codebook families.
//
// Per CTA: a tile of CTA_ROWS x CTA_COLS weights.  Each warp owns 32 rows x 256 columns:
// lane (g = lane/4, t = lane%4) streams its own 64 columns of rows g, g+8, g+16, g+24 straight
// from the packed index stream into registers, looks every index up in a lane-private copy of
// its block's codebook in shared memory (bank = lane, so the gather is conflict-free for any
// index pattern) and feeds the fp16 pairs, untouched, into mma.sync m16n8k16 as the A fragment.
// The activations of the lane's 64 columns sit in registers as the B fragment (batch row = g),
// accumulation is fp32 in the tensor core.  The K dimension is split over the CTAs of a thread
// block cluster; their partial sums are combined in a fixed order through distributed shared
// memory, rounded once to fp16 and stored.  Paper: Sec. 3.2 (packed indices -> LUT -> mat-vec),
// App. A (Q is a look-up of C); the tiling, the replication and the reduction are this library's.
#include <cooperative_groups.h>

#include <cstdlib>
#include <type_traits>
#include <utility>

#include "vq_common.cuh"

namespace cg = cooperative_groups;

#ifdef VQ_TUNING
__device__ unsigned long long* g_vq_trace = nullptr;
extern "C" void vq_debug_set_trace(unsigned long long* p) { cudaMemcpyToSymbol(g_vq_trace, &p, sizeof(p)); }
#define VQ_TRACE(slot)                                                                            \
  do {                                                                                            \
    if (g_vq_trace && threadIdx.x == 0) {                                                         \
      unsigned long long t_;                                                                      \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                      \
      g_vq_trace[(static_cast<size_t>(blockIdx.y) * gridDim.x + blockIdx.x) * 8 + (slot)] = t_;   \
    }                                                                                             \
  } while (0)
#else
#define VQ_TRACE(slot) do {} while (0)
#endif

namespace vq {
namespace {

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

// 24-byte pieces: the three 8-byte loads of a lane share sectors, so let L1 keep the line.
__device__ __forceinline__ uint2 ldg64_stream(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.v2.b32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}

// Cluster barrier split into arrive / wait so that independent work overlaps the wait.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_acquire() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// fp32 store into the shared memory of CTA `rank` of this cluster (same offset as `local_addr`).
__device__ __forceinline__ void st_cluster_f32(uint32_t local_addr, int rank, float v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

__device__ __forceinline__ uint4 ldg128_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// ---- format policies -----------------------------------------------------------------------
// LANE_WORDS : 32-bit words of index stream a lane owns per row (64 columns)
// ENTRY_BYTES: bytes of one codebook entry; TABLE_BYTES: one lane-private table set
template <int D, int B>
struct Policy;

// 2-D, 6-bit indices: 64 columns = 32 indices = 24 bytes per lane and row
template <>
struct Policy<2, 6> {
  static constexpr int LANE_WORDS = 6, ENTRY_BYTES = 4, ENTRIES = 64;
  static constexpr int WARPS = 4, TASKS = 1, SLICES = 1;     // CTA = 128 rows x 256 cols
  static constexpr int TABLE_BYTES = ENTRIES * 128;          // [entry][lane] words
  static constexpr uint32_t MASK = 0x1F80u;                  // 6 index bits at byte offset * 128

  // byte offset (entry * 128) of index I (0..31) of a lane's 6 words
  template <int I>
  static __device__ __forceinline__ uint32_t entry_off(const uint32_t (&w)[LANE_WORDS]) {
    constexpr int p = 6 * I;
    if constexpr (p < 7) {
      return (w[0] << (7 - p)) & MASK;
    } else {
      constexpr int q = p - 7, wi = q >> 5, s = q & 31;
      if constexpr (s == 0) return w[wi] & MASK;
      else if constexpr (s + 13 > 32) return __funnelshift_r(w[wi], w[wi + 1], s) & MASK;
      else return (w[wi] >> s) & MASK;
    }
  }
};

// 4-D, 8-bit indices: 64 columns = 16 indices = 16 bytes per lane and row
template <>
struct Policy<4, 8> {
  static constexpr int LANE_WORDS = 4, ENTRY_BYTES = 8, ENTRIES = 256;
  static constexpr int WARPS = 8, TASKS = 2, SLICES = 2;     // CTA = 256 rows x 512 cols
  static constexpr int TABLE_BYTES = ENTRIES * 128;          // [entry][lane%16] 8-byte entries
  static constexpr uint32_t MASK = 0x7F80u;

  template <int I>
  static __device__ __forceinline__ uint32_t entry_off(const uint32_t (&w)[LANE_WORDS]) {
    constexpr int wi = I >> 2, p = 8 * (I & 3);
    if constexpr (p < 7) return (w[wi] << (7 - p)) & MASK;
    else return (w[wi] >> (p - 7)) & MASK;
  }
};

// bytes of the compact codebook staging area behind the replicated tables
template <int D, int B>
constexpr int kCompactBytes = Policy<D, B>::ENTRIES * 8;

template <int D, int B>
struct Tile {
  using P = Policy<D, B>;
  static constexpr int ROWS_PER_TASK = 32;
  static constexpr int CTA_ROWS = ROWS_PER_TASK * P::WARPS * P::TASKS / P::SLICES;
  static constexpr int CTA_COLS = 256 * P::SLICES;
  static constexpr int THREADS = 32 * P::WARPS;
  // resident CTAs per SM the register budget is tuned for (NB = 1 / NB = 2)
  static constexpr int min_ctas(int nb) { return D == 2 ? (nb == 1 ? 6 : 4) : (nb == 1 ? 2 : 1); }
};

// Gather the A fragments of NSTEPS mma steps (each step = 4 columns per lane) of one 16-row tile:
// wa / wb are the lane's index words of rows g and g+8.
template <int D, int B, int STEP0, int NSTEPS>
__device__ __forceinline__ void gather_steps(uint32_t (&a)[NSTEPS][4], const uint32_t (&wa)[Policy<D, B>::LANE_WORDS],
                                             const uint32_t (&wb)[Policy<D, B>::LANE_WORDS], uint32_t tbl) {
  using P = Policy<D, B>;
  if constexpr (D == 2) {
    [&]<int... S>(std::integer_sequence<int, S...>) {
      ((a[S][0] = lds32(tbl + P::template entry_off<2 * (STEP0 + S)>(wa)),
        a[S][1] = lds32(tbl + P::template entry_off<2 * (STEP0 + S)>(wb)),
        a[S][2] = lds32(tbl + P::template entry_off<2 * (STEP0 + S) + 1>(wa)),
        a[S][3] = lds32(tbl + P::template entry_off<2 * (STEP0 + S) + 1>(wb))), ...);
    }(std::make_integer_sequence<int, NSTEPS>{});
  } else {
    [&]<int... S>(std::integer_sequence<int, S...>) {
      (([&] {
         const uint2 u = lds64(tbl + P::template entry_off<STEP0 + S>(wa));
         const uint2 v = lds64(tbl + P::template entry_off<STEP0 + S>(wb));
         a[S][0] = u.x; a[S][2] = u.y; a[S][1] = v.x; a[S][3] = v.y;
       }()), ...);
    }(std::make_integer_sequence<int, NSTEPS>{});
  }
}

// One task = two 16-row tiles x 64 columns per lane.  The tiles' accumulator chains are
// independent, so their look-ups are issued together and their mmas alternate.
template <int D, int B, int NB, int STEP0, int NSTEPS>
__device__ __forceinline__ void task_steps(float (&acc)[2][NB][4], const uint32_t (&w)[4][Policy<D, B>::LANE_WORDS],
                                           const uint32_t (&xr)[NB][32], uint32_t tbl) {
  uint32_t a0[NSTEPS][4], a1[NSTEPS][4];
  gather_steps<D, B, STEP0, NSTEPS>(a0, w[0], w[1], tbl);
  gather_steps<D, B, STEP0, NSTEPS>(a1, w[2], w[3], tbl);
#pragma unroll
  for (int s = 0; s < NSTEPS; ++s)
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      mma16816(acc[0][nb], a0[s][0], a0[s][1], a0[s][2], a0[s][3], xr[nb][2 * (STEP0 + s)], xr[nb][2 * (STEP0 + s) + 1]);
      mma16816(acc[1][nb], a1[s][0], a1[s][1], a1[s][2], a1[s][3], xr[nb][2 * (STEP0 + s)], xr[nb][2 * (STEP0 + s) + 1]);
    }
}

template <int D, int B, int NB>
__device__ __forceinline__ void task_all(float (&acc)[2][NB][4], const uint32_t (&w)[4][Policy<D, B>::LANE_WORDS],
                                         const uint32_t (&xr)[NB][32], uint32_t tbl) {
  task_steps<D, B, NB, 0, 4>(acc, w, xr, tbl);
  task_steps<D, B, NB, 4, 4>(acc, w, xr, tbl);
  task_steps<D, B, NB, 8, 4>(acc, w, xr, tbl);
  task_steps<D, B, NB, 12, 4>(acc, w, xr, tbl);
}

template <int D, int B, int NB>
__global__ void __launch_bounds__(Tile<D, B>::THREADS, Tile<D, B>::min_ctas(NB))
blockcb_kernel(Geometry g, LayerPtrs p, const __half* __restrict__ X, __half* __restrict__ Y, int batch, int n_chunks) {
  using P = Policy<D, B>;
  using T = Tile<D, B>;
  constexpr int LW = P::LANE_WORDS;
  constexpr int NBT = 8 * NB;
  extern __shared__ __align__(16) unsigned char smem[];
  // smem: [0, TABLE_BYTES) lane-private tables; afterwards reused for the partial sums
  const uint32_t smem_u32 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));

  cg::cluster_group cluster = cg::this_cluster();
  const int n_split = static_cast<int>(cluster.num_blocks());
  const int rank = static_cast<int>(cluster.block_rank());
  cluster_arrive_relaxed();  // waited on just before the first remote store
  // Programmatic dependent launch: the next kernel in the stream may start its own weight
  // streaming now; this kernel waits for its predecessor only where it first touches X.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  bool dep_waited = false;
  VQ_TRACE(0);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gq = lane >> 2, t = lane & 3;
  const int row0 = blockIdx.y * T::CTA_ROWS;
  const int slice = warp % P::SLICES;
  const int rgroup0 = warp / P::SLICES;                          // first row group of this warp
  constexpr int RGROUP_STEP = P::WARPS / P::SLICES;             // next task's row group
  const long long blk_row = static_cast<long long>(row0 / g.Br) * g.blocks_per_row;

  const uint32_t tbl = smem_u32 + (D == 2 ? lane * 4 : (lane & 15) * 8);

  float acc[P::TASKS][2][NB][4];
#pragma unroll
  for (int a = 0; a < P::TASKS; ++a)
#pragma unroll
    for (int b = 0; b < 2; ++b)
#pragma unroll
      for (int c = 0; c < NB; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[a][b][c][e] = 0.f;

  for (int chunk = rank; chunk < n_chunks; chunk += n_split) {
    const int col_cta = chunk * T::CTA_COLS;
    const int col_lane = col_cta + slice * 256 + t * 64;
    const bool lane_on = col_lane < g.K;

    // ---- 0. this thread's share of the chunk's codebooks (the whole CTA waits on these) ----
    typename std::conditional<D == 2, uint32_t, uint2>::type cbv;
    if constexpr (D == 2) {
      const int e = tid & 63, h = tid >> 6;
      const int col = col_cta + h * 128;
      cbv = 0u;
      if (col < g.K) cbv = __ldg(static_cast<const uint32_t*>(p.cb) + (blk_row + col / g.Bc) * P::ENTRIES + e);
    } else {
      cbv = __ldg(static_cast<const uint2*>(p.cb) + (blk_row + col_cta / g.Bc) * P::ENTRIES + tid);
    }

    // ---- 1. index stream -> registers (everything this warp will need for the chunk) ----
    uint32_t w[P::TASKS][4][LW];
#pragma unroll
    for (int task = 0; task < P::TASKS; ++task) {
      const int r = row0 + (rgroup0 + task * RGROUP_STEP) * 32 + gq;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint8_t* src = p.idx + static_cast<long long>(r + 8 * q) * g.stride + (static_cast<long long>(col_lane) / D) * B / 8;
        if (lane_on) {
          if constexpr (LW == 6) {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
              const uint2 v = ldg64_stream(src + 8 * i);
              w[task][q][2 * i] = v.x;
              w[task][q][2 * i + 1] = v.y;
            }
          } else {
            const uint4 v = ldg128_stream(src);
            w[task][q][0] = v.x; w[task][q][1] = v.y; w[task][q][2] = v.z; w[task][q][3] = v.w;
          }
        } else {
#pragma unroll
          for (int i = 0; i < LW; ++i) w[task][q][i] = 0u;
        }
      }
    }

    // ---- 2. activations of the lane's 64 columns -> B fragments ----
    if (!dep_waited) {
      asm volatile("griddepcontrol.wait;" ::: "memory");  // X (and Y) belong to the predecessor until here
      dep_waited = true;
    }
    uint32_t xr[NB][32];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      const int n = nb * 8 + gq;
      if (lane_on && n < batch) {
        const uint4* xs = reinterpret_cast<const uint4*>(X + static_cast<long long>(n) * g.K + col_lane);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 v = __ldg(xs + i);
          xr[nb][4 * i] = v.x; xr[nb][4 * i + 1] = v.y; xr[nb][4 * i + 2] = v.z; xr[nb][4 * i + 3] = v.w;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) xr[nb][i] = 0u;
      }
    }

    // ---- 3. stage the lane-private codebook copies ----
    // One global load per thread fetches the chunk's codebooks into a compact staging area; after
    // a barrier every thread replicates them into the [entry][lane] layout with 128-bit stores.
    if constexpr (D == 2) {
      // compact[e][h] = entry e of the chunk's block h (two 128-column blocks when Bc = 128)
      uint32_t* compact = reinterpret_cast<uint32_t*>(smem + P::TABLE_BYTES);
      {
        const int e = tid & 63, h = tid >> 6;             // 128 threads = 64 entries x 2 halves
        const int col = col_cta + h * 128;
        uint32_t v = 0u;
        if (col < g.K) v = cbv;
        compact[2 * e + h] = v;
      }
      VQ_TRACE(1);
      __syncthreads();
      // lanes 4u..4u+3 of entry e own columns 0-63, 64-127 (half 0) and 128-191, 192-255 (half 1)
#pragma unroll
      for (int j = 0; j < P::ENTRIES * 8 / T::THREADS; ++j) {
        const int item = tid + j * T::THREADS;            // (entry, 4-lane group)
        const int e = item >> 3, u = item & 7;
        const uint2 c = *reinterpret_cast<const uint2*>(compact + 2 * e);
        uint4 v;
        v.x = c.x; v.y = c.x; v.z = c.y; v.w = c.y;
        *reinterpret_cast<uint4*>(smem + e * 128 + u * 16) = v;
      }
    } else {
      // 8-byte word (e, c) <- entry e of the chunk's single codebook, 16 copies
      uint2* compact = reinterpret_cast<uint2*>(smem + P::TABLE_BYTES);
      compact[tid] = cbv;                                 // 256 threads = 256 entries
      __syncthreads();
#pragma unroll
      for (int j = 0; j < P::ENTRIES * 8 / T::THREADS; ++j) {
        const int item = tid + j * T::THREADS;            // (entry, pair of copies)
        const int e = item >> 3, u = item & 7;
        const uint2 c = compact[e];
        *reinterpret_cast<uint4*>(smem + e * 128 + u * 16) = make_uint4(c.x, c.y, c.x, c.y);
      }
    }
    __syncthreads();

    VQ_TRACE(2);
    // ---- 4. look up + multiply-accumulate ----
#pragma unroll
    for (int task = 0; task < P::TASKS; ++task) {
      task_all<D, B, NB>(acc[task], w[task], xr, tbl);
    }
    if (chunk + n_split < n_chunks) __syncthreads();  // the next chunk rewrites the tables
  }

  // ---- 5. push the partial sums to the cluster rank that owns each row ----
  // Row r of the tile is owned by rank r % n_split; the owner receives, from every (rank, slice),
  // one value per (row slot, batch row): recv[src][slot][n], src = rank * SLICES + slice.
  const int slots = (T::CTA_ROWS + n_split - 1) / n_split;
  const uint32_t recv_u32 = smem_u32 + P::TABLE_BYTES + kCompactBytes<D, B>;
  float* recv = reinterpret_cast<float*>(smem + P::TABLE_BYTES + kCompactBytes<D, B>);
  const int src = rank * P::SLICES + slice;
  VQ_TRACE(3);
  cluster_wait_acquire();  // matches the arrive at kernel entry: every CTA of the cluster is running
#pragma unroll
  for (int task = 0; task < P::TASKS; ++task)
#pragma unroll
    for (int half = 0; half < 2; ++half)
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = (rgroup0 + task * RGROUP_STEP) * 32 + half * 16 + gq + (e >> 1) * 8;
          const int n = nb * 8 + 2 * t + (e & 1);
          if (n < batch) {
            const int owner = r % n_split, slot = r / n_split;
            st_cluster_f32(recv_u32 + ((src * slots + slot) * batch + n) * 4, owner, acc[task][half][nb][e]);
          }
        }
  VQ_TRACE(4);
  cluster_arrive_release();
  cluster_wait_acquire();
  VQ_TRACE(5);

  // ---- 6. fixed-order sum over (rank, slice), one rounding, store ----
  const int n_src = n_split * P::SLICES;
  for (int o = tid; o < slots * batch; o += T::THREADS) {
    const int slot = o / batch, n = o % batch;
    const int r = slot * n_split + rank;
    if (r < T::CTA_ROWS) {
      float sum = 0.f;
      for (int q = 0; q < n_src; ++q) sum += recv[(q * slots + slot) * batch + n];
      Y[static_cast<long long>(n) * g.N + row0 + r] = __float2half_rn(sum);
    }
  }
  VQ_TRACE(6);
}

template <int D, int B, int NB>
vq_status launch(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, cudaStream_t s) {
  using P = Policy<D, B>;
  using T = Tile<D, B>;
  const int n_chunks = (g.K + T::CTA_COLS - 1) / T::CTA_COLS;
  const int row_blocks = g.N / T::CTA_ROWS;
  // tables + compact staging + receive buffer for the cluster reduction (worst case over splits)
  const size_t recv_bytes = static_cast<size_t>(P::SLICES) * (T::CTA_ROWS + 16) * 8 * NB * sizeof(float);
  const size_t smem_bytes = static_cast<size_t>(P::TABLE_BYTES) + kCompactBytes<D, B> + recv_bytes;
  auto kern = blockcb_kernel<D, B, NB>;
  // one-time, per-kernel attributes and occupancy (immutable properties of the device + kernel)
  static int slots = 0;
  if (slots == 0) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes)) != cudaSuccess ||
        cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
      return VQ_ERR_CUDA;
    int per_sm = 0, dev = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, T::THREADS, smem_bytes) != cudaSuccess ||
        cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || per_sm < 1)
      return VQ_ERR_CUDA;
    slots = per_sm * sms;
  }
  // K is split over the CTAs of a cluster (<= 16).  Model: time ~ waves * chunks per CTA; ties go
  // to the larger split (more, shorter CTAs balance the tail better).
  int best = 1;
  long long best_cost = -1;
  for (int sp = 1; sp <= 16 && sp <= n_chunks; ++sp) {
    const long long per = (n_chunks + sp - 1) / sp;
    const long long waves = (static_cast<long long>(row_blocks) * sp + slots - 1) / slots;
    const long long cost = per * waves;
    if (best_cost < 0 || cost <= best_cost) {
      best_cost = cost;
      best = sp;
    }
  }
#ifdef VQ_TUNING
  if (const char* e = getenv("VQ_SPLIT")) { const int v = atoi(e); if (v >= 1 && v <= 16 && v <= n_chunks) best = v; }
#endif
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(best, row_blocks, 1);
  cfg.blockDim = dim3(T::THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = best;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;  // programmatic dependent launch measured slower here; attribute left off
#ifdef VQ_TUNING
  if (getenv("VQ_PDL")) cfg.numAttrs = 2;
#endif
  if (cudaLaunchKernelEx(&cfg, kern, g, p, X, Y, batch, n_chunks) != cudaSuccess) return VQ_ERR_CUDA;
  return check_launch();
}

}  // namespace

// Shared-codebook families: fp16 codebooks, block rows a multiple of the CTA tile height,
// block columns a multiple of what one lane (64) / one CTA chunk covers.
vq_status launch_gemm_blockcb(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch,
                              cudaStream_t s) {
  if (g.cb_int8) return VQ_ERR_UNSUPPORTED;
  if (g.K % 64) return VQ_ERR_UNSUPPORTED;
  if (g.d == 2 && g.b == 6) {
    if (g.Br % Tile<2, 6>::CTA_ROWS || g.Bc % 128) return VQ_ERR_UNSUPPORTED;
    return batch <= 8 ? launch<2, 6, 1>(g, p, X, Y, batch, s) : launch<2, 6, 2>(g, p, X, Y, batch, s);
  }
  if (g.d == 4 && g.b == 8) {
    if (g.Br % Tile<4, 8>::CTA_ROWS || g.Bc % Tile<4, 8>::CTA_COLS) return VQ_ERR_UNSUPPORTED;
    return batch <= 8 ? launch<4, 8, 1>(g, p, X, Y, batch, s) : launch<4, 8, 2>(g, p, X, Y, batch, s);
  }
  return VQ_ERR_UNSUPPORTED;
}

}  // namespace vq
