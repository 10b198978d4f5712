// E-step / VQ_quant (paper Sec. 3, Eq. 5): for every d-vector x of a dense matrix (d adjacent
// columns of one row) the index of the centroid of its block that minimises
// (x - c)^T D (x - c), D = diagonal weights of the vector's columns, written in the packed index
// format the decode path reads.  Arithmetic-bound: (4d + 2) operations per (vector, centroid).
//
// A CTA takes a tile of 32 rows x 256*d columns; its codebooks go to shared memory as binary32
// (int8 entries times their block scale, exact).  A thread owns 8 consecutive vectors of a row
// (one group of 8 indices = b whole bytes of the stream), keeps them and their weights in
// registers, walks the centroids once (shared-memory broadcasts) and writes its b bytes.
//
// The decision is taken in binary32 with every operation rounded separately (no fused
// multiply-add), terms added left to right, lowest index among equal distances: the same
// sequence the CPU oracle evaluates, so both sides break near-ties alike.
#include "vq_common.cuh"

namespace vq {
namespace {

constexpr int kRows = 32;
constexpr int kWarps = 8;

struct AssignArgs {
  const __half* W;
  const void* cb;
  const __half* scale;
  const float* hdiag;   // [K] or null (identity)
  uint8_t* idx;
  long long stride;
  int N, K, b, Br, Bc, entries, blocks_per_row, groups;   // groups = K / (8 d) per row
  int used_bytes;       // bytes of a row that hold indices; the rest of the stride is zero-filled
  int bc_shift;         // log2(Bc)
  int br_per_tile, bc_per_seg, rows_per_br;
};

template <int D>
__global__ void __launch_bounds__(32 * kWarps) assign_kernel(const AssignArgs a) {
  extern __shared__ __align__(16) float tables[];   // [block row][block col][entry][D]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int seg_cols = 256 * D;
  const int row0 = blockIdx.y * kRows, col0 = blockIdx.x * seg_cols;
  const int table_floats = a.entries * D;
  {
    const long long br0 = row0 / a.Br, bc0 = col0 / a.Bc;
    const long long last_br = (a.N - 1) / a.Br;
    const int n_tab = a.br_per_tile * a.bc_per_seg;
    for (int o = tid; o < n_tab * table_floats; o += 32 * kWarps) {
      const int tb = o / table_floats, within = o - tb * table_floats;
      const int lbr = tb / a.bc_per_seg, lbc = tb - lbr * a.bc_per_seg;
      long long brow = br0 + lbr, bcol = bc0 + lbc;
      if (brow > last_br) brow = last_br;                        // rows past N: never used
      if (bcol >= a.blocks_per_row) bcol = a.blocks_per_row - 1;  // columns past K: never used
      const long long blk = brow * a.blocks_per_row + bcol;
      float v;
      if (a.scale == nullptr) v = __half2float(__ldg(static_cast<const __half*>(a.cb) + blk * table_floats + within));
      else v = __fmul_rn(static_cast<float>(__ldg(static_cast<const int8_t*>(a.cb) + blk * table_floats + within)),
                         __half2float(__ldg(a.scale + blk)));
      tables[o] = v;
    }
  }
  __syncthreads();

  const int grp = blockIdx.x * 32 + lane;   // group of 8 indices within the row
  if (grp >= a.groups) return;
  const int col = grp * 8 * D;              // first column of the thread's 8 vectors
  float dw[8][D];
#pragma unroll
  for (int v = 0; v < 8; ++v)
#pragma unroll
    for (int t = 0; t < D; ++t) dw[v][t] = a.hdiag ? __ldg(a.hdiag + col + v * D + t) : 1.f;
  const int lbc = (col - col0) >> a.bc_shift;   // 0 when the block is wider than the segment

  for (int r = warp; r < kRows; r += kWarps) {
    const int n = row0 + r;
    if (n >= a.N) break;
    float x[8][D];
    {
      const uint4* src = reinterpret_cast<const uint4*>(a.W + static_cast<long long>(n) * a.K + col);
#pragma unroll
      for (int q = 0; q < D; ++q) {   // 8*D halves = D 128-bit loads
        const uint4 raw = __ldg(src + q);
        const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int h = 0; h < 8; ++h) {
          const int e = q * 8 + h;   // element index among the thread's 8*D weights
          const __half_raw hr = {static_cast<unsigned short>((wds[h >> 1] >> (16 * (h & 1))) & 0xffff)};
          x[e / D][e % D] = __half2float(__half(hr));
        }
      }
    }
    const float* tab = tables + ((r / a.rows_per_br) * a.bc_per_seg + lbc) * table_floats;
    float best[8];
    int bidx[8];
#pragma unroll
    for (int v = 0; v < 8; ++v) {
      best[v] = __int_as_float(0x7f800000);   // +inf
      bidx[v] = 0;
    }
    for (int m = 0; m < a.entries; ++m) {
      float c[D];
#pragma unroll
      for (int t = 0; t < D; ++t) c[t] = tab[m * D + t];
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        float acc = 0.f;
#pragma unroll
        for (int t = 0; t < D; ++t) {
          const float diff = __fsub_rn(x[v][t], c[t]);
          const float term = __fmul_rn(dw[v][t], __fmul_rn(diff, diff));
          acc = t == 0 ? term : __fadd_rn(acc, term);
        }
        if (acc < best[v]) {
          best[v] = acc;
          bidx[v] = m;
        }
      }
    }
    unsigned long long bits = 0;
#pragma unroll
    for (int v = 0; v < 8; ++v) bits |= static_cast<unsigned long long>(bidx[v]) << (v * a.b);
    uint8_t* dst = a.idx + n * a.stride + static_cast<long long>(grp) * a.b;
    for (int i = 0; i < a.b; ++i) dst[i] = static_cast<uint8_t>(bits >> (8 * i));
    if (grp == a.groups - 1)   // padding up to the row stride
      for (long long i = a.used_bytes; i < a.stride; ++i) a.idx[n * a.stride + i] = 0;
  }
}

}  // namespace

// Covers formats with a whole number of 8-index groups per row that do not straddle blocks
// (block_cols a power of two multiple of 8 d), block rows that divide or are divided by 32.
vq_status launch_assign(const Geometry& g, const LayerPtrs& p, const __half* W, const float* hdiag, uint8_t* idx,
                        cudaStream_t s) {
  const int seg_cols = 256 * g.d;
  if (g.cb_int4 || g.J % 8 || g.Bc % (8 * g.d)) return VQ_ERR_UNSUPPORTED;
  int bc_shift = -1;
  for (int sft = 3; sft < 31; ++sft)
    if ((1 << sft) == g.Bc) bc_shift = sft;
  if (bc_shift < 0) return VQ_ERR_UNSUPPORTED;
  if (kRows % g.Br && g.Br % kRows) return VQ_ERR_UNSUPPORTED;
  AssignArgs a;
  a.W = W;
  a.cb = p.cb;
  a.scale = g.cb_int8 ? p.scale : nullptr;
  a.hdiag = hdiag;
  a.idx = idx;
  a.stride = g.stride;
  a.N = g.N;
  a.K = g.K;
  a.b = g.b;
  a.Br = g.Br;
  a.Bc = g.Bc;
  a.entries = g.entries;
  a.blocks_per_row = g.blocks_per_row;
  a.groups = g.J / 8;
  a.used_bytes = a.groups * g.b;
  a.bc_shift = bc_shift;
  a.br_per_tile = g.Br >= kRows ? 1 : kRows / g.Br;
  a.bc_per_seg = g.Bc >= seg_cols ? 1 : seg_cols / g.Bc;
  a.rows_per_br = g.Br >= kRows ? kRows : g.Br;
  const size_t smem = static_cast<size_t>(a.br_per_tile) * a.bc_per_seg * g.entries * g.d * sizeof(float);
  if (smem > 96 * 1024) return VQ_ERR_UNSUPPORTED;
  const dim3 grid((a.groups + 31) / 32, (g.N + kRows - 1) / kRows, 1);
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
  if (g.d == 1) return launch(assign_kernel<1>, 0);
  if (g.d == 2) return launch(assign_kernel<2>, 1);
  return launch(assign_kernel<4>, 2);
}

}  // namespace vq
