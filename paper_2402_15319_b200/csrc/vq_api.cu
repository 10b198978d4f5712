// C-ABI entry points: host-side validation and kernel dispatch.  No kernel lives here.
#include <math.h>
#include <stdlib.h>

#include "vq_common.cuh"

namespace vq {

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static vq_status check_format(const vq_format* f) {
  if (!f) return VQ_ERR_NULL;
  if (!(f->vq_dim == 1 || f->vq_dim == 2 || f->vq_dim == 4)) return VQ_ERR_FORMAT;
  if (f->index_bits < 1 || f->index_bits > 8) return VQ_ERR_FORMAT;
  if (!(f->cb_type == VQ_CB_FP16 || f->cb_type == VQ_CB_INT8_SCALED || f->cb_type == VQ_CB_INT4_G128)) return VQ_ERR_FORMAT;
  if (f->n_rows <= 0 || f->k_cols <= 0 || f->block_rows <= 0 || f->block_cols <= 0) return VQ_ERR_SHAPE;
  if (f->n_rows % f->block_rows || f->k_cols % f->block_cols || f->block_cols % f->vq_dim) return VQ_ERR_SHAPE;
  if (f->cb_type == VQ_CB_INT4_G128 && f->k_cols % 128) return VQ_ERR_SHAPE;
  return VQ_OK;
}

static long long row_stride(const vq_format* f) {
  const long long bits = static_cast<long long>(f->k_cols / f->vq_dim) * f->index_bits;
  return ((bits + 7) / 8 + 15) / 16 * 16;
}

vq_status make_geometry(const vq_format* f, Geometry* g) {
  vq_status st = check_format(f);
  if (st != VQ_OK) return st;
  g->N = f->n_rows;
  g->K = f->k_cols;
  g->d = f->vq_dim;
  g->b = f->index_bits;
  g->Br = f->block_rows;
  g->Bc = f->block_cols;
  g->cb_int8 = f->cb_type == VQ_CB_INT8_SCALED;
  g->cb_int4 = f->cb_type == VQ_CB_INT4_G128;
  g->entries = 1 << f->index_bits;
  g->J = f->k_cols / f->vq_dim;
  g->blocks_per_row = f->k_cols / f->block_cols;
  g->stride = row_stride(f);
  return VQ_OK;
}

static size_t round256(size_t v) { return (v + 255) / 256 * 256; }

static vq_status check_layer(const vq_format* fmt, const void* d_idx, const void* d_cb,
                             const void* d_scale, Geometry* g, LayerPtrs* p) {
  vq_status st = make_geometry(fmt, g);
  if (st != VQ_OK) return st;
  if (!d_idx || !d_cb) return VQ_ERR_NULL;
  if ((g->cb_int8 || g->cb_int4) ? d_scale == nullptr : d_scale != nullptr) return VQ_ERR_NULL;
  if (!aligned16(d_idx) || !aligned16(d_cb) || !aligned16(d_scale)) return VQ_ERR_ALIGN;
  p->idx = static_cast<const uint8_t*>(d_idx);
  p->cb = d_cb;
  p->scale = static_cast<const __half*>(d_scale);
  return VQ_OK;
}

}  // namespace vq

namespace {
// Device-side address of a pinned (page-locked, mapped) host allocation, or null for any other memory.
const void* mapped_device_pointer(const void* h) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, h) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}
// X from mapped host memory into device memory: 16-byte pieces, grid-stride.
__global__ void __launch_bounds__(256) fetch_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int n16) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x) dst[i] = src[i];
}
}  // namespace

using namespace vq;

extern "C" {

vq_status vq_pack_info(const vq_format* fmt, vq_pack_info_t* out) {
  if (!out) return VQ_ERR_NULL;
  vq_status st = check_format(fmt);
  if (st != VQ_OK) return st;
  const long long N = fmt->n_rows, K = fmt->k_cols, d = fmt->vq_dim;
  const long long k = 1LL << fmt->index_bits;
  const int b_c = fmt->cb_type == VQ_CB_INT8_SCALED ? 8 : fmt->cb_type == VQ_CB_INT4_G128 ? 4 : 16;
  const long long l = static_cast<long long>(fmt->block_rows) * fmt->block_cols;
  out->entries = static_cast<int32_t>(k);
  out->codebook_bits = b_c;
  out->indices_per_row = K / d;
  out->row_stride_bytes = row_stride(fmt);
  out->index_bytes = N * out->row_stride_bytes;
  out->n_blocks = (N / fmt->block_rows) * (K / fmt->block_cols);
  out->codebook_bytes_per_block = k * d * b_c / 8;
  out->codebook_bytes = out->n_blocks * out->codebook_bytes_per_block;
  out->scale_bytes = fmt->cb_type == VQ_CB_INT8_SCALED ? 2 * out->n_blocks : fmt->cb_type == VQ_CB_INT4_G128 ? 2 * N * (K / 128) : 0;
  out->total_bytes = out->index_bytes + out->codebook_bytes + out->scale_bytes;
  out->bpv_paper = static_cast<double>(fmt->index_bits) / d + static_cast<double>(k * d * b_c) / static_cast<double>(l);
  out->bpv_stored = 8.0 * static_cast<double>(out->total_bytes) / static_cast<double>(N * K);
  return VQ_OK;
}

size_t vq_workspace_bytes(const vq_format* fmt, int batch) {
  if (check_format(fmt) != VQ_OK || batch < 1 || batch > 16) return 0;
  return stream_workspace_bytes(fmt->n_rows, batch);
}

size_t vq_workspace_bytes_host(const vq_format* fmt, int batch) {
  const size_t base = vq_workspace_bytes(fmt, batch);
  if (!base) return 0;
  return base + round256(static_cast<size_t>(batch) * fmt->k_cols * 2) + round256(static_cast<size_t>(batch) * fmt->n_rows * 2);
}

vq_status vq_decode_weights(const vq_format* fmt, const void* d_idx, const void* d_cb,
                            const void* d_scale, void* d_W, void* stream) {
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);
  if (st != VQ_OK) return st;
  if (!d_W) return VQ_ERR_NULL;
  if (!aligned16(d_W)) return VQ_ERR_ALIGN;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = launch_decode_tuned(g, p, static_cast<__half*>(d_W), s);
  if (st == VQ_ERR_UNSUPPORTED) st = launch_decode_generic(g, p, static_cast<__half*>(d_W), s);
  return st;
}

vq_status vq_assign_indices(const vq_format* fmt, const void* d_W, const void* d_cb, const void* d_scale,
                            const void* d_hdiag, void* d_idx, void* stream) {
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);   // d_idx: checked like an input, written here
  if (st != VQ_OK) return st;
  if (!d_W) return VQ_ERR_NULL;
  if (!aligned16(d_W) || (d_hdiag && !aligned16(d_hdiag))) return VQ_ERR_ALIGN;
  return launch_assign(g, p, static_cast<const __half*>(d_W), static_cast<const float*>(d_hdiag),
                       static_cast<uint8_t*>(d_idx), static_cast<cudaStream_t>(stream));
}

vq_status vq_gemm_small_batch_impl(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                   const void* d_scale, const void* d_X, void* d_Y, int batch,
                                   void* d_ws, size_t ws_bytes, void* stream, int impl) {
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);
  if (st != VQ_OK) return st;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  if (!d_X || !d_Y) return VQ_ERR_NULL;
  if (!aligned16(d_X) || !aligned16(d_Y)) return VQ_ERR_ALIGN;
  if (!d_ws || ws_bytes < vq_workspace_bytes(fmt, batch)) return VQ_ERR_WORKSPACE;
  if (!aligned16(d_ws)) return VQ_ERR_ALIGN;
  if (impl != VQ_IMPL_AUTO && impl != VQ_IMPL_GENERIC && impl != VQ_IMPL_TUNED && impl != VQ_IMPL_STREAM) return VQ_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const __half* X = static_cast<const __half*>(d_X);
  __half* Y = static_cast<__half*>(d_Y);
  if (impl == VQ_IMPL_STREAM) {
    if (g.cb_int4) return VQ_ERR_UNSUPPORTED;
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
    call.ws = d_ws;
    call.ws_bytes = ws_bytes;
    return launch_gemm_stream(call, s);
  }
  if (impl != VQ_IMPL_GENERIC) {
    st = launch_gemm_tuned(g, p, X, Y, batch, d_ws, ws_bytes, s);
    if (st != VQ_ERR_UNSUPPORTED || impl == VQ_IMPL_TUNED) return st;
  }
  return launch_gemm_generic(g, p, X, Y, batch, s);
}

// Which kernel family serves a group in one launch: 2 = the cluster kernels of the shared-codebook
// formats (their K-split meets in distributed shared memory: lowest latency on the small layers those
// formats come with), 1 = the persistent kernel (per-row formats: q/k/v of the 70B-shaped set in one
// launch 11.4 us against 19.5 us for three launches at batch 1, 20.3 against 37.4 us at batch 8),
// 3 = the pair-table kernel (small codebook blocks; index widths other than 4 bits, which the row kernels
// or the persistent kernel take: q/k/v of the Llama-3-8B-shaped set with 5-bit indices and 4 x 256 blocks in
// one launch instead of three), 0 = member by member.
static int group_family(const Geometry& g, int) {
  if (blockcb_covers(g)) return 2;
  if (g.cb_int4) return warptab_covers(g) ? 3 : 0;
  if (g.b != 4 && !stream_covers(g) && warptab_covers(g)) return 3;
  return 1;
}

int vq_grouped_kernel_launches(const vq_format* fmt, int n_members, int batch) {
  Geometry g;
  if (make_geometry(fmt, &g) != VQ_OK || n_members < 1 || n_members > VQ_MAX_GROUP || batch < 1 || batch > 16) return 0;
  if (n_members > 1 && blockcb_covers(g) && group_family(g, batch) == 2) return 1;
  if (n_members > 1 && group_family(g, batch) == 3) return 1;
  return (n_members > 1 && group_family(g, batch) == 1 && stream_covers(g)) ? 1 : n_members;
}

vq_status vq_gemm_small_batch_grouped(const vq_format* fmt, const vq_group_member* members, int n_members,
                                      const void* d_X, int batch, void* d_ws, size_t ws_bytes, void* stream) {
  if (!fmt || !members) return VQ_ERR_NULL;
  if (n_members < 1 || n_members > VQ_MAX_GROUP) return VQ_ERR_SHAPE;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  if (!d_X) return VQ_ERR_NULL;
  if (!aligned16(d_X)) return VQ_ERR_ALIGN;
  if (!d_ws || ws_bytes < vq_workspace_bytes(fmt, batch)) return VQ_ERR_WORKSPACE;
  if (!aligned16(d_ws)) return VQ_ERR_ALIGN;
  StreamCall call = {};
  long long rows = 0;
  vq_format one = *fmt;
  for (int i = 0; i < n_members; ++i) {
    const vq_group_member& m = members[i];
    one.n_rows = m.n_rows;
    Geometry g;
    LayerPtrs p;
    vq_status st = check_layer(&one, m.d_idx, m.d_cb, m.d_scale, &g, &p);
    if (st != VQ_OK) return st;
    if (!m.d_Y) return VQ_ERR_NULL;
    if (!aligned16(m.d_Y)) return VQ_ERR_ALIGN;
    if (i == 0) call.g = g;
    call.idx[i] = p.idx;
    call.cb[i] = p.cb;
    call.scale[i] = p.scale;
    call.Y[i] = static_cast<__half*>(m.d_Y);
    call.N[i] = m.n_rows;
    rows += m.n_rows;
  }
  if (rows != fmt->n_rows) return VQ_ERR_SHAPE;
  call.n_seg = n_members;
  call.X = static_cast<const __half*>(d_X);
  call.batch = batch;
  call.ws = d_ws;
  call.ws_bytes = ws_bytes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  vq_status st = VQ_ERR_UNSUPPORTED;
  if (n_members > 1) {
    int fam = group_family(call.g, batch);
#ifdef VQ_TUNING
    if (getenv("VQ_GROUP_FAMILY")) fam = atoi(getenv("VQ_GROUP_FAMILY"));
#endif
    if (fam == 3) st = launch_gemm_warptab_group(call, s);
    if (fam == 2) st = launch_gemm_blockcb_group(call, s);
    if (fam == 1 || (fam == 2 && st == VQ_ERR_UNSUPPORTED)) st = launch_gemm_stream(call, s);
  }
  if (st != VQ_ERR_UNSUPPORTED) return st;
  for (int i = 0; i < n_members; ++i) {   // formats the persistent kernel does not take: member by member
    one.n_rows = members[i].n_rows;
    st = vq_gemm_small_batch(&one, members[i].d_idx, members[i].d_cb, members[i].d_scale, d_X, members[i].d_Y, batch, d_ws,
                             ws_bytes, stream);
    if (st != VQ_OK) return st;
  }
  return VQ_OK;
}

// Sub-rows of norm_block_cols columns: they tile a codebook block's columns and hold whole VQ vectors.
static vq_status check_norm(const vq_format* fmt, const void* d_codes, const void* d_lut, int norm_block_cols) {
  if (!d_codes || !d_lut) return VQ_ERR_NULL;
  if (norm_block_cols <= 0 || fmt->block_cols % norm_block_cols || norm_block_cols % fmt->vq_dim) return VQ_ERR_SHAPE;
  if (!aligned16(d_codes) || !aligned16(d_lut)) return VQ_ERR_ALIGN;
  return VQ_OK;
}

vq_status vq_norm_info(const vq_format* fmt, int norm_block_cols, vq_norm_info_t* out) {
  if (!out) return VQ_ERR_NULL;
  Geometry g;
  vq_status st = make_geometry(fmt, &g);
  if (st != VQ_OK) return st;
  if (norm_block_cols <= 0 || g.Bc % norm_block_cols || norm_block_cols % g.d) return VQ_ERR_SHAPE;
  out->code_row_bytes = (g.K / norm_block_cols + 1) / 2;
  out->codes_bytes = static_cast<size_t>(g.N) * out->code_row_bytes;
  out->lut_bytes = static_cast<size_t>(g.N / g.Br) * g.blocks_per_row * 16 * sizeof(uint16_t);
  return VQ_OK;
}

vq_status vq_decode_weights_normalized(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                                       const void* d_norm_codes, const void* d_norm_lut, int norm_block_cols, void* d_W,
                                       void* stream) {
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);
  if (st != VQ_OK) return st;
  st = check_norm(fmt, d_norm_codes, d_norm_lut, norm_block_cols);
  if (st != VQ_OK) return st;
  if (!d_W) return VQ_ERR_NULL;
  if (!aligned16(d_W)) return VQ_ERR_ALIGN;
  // the tile kernel where it takes the format and the sub-row size, else the format-generic kernel
  st = launch_decode_tuned(g, p, static_cast<__half*>(d_W), static_cast<cudaStream_t>(stream), d_norm_codes, d_norm_lut, norm_block_cols);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  return launch_decode_norm(g, p, d_norm_codes, d_norm_lut, norm_block_cols, static_cast<__half*>(d_W), static_cast<cudaStream_t>(stream));
}

vq_status vq_gemm_small_batch_normalized(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                                         const void* d_norm_codes, const void* d_norm_lut, int norm_block_cols, const void* d_X,
                                         void* d_Y, int batch, void* stream) {
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);
  if (st != VQ_OK) return st;
  st = check_norm(fmt, d_norm_codes, d_norm_lut, norm_block_cols);
  if (st != VQ_OK) return st;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  if (!d_X || !d_Y) return VQ_ERR_NULL;
  if (!aligned16(d_X) || !aligned16(d_Y)) return VQ_ERR_ALIGN;
  // the pair-table kernel where it takes the format and the sub-row size, else the format-generic kernel
  st = launch_gemm_warptab_norm(g, p, d_norm_codes, d_norm_lut, norm_block_cols, static_cast<const __half*>(d_X),
                                static_cast<__half*>(d_Y), batch, static_cast<cudaStream_t>(stream));
  if (st != VQ_ERR_UNSUPPORTED) return st;
  return launch_gemm_norm(g, p, d_norm_codes, d_norm_lut, norm_block_cols, static_cast<const __half*>(d_X), static_cast<__half*>(d_Y),
                          batch, static_cast<cudaStream_t>(stream));
}

vq_status vq_gemm_small_batch(const vq_format* fmt, const void* d_idx, const void* d_cb,
                              const void* d_scale, const void* d_X, void* d_Y, int batch,
                              void* d_ws, size_t ws_bytes, void* stream) {
  return vq_gemm_small_batch_impl(fmt, d_idx, d_cb, d_scale, d_X, d_Y, batch, d_ws, ws_bytes, stream, VQ_IMPL_AUTO);
}

vq_status vq_gemv(const vq_format* fmt, const void* d_idx, const void* d_cb, const void* d_scale,
                  const void* d_x, void* d_y, void* d_ws, size_t ws_bytes, void* stream) {
  return vq_gemm_small_batch_impl(fmt, d_idx, d_cb, d_scale, d_x, d_y, 1, d_ws, ws_bytes, stream, VQ_IMPL_AUTO);
}

vq_status vq_gemm_small_batch_host(const vq_format* fmt, const void* d_idx, const void* d_cb,
                                   const void* d_scale, const void* h_X, void* h_Y, int batch,
                                   void* d_ws, size_t ws_bytes, void* stream) {
  if (!h_X || !h_Y) return VQ_ERR_NULL;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  Geometry g;
  LayerPtrs p;
  vq_status st = check_layer(fmt, d_idx, d_cb, d_scale, &g, &p);
  if (st != VQ_OK) return st;
  const size_t need = vq_workspace_bytes_host(fmt, batch);
  if (!d_ws || ws_bytes < need) return VQ_ERR_WORKSPACE;
  if (!aligned16(d_ws)) return VQ_ERR_ALIGN;
  const size_t base = vq_workspace_bytes(fmt, batch);
  const size_t x_bytes = static_cast<size_t>(batch) * fmt->k_cols * 2;
  const size_t y_bytes = static_cast<size_t>(batch) * fmt->n_rows * 2;
  char* ws = static_cast<char*>(d_ws);
  void* d_X = ws + base;
  void* d_Y = ws + base + round256(x_bytes);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Pinned host buffers are mapped into the device's address space: one small kernel fetches X and
  // the mat-vec kernel stores Y straight into host memory, so the step stays on the compute engine
  // (two copy-engine hand-overs cost more than the kernel they surround).  Anything else (pageable
  // memory, unaligned Y) takes the two asynchronous copies below.
  {
    const void* dx = mapped_device_pointer(h_X);
    void* dy = const_cast<void*>(mapped_device_pointer(h_Y));
    if (dx && dy && aligned16(dx) && aligned16(dy)) {
      const int n16 = static_cast<int>(x_bytes / 16);
      if (x_bytes % 16 == 0) {   // whole 16-byte pieces only
        int blocks = (n16 + 255) / 256;
        if (blocks > 8) blocks = 8;
        fetch_kernel<<<blocks, 256, 0, s>>>(static_cast<const uint4*>(dx), static_cast<uint4*>(d_X), n16);
        if (check_launch() != VQ_OK) return VQ_ERR_CUDA;
        return vq_gemm_small_batch(fmt, d_idx, d_cb, d_scale, d_X, dy, batch, d_ws, base, stream);
      }
    }
  }
  if (cudaMemcpyAsync(d_X, h_X, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return VQ_ERR_CUDA;
  st = vq_gemm_small_batch(fmt, d_idx, d_cb, d_scale, d_X, d_Y, batch, d_ws, base, stream);
  if (st != VQ_OK) return st;
  if (cudaMemcpyAsync(h_Y, d_Y, y_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VQ_ERR_CUDA;
  return VQ_OK;
}

// Grouped call with host activations and outputs (see vq.h).  The members' d_Y fields are HOST pointers here.
vq_status vq_gemm_small_batch_grouped_host(const vq_format* fmt, const vq_group_member* members, int n_members,
                                           const void* h_X, int batch, void* d_ws, size_t ws_bytes, void* stream) {
  if (!fmt || !members || !h_X) return VQ_ERR_NULL;
  if (n_members < 1 || n_members > VQ_MAX_GROUP) return VQ_ERR_SHAPE;
  if (batch < 1 || batch > 16) return VQ_ERR_BATCH;
  const size_t base = vq_workspace_bytes(fmt, batch);
  if (!base) return VQ_ERR_FORMAT;
  // device copies: X, then every member's Y on a 256-byte boundary
  const size_t x_bytes = static_cast<size_t>(batch) * fmt->k_cols * 2;
  size_t need = base + round256(x_bytes);
  long long rows = 0;
  for (int i = 0; i < n_members; ++i) {
    if (!members[i].d_Y) return VQ_ERR_NULL;
    if (members[i].n_rows <= 0) return VQ_ERR_SHAPE;
    need += round256(static_cast<size_t>(batch) * members[i].n_rows * 2);
    rows += members[i].n_rows;
  }
  if (rows != fmt->n_rows) return VQ_ERR_SHAPE;
  if (!d_ws || ws_bytes < need) return VQ_ERR_WORKSPACE;
  if (!aligned16(d_ws)) return VQ_ERR_ALIGN;
  char* ws = static_cast<char*>(d_ws);
  void* d_X = ws + base;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  vq_group_member dev[VQ_MAX_GROUP];
  // pinned (mapped) buffers: one small kernel fetches X, the mat-vec kernel stores every Y straight
  // into host memory (as vq_gemm_small_batch_host does)
  bool mapped = x_bytes % 16 == 0;
  const void* dx = mapped ? mapped_device_pointer(h_X) : nullptr;
  mapped = mapped && dx && aligned16(dx);
  for (int i = 0; i < n_members && mapped; ++i) {
    dev[i] = members[i];
    dev[i].d_Y = const_cast<void*>(mapped_device_pointer(members[i].d_Y));
    mapped = dev[i].d_Y && aligned16(dev[i].d_Y);
  }
  if (mapped) {
    const int n16 = static_cast<int>(x_bytes / 16);
    int blocks = (n16 + 255) / 256;
    if (blocks > 8) blocks = 8;
    fetch_kernel<<<blocks, 256, 0, s>>>(static_cast<const uint4*>(dx), static_cast<uint4*>(d_X), n16);
    if (check_launch() != VQ_OK) return VQ_ERR_CUDA;
    return vq_gemm_small_batch_grouped(fmt, dev, n_members, d_X, batch, d_ws, base, stream);
  }
  size_t off = base + round256(x_bytes);
  for (int i = 0; i < n_members; ++i) {
    dev[i] = members[i];
    dev[i].d_Y = ws + off;
    off += round256(static_cast<size_t>(batch) * members[i].n_rows * 2);
  }
  if (cudaMemcpyAsync(d_X, h_X, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return VQ_ERR_CUDA;
  const vq_status st = vq_gemm_small_batch_grouped(fmt, dev, n_members, d_X, batch, d_ws, base, stream);
  if (st != VQ_OK) return st;
  for (int i = 0; i < n_members; ++i)
    if (cudaMemcpyAsync(members[i].d_Y, dev[i].d_Y, static_cast<size_t>(batch) * members[i].n_rows * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess)
      return VQ_ERR_CUDA;
  return VQ_OK;
}

size_t vq_workspace_bytes_grouped_host(const vq_format* fmt, int n_members, int batch) {
  const size_t base = vq_workspace_bytes(fmt, batch);
  if (!base || n_members < 1 || n_members > VQ_MAX_GROUP) return 0;
  // every member's Y on its own 256-byte boundary: at most 256 bytes of padding each
  return base + round256(static_cast<size_t>(batch) * fmt->k_cols * 2) + round256(static_cast<size_t>(batch) * fmt->n_rows * 2) +
         256 * static_cast<size_t>(n_members);
}

const char* vq_status_string(vq_status s) {
  switch (s) {
    case VQ_OK: return "VQ_OK";
    case VQ_ERR_NULL: return "VQ_ERR_NULL: missing pointer or scale pointer does not match cb_type";
    case VQ_ERR_FORMAT: return "VQ_ERR_FORMAT: vq_dim/index_bits/cb_type out of range";
    case VQ_ERR_SHAPE: return "VQ_ERR_SHAPE: sizes not positive or not divisible by the block shape";
    case VQ_ERR_ALIGN: return "VQ_ERR_ALIGN: device pointer not 16-byte aligned";
    case VQ_ERR_WORKSPACE: return "VQ_ERR_WORKSPACE: workspace missing or too small";
    case VQ_ERR_BATCH: return "VQ_ERR_BATCH: batch outside 1..16";
    case VQ_ERR_UNSUPPORTED: return "VQ_ERR_UNSUPPORTED: requested kernel variant does not cover this format";
    case VQ_ERR_CUDA: return "VQ_ERR_CUDA: CUDA runtime reported an error";
  }
  return "unknown vq_status";
}

}  // extern "C"
