// Dispatch to the tuned kernel families.
#include "vq_common.cuh"

namespace vq {

namespace {
// Incremented by a kernel whenever one of its bounded waits gives up; stays 0 in a healthy run.
static __device__ int g_wait_failures;
}  // namespace

vq_status encode_index_map(CUtensorMap* tm, const uint8_t* idx, long long stride, int N, int box_bytes, int box_rows,
                           bool swizzle128) {
  using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                     const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  // the driver's encoder, looked up once through the runtime (no link against libcuda)
  static EncodeTiledFn encode = nullptr;
  if (!encode) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !p)
      return VQ_ERR_CUDA;
    encode = reinterpret_cast<EncodeTiledFn>(p);
  }
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(stride), static_cast<cuuint64_t>(N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(stride)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_bytes), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem_strides[2] = {1u, 1u};
  if (encode(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(idx), dims, strides, box, elem_strides,
             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VQ_ERR_CUDA;
  return VQ_OK;
}

vq_status encode_tensor_map(CUtensorMap* tm, const void* base, int elem_bytes, int rank, const uint64_t* dims,
                            const uint64_t* strides, const uint32_t* box, int swizzle) {
  using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                     const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                     CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeTiledFn encode = nullptr;   // (a pointer-sized store; two first callers write the same value)
  if (!encode) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess || !p)
      return VQ_ERR_CUDA;
    encode = reinterpret_cast<EncodeTiledFn>(p);
  }
  if (rank < 1 || rank > 5 || (elem_bytes != 1 && elem_bytes != 2)) return VQ_ERR_CUDA;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    es[i] = 1u;
    if (i + 1 < rank) st[i] = strides[i];
  }
  const CUtensorMapSwizzle sw = swizzle == 2 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle == 1 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE;
  if (encode(tm, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_UINT16, static_cast<cuuint32_t>(rank),
             const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_NONE,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return VQ_ERR_CUDA;
  return VQ_OK;
}

// Per-device values looked up on first use.  Two host threads may make that first call together: both
// then compute the same value and publish it with a release store, readers use an acquire load.
vq_status device_error_counter(int** d_counter) {
  static int* addr_of[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  int* addr = __atomic_load_n(&addr_of[dev], __ATOMIC_ACQUIRE);
  if (!addr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_wait_failures) != cudaSuccess || !p) return VQ_ERR_CUDA;
    addr = static_cast<int*>(p);
    __atomic_store_n(&addr_of[dev], addr, __ATOMIC_RELEASE);
  }
  *d_counter = addr;
  return VQ_OK;
}

vq_status device_sms(int* out) {
  static int sms_of[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return VQ_ERR_CUDA;
  int n = __atomic_load_n(&sms_of[dev], __ATOMIC_ACQUIRE);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return VQ_ERR_CUDA;
    __atomic_store_n(&sms_of[dev], n, __ATOMIC_RELEASE);
  }
  *out = n;
  return VQ_OK;
}

size_t stream_ticket_bytes(long long rows) {
  return (static_cast<size_t>((rows + 15) / 16 + kMaxSegments) * sizeof(int) + 255) / 256 * 256;
}

size_t stream_workspace_bytes(long long rows, int batch) {
  return stream_ticket_bytes(rows) + static_cast<size_t>(kMaxStreamCtas) * 2 * kMaxSlabRows * batch * sizeof(float);
}

vq_status launch_gemm_tuned(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, void* ws,
                            size_t ws_bytes, cudaStream_t s) {
  vq_status st = VQ_ERR_UNSUPPORTED;
  if (g.cb_int4) {   // int4 codebooks: the 2-D shared-codebook kernels, else warp-private pair tables
    st = launch_gemm_blockcb(g, p, X, Y, batch, s);
    return st != VQ_ERR_UNSUPPORTED ? st : launch_gemm_warptab(g, p, X, Y, batch, s);
  }
#ifdef VQ_TUNING
  const char* path_env = getenv("VQ_PATH");
  const int path = path_env ? atoi(path_env) : 0;   // 1: persistent kernel only, 2: cluster kernels only
  if (path == 2) ws = nullptr;
#endif
  // Which family serves a single layer (measured on B200, both families on every benchmark shape at
  // batch 1 / 4 / 16): the persistent kernel wins on the per-row 4-bit 2-D layers of 8192 rows or more
  // (28672 x 8192: 26.7 against 37.8 us at batch 1, 66.5 against 77.6 us at batch 16; 8192 x 8192: 9.9
  // against 11.0 us and 22.9 against 26.2 us; 8192 x 28672: 30.3 against 32.5 us and 72.2 against 76.7 us);
  // at batch 8: 34.7 against 52.5, 13.8 against 17.8, 35.2 against 54.3 us); short layers of few slabs
  // (1024 x 8192: 6.8 against 5.2 us at batch 3) and the shared-codebook formats are faster in the cluster
  // kernels, whose K-split meets in distributed shared memory instead of the workspace.
  bool stream_first = g.b == 4 && g.d == 2 && g.N >= 8192;
#ifdef VQ_TUNING
  if (path == 1) stream_first = true;
#endif
  if (ws && stream_first) {   // (the persistent kernel needs the workspace)
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
    call.ws = ws;
    call.ws_bytes = ws_bytes;
    st = launch_gemm_stream(call, s);
    if (st != VQ_ERR_UNSUPPORTED) return st;
#ifdef VQ_TUNING
    if (path == 1) return st;
#endif
  }
  st = launch_gemm_blockcb(g, p, X, Y, batch, s);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  st = launch_gemm_rowcb(g, p, X, Y, batch, s);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  if (ws && !stream_first) {   // shapes the cluster kernels do not take: the persistent kernel if it does
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
    call.ws = ws;
    call.ws_bytes = ws_bytes;
    st = launch_gemm_stream(call, s);
    if (st != VQ_ERR_UNSUPPORTED) return st;
  }
  // small codebook blocks and the index widths no other family takes: warp-private pair tables
  return launch_gemm_warptab(g, p, X, Y, batch, s);
}


}  // namespace vq

// Number of in-kernel waits that ran out on the current device since the library was loaded
// (synchronises the device).  0 in a healthy run.
extern "C" vq_status vq_device_wait_failures(int* h_count) {
  if (!h_count) return VQ_ERR_NULL;
  int* d = nullptr;
  vq_status st = vq::device_error_counter(&d);
  if (st != VQ_OK) return st;
  if (cudaMemcpy(h_count, d, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return VQ_ERR_CUDA;
  return VQ_OK;
}
