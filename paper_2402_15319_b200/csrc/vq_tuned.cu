// Dispatch to the tuned kernel families.
#include "vq_common.cuh"

namespace vq {

vq_status launch_gemm_tuned(const Geometry& g, const LayerPtrs& p, const __half* X, __half* Y, int batch, float* ws,
                            cudaStream_t s) {
  (void)ws;
  vq_status st = launch_gemm_blockcb(g, p, X, Y, batch, s);
  if (st != VQ_ERR_UNSUPPORTED) return st;
  return launch_gemm_rowcb(g, p, X, Y, batch, s);
}

vq_status launch_decode_tuned(const Geometry&, const LayerPtrs&, __half*, cudaStream_t) {
  return VQ_ERR_UNSUPPORTED;
}

}  // namespace vq
