// Tuned kernels for the benchmark format families (placeholder dispatch: none yet).
#include "vq_common.cuh"

namespace vq {

vq_status launch_gemm_tuned(const Geometry&, const LayerPtrs&, const __half*, __half*, int, float*, cudaStream_t) {
  return VQ_ERR_UNSUPPORTED;
}

vq_status launch_decode_tuned(const Geometry&, const LayerPtrs&, __half*, cudaStream_t) {
  return VQ_ERR_UNSUPPORTED;
}

}  // namespace vq
