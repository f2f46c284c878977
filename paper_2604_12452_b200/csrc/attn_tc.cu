// Tensor-core (tcgen05 / TMEM / TMA) attention kernels.  Placeholder until the kernels land:
// every shape reports "not supported" so that the dispatcher uses the scalar kernel.
#include "lca_common.cuh"

namespace lca {
bool attn_tc_supported(const AttnProblem&) { return false; }
size_t attn_tc_workspace_bytes(const AttnProblem&) { return 0; }
int attn_tc_launch(const AttnProblem&) { return LCA_ERR_UNSUPPORTED_SHAPE; }
int attn_tc_device_status(cudaStream_t stream) {
  return cudaStreamSynchronize(stream) == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}
}  // namespace lca
