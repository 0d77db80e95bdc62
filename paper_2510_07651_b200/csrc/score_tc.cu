// Tensor-core (tcgen05 + TMA) score kernels.  Placeholder until the kernels land: no shape
// qualifies, so obc_score always takes the CUDA-core path and OBC_PATH_TC is rejected.
#include "obc_common.cuh"

namespace obc {
bool tc_supported(const ScoreShape&, int) { return false; }
size_t tc_workspace_bytes(const ScoreShape&) { return 0; }
obc_status launch_score_tc(const ScoreShape&, TensorView, TensorView, TensorView, float*, void*, cudaStream_t) {
    return OBC_ERR_UNSUPPORTED;
}
}  // namespace obc
