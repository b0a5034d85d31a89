// Tensor-core scoring path (placeholder until the tcgen05 kernels land).
#include "refree_internal.cuh"
namespace refree {
bool score_tc_supported(const refree_params &) { return false; }
cudaError_t launch_score_tc(const refree_params &, const void *, const void *, const int32_t *, const int32_t *,
                            int64_t, float *, char *, const Workspace &, int32_t *, cudaStream_t)
{
    return cudaErrorNotSupported;
}
}  // namespace refree
