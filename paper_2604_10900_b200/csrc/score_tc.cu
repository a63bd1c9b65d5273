// Tensor-core scoring path (tcgen05 + TMA).  Placeholder until the kernels land: reports
// "shape not supported" so that every call takes the SIMT kernels.
#include "cask_internal.cuh"

namespace cask {

bool score_tc_supported(const Launch&) { return false; }

cudaError_t launch_score_tc(const Launch&, const float*, float*, float*, Workspace&, void*) {
    return cudaErrorNotSupported;
}

}  // namespace cask
