// Instantiations of the fused decode-step kernel for the symmetric block-absmax integer stores (INT8/7/6/4 in an
// int8 container; q_max is a run-time parameter).
#include "ssdq_stream.cuh"
#include "ssdq_mamba1.cuh"
#include "ssdq_headscale.cuh"

namespace ssdq {
cudaError_t launch_update_int8(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s) {
    return launch_update_fmt<FMT_INT>(p, rule, a_per_state, s);
}
}  // namespace ssdq
