// Instantiations of the fused decode-step kernel for the bf16 state store.
#include "ssdq_update.cuh"
#include "ssdq_mamba1.cuh"

namespace ssdq {
cudaError_t launch_update_bf16(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s) {
    return launch_update_fmt<FMT_BF16>(p, rule, a_per_state, s);
}
}  // namespace ssdq
