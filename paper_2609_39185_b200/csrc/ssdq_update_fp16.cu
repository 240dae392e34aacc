// Instantiations of the fused decode-step kernel for the fp16 state store.
#include "ssdq_update.cuh"
#include "ssdq_mamba1.cuh"

namespace ssdq {
cudaError_t launch_update_fp16(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s) {
    return launch_update_fmt<FMT_FP16>(p, rule, a_per_state, s);
}
}  // namespace ssdq
