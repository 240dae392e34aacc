// Instantiations of the fused decode-step kernel for the e4m3 state store.
#include "ssdq_stream.cuh"
#include "ssdq_mamba1.cuh"
#include "ssdq_headscale.cuh"

namespace ssdq {
cudaError_t launch_update_e4m3(const UpdateParams& p, int rule, bool a_per_state, cudaStream_t s) {
    return launch_update_fmt<FMT_E4M3>(p, rule, a_per_state, s);
}
}  // namespace ssdq
