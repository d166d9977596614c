// Fused RPS step, direct form: the tracked instantiations (distance to the optimum and consensus
// error as a by-product of the pass), for model averaging and for gradient averaging.
#include "rps_direct.cuh"

namespace rps {

cudaError_t launch_direct_tracked(const FusedParams& prm, bool bf16, int sm_count, cudaStream_t stream)
{
    if (prm.average_gradients) {
        if (bf16) return launch_direct_light<__nv_bfloat16, 8, true, true>(prm, sm_count, stream);
        return launch_direct_light<float, 4, true, true>(prm, sm_count, stream);
    }
    if (bf16) return launch_direct_light<__nv_bfloat16, 8, false, true>(prm, sm_count, stream);
    return launch_direct_light<float, 4, false, true>(prm, sm_count, stream);
}

}  // namespace rps
