// Fused RPS step, staged form: the tracked instantiations (distance to the optimum and consensus
// error as a by-product of the pass), for model averaging and for gradient averaging.
#include "rps_staged.cuh"

namespace rps {

cudaError_t launch_staged_tracked(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                  cudaStream_t stream)
{
    if (prm.average_gradients) {
        if (bf16) return launch_staged_light<__nv_bfloat16, 8, true, true>(prm, tune, sm_count, stream);
        return launch_staged_light<float, 4, true, true>(prm, tune, sm_count, stream);
    }
    if (bf16) return launch_staged_light<__nv_bfloat16, 8, false, true>(prm, tune, sm_count, stream);
    return launch_staged_light<float, 4, false, true>(prm, tune, sm_count, stream);
}

}  // namespace rps
