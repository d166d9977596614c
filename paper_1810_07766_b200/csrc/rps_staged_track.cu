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
    if (bf16 && prm.n > 8 && tune.workers_per_lane != 4) {
        if (prm.n <= 16) return launch_staged_as<__nv_bfloat16, 8, 8, 2, false, true>(prm, tune, sm_count, stream);
        if (prm.n <= 32) return launch_staged_as<__nv_bfloat16, 8, 8, 4, false, true>(prm, tune, sm_count, stream);
        return launch_staged_as<__nv_bfloat16, 8, 8, 8, false, true>(prm, tune, sm_count, stream);
    }
    if (bf16) return launch_staged_light<__nv_bfloat16, 8, false, true>(prm, tune, sm_count, stream);
    // model averaging with more than 4 workers (bf16: more than 8): 8 workers per lane, which halves the
    // butterfly stages of the three reductions a tracked step makes per column (none are left at n <= 8)
    if (prm.n > 4 && tune.workers_per_lane != 4) {
        if (prm.n <= 8) return launch_staged_as<float, 4, 8, 1, false, true>(prm, tune, sm_count, stream);
        if (prm.n <= 16) return launch_staged_as<float, 4, 8, 2, false, true>(prm, tune, sm_count, stream);
        if (prm.n <= 32) return launch_staged_as<float, 4, 8, 4, false, true>(prm, tune, sm_count, stream);
        return launch_staged_as<float, 4, 8, 8, false, true>(prm, tune, sm_count, stream);
    }
    return launch_staged_light<float, 4, false, true>(prm, tune, sm_count, stream);
}

}  // namespace rps
