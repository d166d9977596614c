// Fused RPS step, staged form: the gradient-averaging instantiations (Section 5's comparison).
#include "rps_staged.cuh"

namespace rps {

cudaError_t launch_staged_gradavg(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                  cudaStream_t stream)
{
    if (bf16) return launch_staged_light<__nv_bfloat16, 8, true, false>(prm, tune, sm_count, stream);
    // fp32 with more than 8 workers: 8 workers per lane, as the plain step (its in-place store mode holds the
    // stage until the results are written anyway, which is what reading x a second time needs)
    if (prm.n > 8 && tune.workers_per_lane != 4) {
        if (prm.n <= 16) return launch_staged_as<float, 4, 8, 2, true, false>(prm, tune, sm_count, stream);
        if (prm.n <= 32) return launch_staged_as<float, 4, 8, 4, true, false>(prm, tune, sm_count, stream);
        return launch_staged_as<float, 4, 8, 8, true, false>(prm, tune, sm_count, stream);
    }
    return launch_staged_light<float, 4, true, false>(prm, tune, sm_count, stream);
}

}  // namespace rps
