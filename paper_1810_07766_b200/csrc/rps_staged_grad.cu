// Fused RPS step, staged form: the gradient-averaging instantiations (Section 5's comparison).
#include "rps_staged.cuh"

namespace rps {

cudaError_t launch_staged_gradavg(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                  cudaStream_t stream)
{
    if (bf16) return launch_staged_light<__nv_bfloat16, 8, true, false>(prm, tune, sm_count, stream);
    return launch_staged_light<float, 4, true, false>(prm, tune, sm_count, stream);
}

}  // namespace rps
