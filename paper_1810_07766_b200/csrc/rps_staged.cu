// Fused RPS step, staged form: the plain instantiations (every lane shape) and the dispatch to
// the groups built elsewhere.  The kernel itself is in rps_staged.cuh.
#include "rps_staged.cuh"

namespace rps {

namespace {

template <typename T, int VEC>
cudaError_t launch_staged_for_n(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    const int n = prm.n;
    // workers per lane: asked for, or 8 where that halves the shuffle stages and pays for its
    // registers (bf16 replicas, or more than 8 workers), else 4
    int wpt = tune.workers_per_lane;
    if (wpt == 0) wpt = (n > 4 && (sizeof(T) == 2 || n > 8)) ? 8 : 4;
    if (wpt == 8) {
        if (n <= 8) return launch_staged_as<T, VEC, 8, 1>(prm, tune, sm_count, stream);
        if (n <= 16) return launch_staged_as<T, VEC, 8, 2>(prm, tune, sm_count, stream);
        if (n <= 32) return launch_staged_as<T, VEC, 8, 4>(prm, tune, sm_count, stream);
        return launch_staged_as<T, VEC, 8, 8>(prm, tune, sm_count, stream);
    }
    if (wpt == 2) {
        if (n <= 2) return launch_staged_as<T, VEC, 2, 1>(prm, tune, sm_count, stream);
        if (n <= 4) return launch_staged_as<T, VEC, 2, 2>(prm, tune, sm_count, stream);
        if (n <= 8) return launch_staged_as<T, VEC, 2, 4>(prm, tune, sm_count, stream);
        if (n <= 16) return launch_staged_as<T, VEC, 2, 8>(prm, tune, sm_count, stream);
        if (n <= 32) return launch_staged_as<T, VEC, 2, 16>(prm, tune, sm_count, stream);
        return launch_staged_as<T, VEC, 4, 16>(prm, tune, sm_count, stream);
    }
    if (n <= 2) return launch_staged_as<T, VEC, 2, 1>(prm, tune, sm_count, stream);
    if (n <= 4) return launch_staged_as<T, VEC, 4, 1>(prm, tune, sm_count, stream);
    if (n <= 8) return launch_staged_as<T, VEC, 4, 2>(prm, tune, sm_count, stream);
    if (n <= 16) return launch_staged_as<T, VEC, 4, 4>(prm, tune, sm_count, stream);
    if (n <= 32) return launch_staged_as<T, VEC, 4, 8>(prm, tune, sm_count, stream);
    return launch_staged_as<T, VEC, 4, 16>(prm, tune, sm_count, stream);
}

}  // namespace

cudaError_t launch_fused_staged(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream)
{
    // TMA coordinates are 32-bit: rows of 2^31 elements or more go through the direct kernel
    if (prm.pitch >= ((int64_t)1 << 31)) return launch_fused_direct(prm, tune, bf16, sm_count, stream);
    // the optional forms are built in one family of lane shapes, each group in a file of its own
    if (prm.trace != nullptr) return launch_staged_tracked(prm, tune, bf16, sm_count, stream);
    if (prm.average_gradients) return launch_staged_gradavg(prm, tune, bf16, sm_count, stream);
    if (bf16 && tune.slice_bytes == 8) {
        // narrow bf16 slices exist for 8 workers per lane only
        const int n = prm.n;
        if (n <= 8) return launch_staged_as<__nv_bfloat16, 4, 8, 1>(prm, tune, sm_count, stream);
        if (n <= 16) return launch_staged_as<__nv_bfloat16, 4, 8, 2>(prm, tune, sm_count, stream);
        if (n <= 32) return launch_staged_as<__nv_bfloat16, 4, 8, 4>(prm, tune, sm_count, stream);
        return launch_staged_as<__nv_bfloat16, 4, 8, 8>(prm, tune, sm_count, stream);
    }
    if (bf16) return launch_staged_for_n<__nv_bfloat16, 8>(prm, tune, sm_count, stream);
    return launch_staged_for_n<float, 4>(prm, tune, sm_count, stream);
}

}  // namespace rps
