// Several consecutive RPS steps in one pass over x and b (temporal blocking).  Columns never interact
// and, with the quadratic objective, the gradient of a column needs only that column, so a lane can keep its
// slices of x and b in registers, run step t, t+1, ... t+S-1 on them (each with its own drop masks and its
// own noise, each rounding x to the replica type as the store of a single step would) and write x once.
// HBM traffic per step falls to 1/S of the single-step kernel's; the pass is bound by the arithmetic of the
// gradient noise instead.  The arithmetic of one step is the code the single-step kernels run
// (rps_device.cuh), in the lane shape with 4 workers per lane, so the result equals S single steps bit
// for bit.  Not Algorithm 1's setting (a real model's gradient sits between two synchronisations); it is an
// option of rps_step_n (rps_options.block_steps), off by default.
#include "rps_kernels.h"

#include "rps_device.cuh"

namespace rps {

namespace {

// 256 threads; three CTAs per SM for fp32 replicas (80 registers), two for bf16 (a lane holds twice the columns)
constexpr int kBlockedThreads = 256;

template <typename T, int VEC, int WPT, int G>
__global__ void __launch_bounds__(kBlockedThreads, sizeof(T) == 4 ? 3 : 2)
    rps_fused_blocked_kernel(const FusedParams prm, const int steps)
{
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    const int lane = threadIdx.x & 31;
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;  // first worker of this lane's group
    const int n = prm.n;
    T* __restrict__ x = static_cast<T*>(prm.x);
    const T* __restrict__ b = static_cast<const T*>(prm.b);

    const int64_t warps_total = (int64_t)gridDim.x * (kBlockedThreads / 32);
    const int64_t tiles = (prm.d + WARP_COLS - 1) / WARP_COLS;
    const uint64_t t0 = ((uint64_t)prm.t_hi << 32) | prm.t_lo;
    BlockCursor cursor;
    for (int64_t tile = (int64_t)blockIdx.x * (kBlockedThreads / 32) + (threadIdx.x >> 5); tile < tiles;
         tile += warps_total) {
        const int64_t c = tile * WARP_COLS + (int64_t)sub * VEC;
        const bool col_live = c < prm.d;
        const int64_t c_read = col_live ? c : 0;  // lanes past the end read a real slice; it is never stored

        float v[WPT][VEC], bv[WPT][VEC];
#pragma unroll
        for (int w = 0; w < WPT; ++w) {
            const int row = w_first + w < n ? w_first + w : n - 1;  // workers past n: masked out, never stored
            const int64_t at = (int64_t)row * prm.pitch + c_read;
            using Raw = typename RowVec<T, VEC>::Raw;
            RowVec<T, VEC>::unpack(__ldcs(reinterpret_cast<const Raw*>(x + at)), v[w]);
            RowVec<T, VEC>::unpack(__ldcs(reinterpret_cast<const Raw*>(b + at)), bv[w]);
        }
        uint32_t live_bits = 0;
#pragma unroll 1
        for (int s = 0; s < steps; ++s) {
            const StepMasks* rec = prm.masks + s;
            const MaskView masks{rec->up, rec->down, rec->inv_cnt};
            const uint64_t t = t0 + (uint64_t)s;
            // local SGD step, as local_sgd() evaluates it: v = x + gamma * (b - x) - (gamma * sigma) * xi
#pragma unroll
            for (int w = 0; w < WPT; ++w)
#pragma unroll
                for (int e = 0; e < VEC; ++e) v[w][e] = fmaf(prm.gamma, bv[w][e] - v[w][e], v[w][e]);
            if (prm.noisy) add_gradient_noise<VEC, WPT>(v, c, w_first, prm, (uint32_t)t, (uint32_t)(t >> 32));
            live_bits = average_and_select<VEC, WPT, G>(v, c, col_live, w_first, masks, cursor, prm);
            // what a single step would have stored and the next one read back
#pragma unroll
            for (int w = 0; w < WPT; ++w) as_stored<T, VEC>(v[w]);
        }
        T* dst = x + (int64_t)w_first * prm.pitch + c;
        if (live_bits == (1u << VEC) - 1u) {
#pragma unroll
            for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                if (w_first + w < n)
                    __stcs(reinterpret_cast<typename RowVec<T, VEC>::Raw*>(dst), RowVec<T, VEC>::pack(v[w]));
        } else if (live_bits != 0) {
#pragma unroll
            for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                if (w_first + w < n) store_ragged<T, VEC>(dst, v[w], live_bits);
        }
    }
}

template <typename T, int VEC, int WPT, int G>
cudaError_t launch_blocked_as(const FusedParams& prm, int steps, int sm_count, cudaStream_t stream)
{
    constexpr int warp_cols = (32 / G) * VEC;
    const int64_t tiles = (prm.d + warp_cols - 1) / warp_cols;
    const int64_t ctas_needed = (tiles + kBlockedThreads / 32 - 1) / (kBlockedThreads / 32);
    static LaunchState state;  // of this instantiation, per device
    int per_sm = 1;                // resident CTAs per SM, asked once per device
    cudaError_t err = resident_ctas_per_sm(state, rps_fused_blocked_kernel<T, VEC, WPT, G>, kBlockedThreads, 0, &per_sm);
    if (err != cudaSuccess) return err;
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > ctas_needed) grid = ctas_needed;
    if (grid < 1) grid = 1;
    rps_fused_blocked_kernel<T, VEC, WPT, G><<<(unsigned)grid, kBlockedThreads, 0, stream>>>(prm, steps);
    return cudaGetLastError();
}

template <typename T, int VEC>
cudaError_t launch_blocked_for_n(const FusedParams& prm, int steps, int sm_count, cudaStream_t stream)
{
    const int n = prm.n;
    if (n <= 2) return launch_blocked_as<T, VEC, 2, 1>(prm, steps, sm_count, stream);
    if (n <= 4) return launch_blocked_as<T, VEC, 4, 1>(prm, steps, sm_count, stream);
    if (n <= 8) return launch_blocked_as<T, VEC, 4, 2>(prm, steps, sm_count, stream);
    if (n <= 16) return launch_blocked_as<T, VEC, 4, 4>(prm, steps, sm_count, stream);
    if (n <= 32) return launch_blocked_as<T, VEC, 4, 8>(prm, steps, sm_count, stream);
    return launch_blocked_as<T, VEC, 4, 16>(prm, steps, sm_count, stream);
}

}  // namespace

cudaError_t launch_fused_blocked(const FusedParams& prm, int steps, bool bf16, int sm_count, cudaStream_t stream)
{
    if (bf16) return launch_blocked_for_n<__nv_bfloat16, 8>(prm, steps, sm_count, stream);
    return launch_blocked_for_n<float, 4>(prm, steps, sm_count, stream);
}

}  // namespace rps
