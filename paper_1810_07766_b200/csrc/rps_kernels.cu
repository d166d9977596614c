// CUDA kernels of the RPS step for sm_100a: the Philox drop-mask generator, the plain and
// gradient-averaging instantiations of the direct form of the fused local-SGD + masked-average +
// masked-write-back pass (rps_direct.cuh), and an off-path diagnostic reduction.  Host launch
// wrappers are at the bottom.
#include "rps_direct.cuh"

namespace rps {

// --------------------------------------------------------------------------
// Drop masks (Section 3: every message is lost independently with probability
// p).  One CTA per step of the window; warp w takes blocks j = w, w+8, ...; a
// lane takes workers i = lane and lane + 32 and the two directions of each, and
// __ballot_sync packs the outcomes into the mask words.
// --------------------------------------------------------------------------
__global__ void __launch_bounds__(256) rps_mask_kernel(const MaskParams prm)
{
    __shared__ int32_t server[kMaxWorkers];
    const uint64_t t = prm.t0 + blockIdx.x;
    const uint32_t t_lo = (uint32_t)t, t_hi = (uint32_t)(t >> 32);
    StepMasks* out = prm.out + blockIdx.x;
    const int n = prm.n;

    if (threadIdx.x < kMaxWorkers) server[threadIdx.x] = threadIdx.x;
    __syncthreads();
    if (prm.assign_perm && threadIdx.x == 0) {
        // Algorithm 1 draws the server of every block without replacement:
        // a Fisher-Yates shuffle, one Philox draw per position.
        for (int k = n - 1; k >= 1; --k) {
            const Philox4 r = philox4x32_10(t_lo, t_hi, (uint32_t)k, kStreamPerm, prm.key0, prm.key1);
            const int pick = (int)(((uint64_t)r.x * (uint64_t)(k + 1)) >> 32);
            const int32_t tmp = server[k];
            server[k] = server[pick];
            server[pick] = tmp;
        }
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    for (int j = warp; j < n; j += 8) {
        uint32_t up_half[2], down_half[2];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int i = lane + 32 * half;
            bool up_ok = false, down_ok = false;
            if (i < n) {
                const uint32_t which = ((uint32_t)j << 16) | (uint32_t)i;
                const Philox4 ru = philox4x32_10(t_lo, t_hi, which, kStreamUp, prm.key0, prm.key1);
                const Philox4 rd = philox4x32_10(t_lo, t_hi, which, kStreamDown, prm.key0, prm.key1);
                up_ok = !((uint64_t)ru.x < prm.drop_threshold);
                down_ok = !((uint64_t)rd.x < prm.drop_threshold);
                if (prm.self_delivery && i == server[j]) up_ok = down_ok = true;
            }
            up_half[half] = __ballot_sync(0xFFFFFFFFu, up_ok);
            down_half[half] = __ballot_sync(0xFFFFFFFFu, down_ok);
        }
        if (lane == 0) {
            const uint64_t up = (uint64_t)up_half[0] | ((uint64_t)up_half[1] << 32);
            uint64_t down = (uint64_t)down_half[0] | ((uint64_t)down_half[1] << 32);
            const int cnt = __popcll(up);
            if (cnt == 0) down = 0;  // nothing arrived: no average exists, nothing is broadcast
            out->up[j] = up;
            out->down[j] = down;
            out->cnt[j] = cnt;
            out->server[j] = server[j];
            out->inv_cnt[j] = cnt > 0 ? 1.0f / (float)cnt : 0.0f;
        }
    }
}

// --------------------------------------------------------------------------
// Diagnostics (off the hot path): squared distance of the mean model to the
// optimum mean_i(b_i) of the quadratic objective, and the consensus error
// sum_i ||x^(i) - xbar||^2 (the quantity Lemma 3 bounds).  fp64 accumulation.
// --------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ double widen(T v);
template <>
__device__ __forceinline__ double widen<float>(float v)
{
    return (double)v;
}
template <>
__device__ __forceinline__ double widen<__nv_bfloat16>(__nv_bfloat16 v)
{
    return (double)__bfloat162float(v);
}

template <typename T>
__global__ void __launch_bounds__(256) rps_diag_kernel(const DiagParams prm)
{
    const T* __restrict__ x = static_cast<const T*>(prm.x);
    const T* __restrict__ b = static_cast<const T*>(prm.b);
    double dist2 = 0.0, cons = 0.0;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < prm.d; c += (int64_t)gridDim.x * blockDim.x) {
        double xbar = 0.0, bbar = 0.0;
        for (int i = 0; i < prm.n; ++i) {
            xbar += widen<T>(x[(int64_t)i * prm.pitch + c]);
            bbar += widen<T>(b[(int64_t)i * prm.pitch + c]);
        }
        xbar /= prm.n;
        bbar /= prm.n;
        dist2 += (xbar - bbar) * (xbar - bbar);
        for (int i = 0; i < prm.n; ++i) {
            const double dev = widen<T>(x[(int64_t)i * prm.pitch + c]) - xbar;
            cons += dev * dev;
        }
    }
    __shared__ double part[2][8];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        dist2 += __shfl_xor_sync(0xFFFFFFFFu, dist2, off);
        cons += __shfl_xor_sync(0xFFFFFFFFu, cons, off);
    }
    if ((threadIdx.x & 31) == 0) {
        part[0][threadIdx.x >> 5] = dist2;
        part[1][threadIdx.x >> 5] = cons;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, k = 0.0;
        for (int w = 0; w < 8; ++w) a += part[0][w], k += part[1][w];
        atomicAdd(prm.out, a);
        atomicAdd(prm.out + 1, k);
    }
}

// --------------------------------------------------------------------------
// Monte-Carlo estimate of alpha_1 and alpha_2 (Eqs. 4 and 5) from generated drop masks.  For block j
// of one step let N be the set of workers whose copy arrived (c of them) and R the number of workers
// that receive the average.  Column k of W_t^(j) (Eq. 3) is the uniform average over N if k receives
// and the unit vector e_k otherwise, hence
//   (W W^T)[m][m']     = R [m in N][m' in N] / c^2 + [m = m'][m does not receive]
//   (W A_n W^T)[m][m'] = s_m s_m' / n,   s_m = R [m in N] / c + [m does not receive]   (row sums of W).
// Both matrices have all entries summing to n, so with their traces T the sample of
// alpha = (mean diagonal) - (mean off-diagonal) is T/n - (n - T)/(n (n - 1)).  One CTA per step,
// one thread per block; sums in fp64.
// --------------------------------------------------------------------------
__global__ void __launch_bounds__(kMaxWorkers) rps_alpha_kernel(const AlphaParams prm)
{
    const StepMasks* rec = prm.masks + blockIdx.x;
    const int n = prm.n;
    const int j = threadIdx.x;
    double a1 = 0.0, a2 = 0.0;
    if (j < n) {
        const uint64_t up = rec->up[j], down = rec->down[j];
        const int c = rec->cnt[j];
        const int receivers = __popcll(down);
        const double share = c > 0 ? (double)receivers / (double)c : 0.0;  // R / c; no average exists when c = 0
        const double trace1 = share + (double)(n - receivers);
        const int in_and_recv = __popcll(up & down);     // s = R/c
        const int in_not_recv = __popcll(up & ~down);    // s = R/c + 1
        const int out_not_recv = n - __popcll(up | down);  // s = 1 (outside N and receiving: s = 0)
        const double trace2 =
            ((double)in_and_recv * share * share + (double)in_not_recv * (share + 1.0) * (share + 1.0) +
             (double)out_not_recv) / (double)n;
        const double off = 1.0 / ((double)n * (double)(n - 1));
        a1 = trace1 / n - ((double)n - trace1) * off;
        a2 = trace2 / n - ((double)n - trace2) * off;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a1 += __shfl_xor_sync(0xFFFFFFFFu, a1, o);
        a2 += __shfl_xor_sync(0xFFFFFFFFu, a2, o);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(prm.out, a1);
        atomicAdd(prm.out + 1, a2);
    }
}

// --------------------------------------------------------------------------
// Launch wrappers
// --------------------------------------------------------------------------
cudaError_t launch_alpha(const AlphaParams& prm, int steps, cudaStream_t stream)
{
    rps_alpha_kernel<<<steps, kMaxWorkers, 0, stream>>>(prm);
    return cudaGetLastError();
}

cudaError_t launch_masks(const MaskParams& prm, int steps, cudaStream_t stream)
{
    rps_mask_kernel<<<steps, 256, 0, stream>>>(prm);
    return cudaGetLastError();
}

namespace {

template <typename T, int VEC>
cudaError_t launch_direct_for_n(const FusedParams& prm, int wpt, int sm_count, cudaStream_t stream, bool overlap)
{
    const int n = prm.n;
    // the gradient-averaging comparison is built in one family of lane shapes only
    if (prm.average_gradients) return launch_direct_light<T, VEC, true, false>(prm, sm_count, stream, overlap);
    if (wpt == 4) {
        if (n <= 4) return launch_direct_as<T, VEC, 4, 1>(prm, sm_count, stream, overlap);
        if (n <= 8) return launch_direct_as<T, VEC, 4, 2>(prm, sm_count, stream, overlap);
        if (n <= 16) return launch_direct_as<T, VEC, 4, 4>(prm, sm_count, stream, overlap);
        if (n <= 32) return launch_direct_as<T, VEC, 4, 8>(prm, sm_count, stream, overlap);
        return launch_direct_as<T, VEC, 4, 16>(prm, sm_count, stream, overlap);
    }
    if (n <= 2) return launch_direct_as<T, VEC, 2, 1>(prm, sm_count, stream, overlap);
    if (n <= 4) return launch_direct_as<T, VEC, 4, 1>(prm, sm_count, stream, overlap);
    if (n <= 8) return launch_direct_as<T, VEC, 8, 1>(prm, sm_count, stream, overlap);
    if (n <= 16) return launch_direct_as<T, VEC, 8, 2>(prm, sm_count, stream, overlap);
    if (n <= 32) return launch_direct_as<T, VEC, 8, 4>(prm, sm_count, stream, overlap);
    return launch_direct_as<T, VEC, 8, 8>(prm, sm_count, stream, overlap);
}

}  // namespace

cudaError_t launch_fused_direct(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream)
{
    if (prm.trace != nullptr) return launch_direct_tracked(prm, bf16, sm_count, stream);
    const bool overlap = tune.launch_overlap != 1;  // programmatic stream serialization unless plain launches are asked for
    if (bf16) return launch_direct_for_n<__nv_bfloat16, 8>(prm, tune.workers_per_lane, sm_count, stream, overlap);
    return launch_direct_for_n<float, 4>(prm, tune.workers_per_lane, sm_count, stream, overlap);
}

namespace {

enum class FusedKernel { kDirect, kStaged, kRing, kStream };

// Which form of the fused step runs: the one asked for where it is built for this step, else the library's choice.
FusedKernel choose_fused_kernel(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count)
{
    if (tune.kernel == 1) return FusedKernel::kDirect;
    if (tune.kernel == 3 && ring_kernel_covers(prm, bf16)) return FusedKernel::kRing;
    if (tune.kernel == 4 && stream_kernel_covers(prm, bf16)) return FusedKernel::kStream;
    if (tune.kernel == 0) {
        // A model this short gives the staged kernel's ring less than a tile per SM: there
        // is nothing to pipeline and its set-up dominates; the step is launch bound and L2 resident.
        const int64_t bytes_per_column = (int64_t)prm.n * (bf16 ? 2 : 4);
        if (prm.d * bytes_per_column < (int64_t)sm_count * 8192) return FusedKernel::kDirect;
    }
    // Workers streamed through the teams' rings (what is staged does not grow with n, every row piece is 2 KB).  The
    // lane groups of the staged and ring kernels hold 4 or 8 workers per lane times a power of two of lanes, so a
    // worker count between two powers of two runs at the speed of the next one; the streamed kernel's time is
    // proportional to n.  Measured side by side (ms per step, bf16 d = 16.8 M / fp32 d = 4 M; lane-group form first):
    //   bf16 plain   n = 8 0.126 / 0.128, 16 0.247 / 0.247, 32 0.489 / 0.499; 2 0.079 / 0.048, 4 0.099 / 0.073,
    //                6 0.125 / 0.111, 12 0.247 / 0.193, 20 0.489 / 0.322, 28 0.488 / 0.456, 48 1.33x, 64 0.95x
    //   bf16 tracked streamed ahead at every n from 2 (0.092 / 0.061) to 64 (1.62 / 1.16)
    //   fp32         n = 8, 16, 32 staged ahead by 2-9 %; 12 0.100 / 0.083, 20 0.187 / 0.146, 24 0.199 / 0.178,
    //                48 0.418 / 0.364, tracked and gradient averaging likewise; at d = 25.6 M: 2 0.147 / 0.105
    //                (tracked 0.166 / 0.130), 4 0.181 / 0.190 (tracked 0.213 / 0.193), 12 0.609 / 0.579
    // Gradient averaging reads x twice in this form, part of it from DRAM again when n is large (n = 64: 1.25 ms
    // against 1.18 for the ring kernel, which holds the tile), so there it is taken only where the ring kernel's
    // lane groups are at most four fifths full: 10 0.269 / 0.225, 12 0.269 / 0.256, 20 0.546 / 0.422,
    // 24 0.548 / 0.499, 28 0.548 / 0.581, 40 1.115 / 0.826, 48 1.12 / 0.98, 56 1.155 / 1.173; and below 5 workers,
    // which the ring kernel does not take (4 0.105 / 0.092).
    if (tune.kernel == 0 && stream_kernel_covers(prm, bf16) && tune.workers_per_lane == 0 && tune.copy_mode == 0 &&
        tune.slice_bytes == 0) {
        const int n = prm.n;
        const bool power_of_two = (n & (n - 1)) == 0;
        int padded = 8;  // what the ring kernel's lane groups pad n to
        while (padded < n) padded *= 2;
        bool streamed;
        if (!bf16) streamed = !power_of_two || (!prm.average_gradients && (n == 2 || (n == 4 && prm.trace != nullptr)));
        else if (prm.trace != nullptr) streamed = true;
        else if (prm.average_gradients) streamed = n < 5 || (n >= 9 && 5 * n <= 4 * padded);
        else streamed = !power_of_two || n > 32 || n < 8;
        if (streamed) return FusedKernel::kStream;
    }
    // bf16 replicas of more than 4 workers: the self-refilling ring (16 compute warps, no producer warp), unless an
    // option that shapes the staged kernel only was set.  Measured side by side it is 3-8 % ahead at every n.
    if (tune.kernel == 0 && bf16 && ring_kernel_covers(prm, bf16) && tune.workers_per_lane == 0 &&
        tune.consumer_warps == 0 && tune.copy_mode == 0 && tune.slice_bytes == 0)
        return FusedKernel::kRing;
    return FusedKernel::kStaged;
}

}  // namespace

cudaError_t launch_fused(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                         cudaStream_t stream)
{
    switch (choose_fused_kernel(prm, tune, bf16, sm_count)) {
        case FusedKernel::kDirect: return launch_fused_direct(prm, tune, bf16, sm_count, stream);
        case FusedKernel::kRing: return launch_fused_ring(prm, tune, bf16, sm_count, stream);
        case FusedKernel::kStream: return launch_fused_stream(prm, tune, bf16, sm_count, stream);
        default: return launch_fused_staged(prm, tune, bf16, sm_count, stream);
    }
}

bool fused_steps_supported(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count)
{
    // untracked steps of the streamed kernel: its teams go from step to step on their own tiles
    return prm.trace == nullptr && choose_fused_kernel(prm, tune, bf16, sm_count) == FusedKernel::kStream;
}

cudaError_t launch_fused_steps(const FusedParams& prm, const FusedTuning& tune, int steps, bool bf16, int sm_count,
                               cudaStream_t stream)
{
    if (!fused_steps_supported(prm, tune, bf16, sm_count)) return cudaErrorInvalidConfiguration;
    return launch_fused_stream(prm, tune, bf16, sm_count, stream, steps);
}

void set_philox_key(FusedParams& prm, uint64_t seed)
{
    prm.key0 = (uint32_t)seed;
    prm.key1 = (uint32_t)(seed >> 32);
    for (uint32_t r = 0; r < 10; ++r) {
        prm.round_key[r][0] = prm.key0 + r * 0x9E3779B9u;
        prm.round_key[r][1] = prm.key1 + r * 0xBB67AE85u;
    }
}

void set_sgd_scalars(FusedParams& prm, float gamma, float sigma)
{
    prm.gamma = gamma;
    const double gs = (double)gamma * (double)sigma;
    prm.noise_scale = (float)(-2.0 * 0.6931471805599453 * gs * gs);
    prm.noisy = sigma != 0.0f;
}

cudaError_t launch_diag(const DiagParams& prm, bool bf16, int sm_count, cudaStream_t stream)
{
    int64_t grid = (prm.d + 255) / 256;
    if (grid > (int64_t)sm_count * 8) grid = (int64_t)sm_count * 8;
    if (bf16)
        rps_diag_kernel<__nv_bfloat16><<<(unsigned)grid, 256, 0, stream>>>(prm);
    else
        rps_diag_kernel<float><<<(unsigned)grid, 256, 0, stream>>>(prm);
    return cudaGetLastError();
}

}  // namespace rps
