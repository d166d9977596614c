// Fused RPS step, direct form (sm_100a): the kernel template and its launch; the translation
// units that include this header each build one group of instantiations.
#pragma once

#include "rps_kernels.h"

#include "rps_device.cuh"

namespace rps {

namespace {

// --------------------------------------------------------------------------
// Fused step, direct form: every lane loads its row slices straight from global
// memory into registers.  A warp owns LPG * VEC consecutive columns per
// iteration; its 32 lanes are G groups of LPG = 32 / G lanes.  Group g handles
// workers g*WPT .. g*WPT + WPT - 1, lane `sub` of a group handles VEC consecutive
// columns of each of those workers with one 16-byte load per row, so a group
// reads whole contiguous row segments.  x is read once and written once, b is
// read once.  (The staged form in rps_staged.cu does the same arithmetic with
// the loads decoupled from the warps through shared memory.)
// --------------------------------------------------------------------------
template <typename T, int VEC, int WPT, int G, int THREADS, bool GRAD, bool DIAG>
__global__ void __launch_bounds__(THREADS) rps_fused_direct_kernel(const FusedParams prm)
{
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    const int lane = threadIdx.x & 31;
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;  // first worker of this lane's group
    const int n = prm.n;
    T* __restrict__ x = static_cast<T*>(prm.x);
    const T* __restrict__ b = static_cast<const T*>(prm.b);
    const MaskView masks{prm.masks->up, prm.masks->down, prm.masks->inv_cnt};
    // Launched with programmatic stream serialization this CTA may have been placed while the kernel before
    // it in the stream was still running: let the kernel after this one do the same, then wait for the one
    // before to complete (its writes visible) before reading anything from global memory.  At the sizes this
    // kernel serves a step is as long as a launch, so hiding the launch is most of what there is to gain.
    // Both are no-ops in a plain launch.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int64_t warps_total = (int64_t)gridDim.x * (THREADS / 32);
    const int64_t tiles = (prm.d + WARP_COLS - 1) / WARP_COLS;
    BlockCursor cursor;
    // tracked steps: the CTA's pair of sums and the count of warps that have added theirs
    __shared__ double track_pair[2];
    __shared__ int track_arrivals;
    Tracker<VEC, WPT, G> tracker;
    const uint32_t present = Tracker<VEC, WPT, G>::present_workers(w_first, n);
    if (DIAG) {
        if (threadIdx.x == 0) {
            track_pair[0] = 0.0;
            track_pair[1] = 0.0;
            track_arrivals = 0;
        }
        __syncthreads();
    }
    // odd steps take the tiles from the last to the first: a step starts on the columns that the step
    // before it touched last, which are still in L2
    const bool descending = prm.descending != 0;
    for (int64_t turn = (int64_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5); turn < tiles;
         turn += warps_total) {
        const int64_t tile = descending ? tiles - 1 - turn : turn;
        const int64_t c = tile * WARP_COLS + (int64_t)sub * VEC;
        const bool col_live = c < prm.d;  // the row pitch covers the whole slice even when c + VEC > d

        float v[WPT][VEC];
        {
            float xv[WPT][VEC], bv[WPT][VEC];
            // lanes past the end of the row and workers past n read a real slice all the same (column
            // 0 / the last row): their values are masked out and never stored
            const int64_t c_read = col_live ? c : 0;
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                const int row = w_first + w < n ? w_first + w : n - 1;
                const int64_t at = (int64_t)row * prm.pitch + c_read;
                using Raw = typename RowVec<T, VEC>::Raw;
                const Raw raw_x = __ldcs(reinterpret_cast<const Raw*>(x + at));
                const Raw raw_b = __ldcs(reinterpret_cast<const Raw*>(b + at));
                RowVec<T, VEC>::unpack(raw_x, xv[w]);
                RowVec<T, VEC>::unpack(raw_b, bv[w]);
            }
            if (DIAG) tracker.targets(bv, present);
            local_sgd<VEC, WPT, GRAD>(xv, bv, v, c, w_first, prm);
        }
        const uint32_t live_bits = average_and_select<VEC, WPT, G>(v, c, col_live, w_first, masks, cursor, prm);
        if (GRAD) {
            // v holds the update each worker applies (the average one where it arrived): x_{t+1} = x + update
            const int64_t c_read = col_live ? c : 0;
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                const int row = w_first + w < n ? w_first + w : n - 1;
                float xv[VEC];
                RowVec<T, VEC>::unpack(__ldcs(reinterpret_cast<const typename RowVec<T, VEC>::Raw*>(
                                           x + (int64_t)row * prm.pitch + c_read)),
                                       xv);
#pragma unroll
                for (int e = 0; e < VEC; ++e) v[w][e] += xv[e];
            }
        }
        if (DIAG) {
#pragma unroll
            for (int w = 0; w < WPT; ++w) as_stored<T, VEC>(v[w]);
            tracker.models(v, present, live_bits, prm.inv_n);
        }
        T* dst = x + (int64_t)w_first * prm.pitch + c;  // this lane's slice of its first worker's row
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
    if (DIAG) tracker.flush(track_pair, &track_arrivals, THREADS / 32, prm.trace);
}

constexpr int kThreads = 256;

template <typename T, int VEC, int WPT, int G, bool GRAD = false, bool DIAG = false>
cudaError_t launch_direct_as(const FusedParams& prm, int sm_count, cudaStream_t stream, bool overlap = true)
{
    constexpr int warp_cols = (32 / G) * VEC;
    const int64_t tiles = (prm.d + warp_cols - 1) / warp_cols;
    const int64_t ctas_needed = (tiles + kThreads / 32 - 1) / (kThreads / 32);
    static LaunchState state;  // of this instantiation, per device
    int per_sm = 1;                // resident CTAs per SM, asked once per device
    cudaError_t err = resident_ctas_per_sm(state, rps_fused_direct_kernel<T, VEC, WPT, G, kThreads, GRAD, DIAG>,
                                           kThreads, 0, &per_sm);
    if (err != cudaSuccess) return err;
    // a whole number of waves of resident CTAs, each striding over the tiles
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > ctas_needed) grid = ctas_needed;
    if (grid < 1) grid = 1;
    if (overlap) {
        cudaLaunchConfig_t config = {};
        config.gridDim = dim3((unsigned)grid);
        config.blockDim = dim3(kThreads);
        config.dynamicSmemBytes = 0;
        config.stream = stream;
        cudaLaunchAttribute attribute[1];
        attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attribute[0].val.programmaticStreamSerializationAllowed = 1;
        config.attrs = attribute;
        config.numAttrs = 1;
        return cudaLaunchKernelEx(&config, rps_fused_direct_kernel<T, VEC, WPT, G, kThreads, GRAD, DIAG>, prm);
    }
    rps_fused_direct_kernel<T, VEC, WPT, G, kThreads, GRAD, DIAG><<<(unsigned)grid, kThreads, 0, stream>>>(prm);
    return cudaGetLastError();
}

// The one family of lane shapes (4 workers per lane, 2 for n <= 2) in which the optional forms of the
// step (gradient averaging, tracking) are built.
template <typename T, int VEC, bool GRAD, bool DIAG>
cudaError_t launch_direct_light(const FusedParams& prm, int sm_count, cudaStream_t stream, bool overlap = true)
{
    const int n = prm.n;
    if (n <= 2) return launch_direct_as<T, VEC, 2, 1, GRAD, DIAG>(prm, sm_count, stream, overlap);
    if (n <= 4) return launch_direct_as<T, VEC, 4, 1, GRAD, DIAG>(prm, sm_count, stream, overlap);
    if (n <= 8) return launch_direct_as<T, VEC, 4, 2, GRAD, DIAG>(prm, sm_count, stream, overlap);
    if (n <= 16) return launch_direct_as<T, VEC, 4, 4, GRAD, DIAG>(prm, sm_count, stream, overlap);
    if (n <= 32) return launch_direct_as<T, VEC, 4, 8, GRAD, DIAG>(prm, sm_count, stream, overlap);
    return launch_direct_as<T, VEC, 4, 16, GRAD, DIAG>(prm, sm_count, stream, overlap);
}

}  // namespace

}  // namespace rps
