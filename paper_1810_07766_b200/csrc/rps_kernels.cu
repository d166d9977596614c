// CUDA kernels of the RPS step for sm_100a: the Philox drop-mask generator, the
// fused local-SGD + masked-average + masked-write-back pass, and an off-path
// diagnostic reduction.  Host launch wrappers are at the bottom.
#include "rps_kernels.h"

#include "rps_device.cuh"

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
        }
    }
}

// --------------------------------------------------------------------------
// Fused step.  A warp owns LPG * VEC consecutive columns per iteration; its 32
// lanes are G groups of LPG = 32 / G lanes.  Group g handles workers
// g*WPT .. g*WPT + WPT - 1, lane `sub` of a group handles VEC consecutive columns
// of each of those workers with one vector load per row, so a group reads whole
// contiguous row segments.  Each lane keeps its WPT x VEC values of v in
// registers, sums the ones whose up-bit is set, the G partial sums are combined
// with xor-shuffles (every lane ends with the same total, bit for bit), and
// each lane writes back either the average or its own v according to the
// down-bit.  x is read once and written once, b is read once.
// --------------------------------------------------------------------------
template <typename T, int VEC>
struct RowVec;

template <>
struct RowVec<float, 4> {
    static __device__ __forceinline__ void load(const float* p, float (&out)[4])
    {
        const float4 v = __ldcs(reinterpret_cast<const float4*>(p));
        out[0] = v.x, out[1] = v.y, out[2] = v.z, out[3] = v.w;
    }
    static __device__ __forceinline__ void store(float* p, const float (&in)[4])
    {
        __stcs(reinterpret_cast<float4*>(p), make_float4(in[0], in[1], in[2], in[3]));
    }
};

template <>
struct RowVec<__nv_bfloat16, 8> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&out)[8])
    {
        const uint4 v = __ldcs(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            out[2 * k] = __uint_as_float(w[k] << 16);            // bf16 -> fp32 is exact
            out[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&in)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 pair = __floats2bfloat162_rn(in[2 * k], in[2 * k + 1]);  // nearest-even
            w[k] = *reinterpret_cast<const uint32_t*>(&pair);
        }
        __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
    }
};

template <int G>
__device__ __forceinline__ float sum_over_groups(float s)
{
#pragma unroll
    for (int off = 32 / G; off < 32; off <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    return s;
}

__device__ __forceinline__ int block_of(int64_t c, const FusedParams& prm)
{
    // columns are cut into n blocks of block_cols = ceil(d / n) columns (Step 0)
    return prm.narrow ? (int)((uint32_t)c / (uint32_t)prm.block_cols) : (int)(c / prm.block_cols);
}

template <typename T, int VEC, int WPT, int G, int THREADS>
__global__ void __launch_bounds__(THREADS) rps_fused_kernel(const FusedParams prm)
{
    static_assert(WPT % 2 == 0 && VEC % 4 == 0, "noise draws cover worker pairs and 4 columns");
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    const int lane = threadIdx.x & 31;
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;  // first worker of this lane's group
    const int n = prm.n;
    const int64_t d = prm.d;
    T* __restrict__ x = static_cast<T*>(prm.x);
    const T* __restrict__ b = static_cast<const T*>(prm.b);
    const StepMasks* __restrict__ masks = prm.masks;
    const float gamma = prm.gamma, sigma = prm.sigma;

    const int64_t warps_total = (int64_t)gridDim.x * (THREADS / 32);
    const int64_t tiles = (d + WARP_COLS - 1) / WARP_COLS;
    for (int64_t tile = (int64_t)blockIdx.x * (THREADS / 32) + (threadIdx.x >> 5); tile < tiles;
         tile += warps_total) {
        const int64_t c = tile * WARP_COLS + (int64_t)sub * VEC;
        const bool col_live = c < d;  // the row pitch covers the whole vector even when c + VEC > d

        float xv[WPT][VEC], v[WPT][VEC];
        {
            float bv[WPT][VEC];
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                if (col_live && w_first + w < n) {
                    const int64_t at = (int64_t)(w_first + w) * prm.pitch + c;
                    RowVec<T, VEC>::load(x + at, xv[w]);
                    RowVec<T, VEC>::load(b + at, bv[w]);
                } else {
#pragma unroll
                    for (int e = 0; e < VEC; ++e) xv[w][e] = bv[w][e] = 0.0f;
                }
            }
            // local SGD step: v = x - gamma * grad F_i(x; xi), grad = (x - b_i) + sigma * xi
            if (sigma != 0.0f) {
#pragma unroll
                for (int w = 0; w < WPT; w += 2) {
#pragma unroll
                    for (int q = 0; q < VEC / 4; ++q) {
                        const Philox4 r = philox4x32_10(prm.t_lo, prm.t_hi, (uint32_t)(c >> 2) + q,
                                                        kStreamNoise | ((uint32_t)((w_first + w) >> 1) << 8),
                                                        prm.key0, prm.key1);
                        const float2 z0 = gaussian_pair(r.x), z1 = gaussian_pair(r.y);
                        const float2 z2 = gaussian_pair(r.z), z3 = gaussian_pair(r.w);
                        const float za[4] = {z0.x, z0.y, z1.x, z1.y};
                        const float zb[4] = {z2.x, z2.y, z3.x, z3.y};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int k = 4 * q + e;
                            v[w][k] = fmaf(-gamma, fmaf(sigma, za[e], xv[w][k] - bv[w][k]), xv[w][k]);
                            v[w + 1][k] = fmaf(-gamma, fmaf(sigma, zb[e], xv[w + 1][k] - bv[w + 1][k]), xv[w + 1][k]);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int w = 0; w < WPT; ++w)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) v[w][e] = fmaf(-gamma, xv[w][e] - bv[w][e], xv[w][e]);
            }
        }

        const int j_first = col_live ? block_of(c, prm) : 0;
        const bool uniform = !col_live || (c + VEC <= d && block_of(c + VEC - 1, prm) == j_first);
        if (__all_sync(0xFFFFFFFFu, uniform)) {
            // all VEC columns of this lane lie in one block: one mask word serves them
            const uint32_t up = (uint32_t)(masks->up[j_first] >> w_first);
            const uint32_t down = (uint32_t)(masks->down[j_first] >> w_first);
            const int cnt = masks->cnt[j_first];
            float avg[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                float s = 0.0f;
#pragma unroll
                for (int w = 0; w < WPT; ++w) s += ((up >> w) & 1u) ? v[w][e] : 0.0f;
                s = sum_over_groups<G>(s);
                avg[e] = cnt > 0 ? s / (float)cnt : 0.0f;  // 1/|N| * sum over N (RS step)
            }
            if (col_live) {
#pragma unroll
                for (int w = 0; w < WPT; ++w) {
                    if (w_first + w < n) {
                        float out[VEC];
#pragma unroll
                        for (int e = 0; e < VEC; ++e) out[e] = ((down >> w) & 1u) ? avg[e] : v[w][e];  // AG step
                        RowVec<T, VEC>::store(x + (int64_t)(w_first + w) * prm.pitch + c, out);
                    }
                }
            }
        } else {
            // a lane of this warp straddles a block boundary or the end of the row:
            // every column looks up its own block
            float avg[VEC];
            uint32_t down[VEC];
            bool live[VEC];
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                live[e] = c + e < d;
                const int j = live[e] ? block_of(c + e, prm) : 0;
                const uint32_t up = (uint32_t)(masks->up[j] >> w_first);
                down[e] = (uint32_t)(masks->down[j] >> w_first);
                const int cnt = masks->cnt[j];
                float s = 0.0f;
#pragma unroll
                for (int w = 0; w < WPT; ++w) s += ((up >> w) & 1u) ? v[w][e] : 0.0f;
                s = sum_over_groups<G>(s);
                avg[e] = cnt > 0 ? s / (float)cnt : 0.0f;
            }
            if (col_live) {
#pragma unroll
                for (int w = 0; w < WPT; ++w) {
                    if (w_first + w < n) {
                        float out[VEC];
#pragma unroll
                        for (int e = 0; e < VEC; ++e)
                            out[e] = !live[e] ? xv[w][e] : (((down[e] >> w) & 1u) ? avg[e] : v[w][e]);
                        RowVec<T, VEC>::store(x + (int64_t)(w_first + w) * prm.pitch + c, out);
                    }
                }
            }
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
// Launch wrappers
// --------------------------------------------------------------------------
cudaError_t launch_masks(const MaskParams& prm, int steps, cudaStream_t stream)
{
    rps_mask_kernel<<<steps, 256, 0, stream>>>(prm);
    return cudaGetLastError();
}

namespace {

constexpr int kThreads = 256;

template <typename T, int VEC, int WPT, int G>
cudaError_t launch_fused_as(const FusedParams& prm, int sm_count, cudaStream_t stream)
{
    constexpr int warp_cols = (32 / G) * VEC;
    const int64_t tiles = (prm.d + warp_cols - 1) / warp_cols;
    const int64_t ctas_needed = (tiles + kThreads / 32 - 1) / (kThreads / 32);
    static int per_sm = 0;  // resident CTAs per SM of this instantiation, asked once
    if (per_sm == 0) {
        int occ = 0;
        cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
            &occ, rps_fused_kernel<T, VEC, WPT, G, kThreads>, kThreads, 0);
        if (err != cudaSuccess) return err;
        per_sm = occ < 1 ? 1 : occ;
    }
    // a whole number of waves of resident CTAs, each striding over the tiles
    int64_t grid = (int64_t)sm_count * per_sm;
    if (grid > ctas_needed) grid = ctas_needed;
    if (grid < 1) grid = 1;
    rps_fused_kernel<T, VEC, WPT, G, kThreads><<<(unsigned)grid, kThreads, 0, stream>>>(prm);
    return cudaGetLastError();
}

template <typename T, int VEC>
cudaError_t launch_fused_for_n(const FusedParams& prm, int sm_count, cudaStream_t stream)
{
    const int n = prm.n;
    if (n <= 2) return launch_fused_as<T, VEC, 2, 1>(prm, sm_count, stream);
    if (n <= 4) return launch_fused_as<T, VEC, 4, 1>(prm, sm_count, stream);
    if (n <= 8) return launch_fused_as<T, VEC, 8, 1>(prm, sm_count, stream);
    if (n <= 16) return launch_fused_as<T, VEC, 8, 2>(prm, sm_count, stream);
    if (n <= 32) return launch_fused_as<T, VEC, 8, 4>(prm, sm_count, stream);
    return launch_fused_as<T, VEC, 8, 8>(prm, sm_count, stream);
}

}  // namespace

cudaError_t launch_fused(const FusedParams& prm, bool bf16, int sm_count, cudaStream_t stream)
{
    if (bf16) return launch_fused_for_n<__nv_bfloat16, 8>(prm, sm_count, stream);
    return launch_fused_for_n<float, 4>(prm, sm_count, stream);
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
