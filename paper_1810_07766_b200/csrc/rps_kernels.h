// Host-visible parameter blocks and launch wrappers of the RPS kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace rps {

// What a launch wrapper remembers about one kernel instantiation, PER DEVICE and under a lock: the dynamic
// shared memory the kernel has been granted (cudaFuncSetAttribute acts on the current device's copy of the
// function) and its resident CTAs per SM.  Handles bound on several devices, and host threads stepping
// distinct handles, may launch the same instantiation at the same time.
constexpr int kMaxDevices = 64;

struct LaunchState {
    std::mutex lock;
    size_t smem_limit[kMaxDevices] = {};     // opt-in shared memory per CTA of the device (0 = not asked yet)
    uint32_t smem_granted[kMaxDevices] = {};
    int occ_threads[kMaxDevices] = {};       // the launch shape the occupancy below was asked for
    uint32_t occ_smem[kMaxDevices] = {};
    int occ_per_sm[kMaxDevices] = {};        // 0 = not asked yet
};

inline cudaError_t current_device(int* dev)
{
    cudaError_t err = cudaGetDevice(dev);
    if (err != cudaSuccess) return err;
    return *dev >= 0 && *dev < kMaxDevices ? cudaSuccess : cudaErrorInvalidDevice;
}

// Opt-in shared memory per CTA of the current device.
inline cudaError_t smem_limit_of_device(LaunchState& st, size_t* out)
{
    int dev = 0;
    cudaError_t err = current_device(&dev);
    if (err != cudaSuccess) return err;
    std::lock_guard<std::mutex> hold(st.lock);
    if (st.smem_limit[dev] == 0) {
        int optin = 0;
        if ((err = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
            return err;
        st.smem_limit[dev] = (size_t)optin;
    }
    *out = st.smem_limit[dev];
    return cudaSuccess;
}

// Makes sure `kernel` may be launched with `bytes` of dynamic shared memory on the current device.
template <typename Kernel>
cudaError_t grant_smem(LaunchState& st, Kernel kernel, uint32_t bytes)
{
    int dev = 0;
    cudaError_t err = current_device(&dev);
    if (err != cudaSuccess) return err;
    std::lock_guard<std::mutex> hold(st.lock);
    if (bytes > st.smem_granted[dev]) {
        if ((err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes)) != cudaSuccess)
            return err;
        st.smem_granted[dev] = bytes;
    }
    return cudaSuccess;
}

// Resident CTAs per SM of `kernel` in this launch shape on the current device (at least 1).
template <typename Kernel>
cudaError_t resident_ctas_per_sm(LaunchState& st, Kernel kernel, int threads, uint32_t smem_bytes, int* out)
{
    int dev = 0;
    cudaError_t err = current_device(&dev);
    if (err != cudaSuccess) return err;
    std::lock_guard<std::mutex> hold(st.lock);
    if (st.occ_per_sm[dev] == 0 || st.occ_threads[dev] != threads || st.occ_smem[dev] != smem_bytes) {
        int occ = 0;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, threads, smem_bytes)) != cudaSuccess)
            return err;
        st.occ_per_sm[dev] = occ < 1 ? 1 : occ;
        st.occ_threads[dev] = threads;
        st.occ_smem[dev] = smem_bytes;
    }
    *out = st.occ_per_sm[dev];
    return cudaSuccess;
}

struct StepMasks;  // defined in rps_device.cuh

constexpr size_t kStepMasksBytes = 64 * 8 * 2 + 64 * 4 * 3;  // 1792 bytes per step

struct MaskParams {
    StepMasks* out;           // [steps] mask records, device
    uint64_t t0;              // first step of the window
    uint64_t drop_threshold;  // floor(p * 2^32): a message is lost iff its 32-bit draw is below it
    uint32_t key0, key1;      // Philox key = seed
    int32_t n;
    int32_t self_delivery;
    int32_t assign_perm;
};

// Which fused kernel runs and how it is shaped; 0 everywhere = the library's choice.
struct FusedTuning {
    int32_t kernel;            // 1 direct (register loads), 2 staged (a producer warp fills a shared-memory ring),
                               // 3 self-refilling ring (every warp computes; bf16 replicas), 4 workers streamed
                               // through a ring per warp
    int32_t workers_per_lane;  // 2, 4 or 8
    int32_t stages;            // shared-memory ring depth of the staged kernel
    int32_t consumer_warps;    // compute warps per CTA of the staged kernel
    int32_t copy_mode;         // staged kernel: 1 one bulk copy per row, 2 two-dimensional TMA boxes
    int32_t slice_bytes;       // staged kernel, bf16: bytes of a row one lane handles, 16 or 8
    int32_t store_mode;        // staged kernel: 1 stores from registers, 2 TMA stores from an output tile, 3 TMA stores in place
    int32_t wait_limit_ms;     // staged kernel: bound of every mbarrier wait (0 = 2000 ms)
    int32_t withhold_copies;   // staged kernel, test aid: issue no copies so that the bounded waits run out
    int32_t traversal;         // 0 odd steps walk the tiles downwards, 1 always upwards
    int32_t l2_policy;         // staged kernel: 1 plain loads, 2 targets loaded with the L2 evict-first hint
    int32_t launch_overlap;    // staged kernel: 1 plain launch, 2 programmatic stream serialization
    int32_t team_warps;        // ring kernel: warp slices per tile (1..16)
    int32_t early_targets;     // staged and streamed kernels: 1 every copy waits for the kernel ahead in the stream,
                               // 2 the copies of b for the first stages are issued before that wait
    int32_t fuse_steps;        // rps_step_n: 1 one launch per step, 2 as many steps per launch as the kernel takes
};

struct FusedParams {
    void* x;        // [n][pitch] replicas, updated in place
    const void* b;  // [n][pitch] targets of the quadratic objective
    const StepMasks* masks;
    int32_t* error;      // device word set non-zero when a bounded wait gave up (may be NULL)
    double* trace;       // tracked step: [2] sums this launch adds to (see Tracker), zeroed beforehand; else NULL
    int64_t pitch;       // row pitch in elements
    int64_t d;           // columns to process: the model size, or the width of a window of its columns
    int64_t col_offset;  // index in the whole model of column 0 of x and b (0 unless this is a window; a multiple of 64)
    int64_t cols_in_row; // columns that may be read in a row from its first one (the pitch, less what precedes a window)
    int64_t block_cols;  // ceil(model size / n): columns per parameter-server block
    int32_t n;
    int32_t narrow;  // model size < 2^31: block index by 32-bit division
    // v = x + gamma * (b - x) - (gamma * sigma) * xi
    float gamma;
    float noise_scale;  // -2 ln 2 * (gamma * sigma)^2
    int32_t noisy;      // sigma != 0
    int32_t average_gradients;  // 1: the updates -gamma*g are averaged and applied to x (Section 5's comparison)
    int32_t descending;         // 1: take the tiles from the last to the first (odd steps, see FusedTuning::traversal)
    float inv_n;                // 1 / n
    uint32_t t_lo, t_hi;
    uint32_t key0, key1;
    uint32_t round_key[10][2];  // Philox round keys: key + r * (0x9E3779B9, 0xBB67AE85)
};

// Fills key0, key1 and round_key from the 64-bit seed.
void set_philox_key(FusedParams& prm, uint64_t seed);

// Fills gamma, noise_scale and noisy from the float learning rate and noise level.
void set_sgd_scalars(FusedParams& prm, float gamma, float sigma);

struct DiagParams {
    const void* x;
    const void* b;
    double* out;  // [2] accumulators, zeroed by the caller
    int64_t pitch;
    int64_t d;
    int32_t n;
};

struct AlphaParams {
    const StepMasks* masks;  // one record per step
    double* out;             // [2] sums over all blocks of all records, added to
    int32_t n;
};

cudaError_t launch_alpha(const AlphaParams& prm, int steps, cudaStream_t stream);
cudaError_t launch_masks(const MaskParams& prm, int steps, cudaStream_t stream);
cudaError_t launch_fused(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                         cudaStream_t stream);
cudaError_t launch_fused_direct(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream);
cudaError_t launch_fused_staged(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream);
// The self-refilling ring (rps_ring.cu): whether it is built for this step, and its launch.
bool ring_kernel_covers(const FusedParams& prm, bool bf16);
cudaError_t launch_fused_ring(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                              cudaStream_t stream);
// Workers streamed through per-warp rings (rps_stream.cu): whether it is built for this step, and its launch.
bool stream_kernel_covers(const FusedParams& prm, bool bf16);
// `steps` consecutive steps from step (prm.t_hi, prm.t_lo) in one launch, with the mask records of those steps at
// prm.masks[0 .. steps-1] (untracked steps; each team of warps goes from step to step on its own tiles).
cudaError_t launch_fused_stream(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream, int steps = 1);
// Whether launch_fused would run this step as a kernel that can take several steps per launch, and that launch.
bool fused_steps_supported(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count);
cudaError_t launch_fused_steps(const FusedParams& prm, const FusedTuning& tune, int steps, bool bf16, int sm_count,
                               cudaStream_t stream);
// The optional forms of the fused step, built in one family of lane shapes, each group in a
// translation unit of its own: gradient averaging (prm.average_gradients) and tracked steps
// (prm.trace != NULL, with either kind of averaging).
cudaError_t launch_staged_gradavg(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                  cudaStream_t stream);
cudaError_t launch_staged_tracked(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                  cudaStream_t stream);
cudaError_t launch_direct_tracked(const FusedParams& prm, bool bf16, int sm_count, cudaStream_t stream);
// `steps` consecutive steps from step (prm.t_hi, prm.t_lo) in one pass, with the mask records of those steps
// at prm.masks[0 .. steps-1]; plain model averaging, untracked (rps_blocked.cu).
cudaError_t launch_fused_blocked(const FusedParams& prm, int steps, bool bf16, int sm_count, cudaStream_t stream);
cudaError_t launch_diag(const DiagParams& prm, bool bf16, int sm_count, cudaStream_t stream);

}  // namespace rps
