// Host-visible parameter blocks and launch wrappers of the RPS kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace rps {

struct StepMasks;  // defined in rps_device.cuh; 1536 bytes per step

constexpr size_t kStepMasksBytes = 64 * 8 * 2 + 64 * 4 * 2;

struct MaskParams {
    StepMasks* out;           // [steps] mask records, device
    uint64_t t0;              // first step of the window
    uint64_t drop_threshold;  // floor(p * 2^32): a message is lost iff its 32-bit draw is below it
    uint32_t key0, key1;      // Philox key = seed
    int32_t n;
    int32_t self_delivery;
    int32_t assign_perm;
};

struct FusedParams {
    void* x;        // [n][pitch] replicas, updated in place
    const void* b;  // [n][pitch] targets of the quadratic objective
    const StepMasks* masks;
    int64_t pitch;       // row pitch in elements
    int64_t d;           // model size
    int64_t block_cols;  // ceil(d / n): columns per parameter-server block
    int32_t n;
    int32_t narrow;  // d < 2^31: block index by 32-bit division
    float gamma, sigma;
    uint32_t t_lo, t_hi;
    uint32_t key0, key1;
};

struct DiagParams {
    const void* x;
    const void* b;
    double* out;  // [2] accumulators, zeroed by the caller
    int64_t pitch;
    int64_t d;
    int32_t n;
};

cudaError_t launch_masks(const MaskParams& prm, int steps, cudaStream_t stream);
cudaError_t launch_fused(const FusedParams& prm, bool bf16, int sm_count, cudaStream_t stream);
cudaError_t launch_diag(const DiagParams& prm, bool bf16, int sm_count, cudaStream_t stream);

}  // namespace rps
