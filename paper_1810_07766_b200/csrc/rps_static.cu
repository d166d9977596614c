// rps_step_static: one RPS step for callers that must not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside another
// framework's memory pool whose budget is fixed up front, in a real-time loop
// that may not block on the driver's allocator, or in a plug-in that is handed
// its buffers and nothing else.  The ordinary path needs a few KB of scratch for
// the drop masks of a step, lent by the caller through rps_bind().  Here that
// scratch is a fixed array inside the library image instead, so the caller
// passes only its inputs and outputs.
#include "rps.h"

#include <cmath>
#include <mutex>

#include "rps_device.cuh"
#include "rps_kernels.h"

namespace {

// Drop masks of ONE step for up to RPS_MAX_WORKERS workers (1792 bytes).  Every GPU
// that loads the library holds this array until the process exits.  In host code
// the name below is only a stand-in for the symbol, not a device address: its
// address on a device comes from cudaGetSymbolAddress (see device_state()).
static __device__ __align__(256) unsigned char rps_static_mask_scratch[sizeof(rps::StepMasks)];

constexpr int kMaxDevices = 64;

struct DeviceState {
    bool ready = false;
    rps::StepMasks* masks = nullptr;  // device address of rps_static_mask_scratch on this device
    int sm_count = 0;
};

std::mutex g_lock;
DeviceState g_devices[kMaxDevices];

// Once per device, with that device current: resolve the array's device address
// and the SM count.  Neither call allocates.
int device_state(DeviceState** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return RPS_ECUDA;
    if (dev < 0 || dev >= kMaxDevices) return RPS_EINVAL;
    std::lock_guard<std::mutex> hold(g_lock);
    DeviceState& st = g_devices[dev];
    if (!st.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, rps_static_mask_scratch) != cudaSuccess || ptr == nullptr) return RPS_ECUDA;
        if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RPS_ECUDA;
        st.masks = static_cast<rps::StepMasks*>(ptr);
        st.ready = true;
    }
    *out = &st;
    return RPS_OK;
}

}  // namespace

extern "C" int rps_step_static(int n, int64_t d, int dtype, void* x_dev, const void* b_dev, int64_t pitch, double p,
                               double gamma, double sigma, uint64_t seed, uint64_t t, void* cuda_stream)
{
    // the scratch record has room for RPS_MAX_WORKERS workers and no more
    if (n > RPS_MAX_WORKERS) return RPS_ELIMIT;
    if (n < 1 || d < 1 || d >= ((int64_t)1 << 34)) return RPS_EINVAL;
    if (dtype != RPS_F32 && dtype != RPS_BF16) return RPS_EINVAL;
    if (!(p >= 0.0 && p <= 1.0) || !std::isfinite(gamma) || !std::isfinite(sigma) || sigma < 0.0) return RPS_EINVAL;
    if (!x_dev || !b_dev || ((uintptr_t)x_dev | (uintptr_t)b_dev) % 128 != 0) return RPS_EINVAL;
    const int64_t per_line = dtype == RPS_BF16 ? 64 : 32;
    if (pitch < d || pitch % per_line != 0) return RPS_EINVAL;

    DeviceState* st = nullptr;
    int rc = device_state(&st);
    if (rc != RPS_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    // masks of step t, written in full for blocks 0..n-1 (nothing in the array has to start at zero)
    rps::MaskParams mp{};
    mp.out = st->masks;
    mp.t0 = t;
    mp.drop_threshold = (uint64_t)std::floor(p * 4294967296.0);
    mp.key0 = (uint32_t)seed;
    mp.key1 = (uint32_t)(seed >> 32);
    mp.n = n;
    mp.self_delivery = 1;
    mp.assign_perm = 0;
    if (rps::launch_masks(mp, 1, stream) != cudaSuccess) return RPS_ECUDA;

    rps::FusedParams fp{};
    fp.x = x_dev;
    fp.b = b_dev;
    fp.masks = st->masks;
    fp.pitch = pitch;
    fp.d = d;
    fp.col_offset = 0;
    fp.cols_in_row = pitch;
    fp.block_cols = (d + n - 1) / n;
    fp.n = n;
    fp.narrow = d < ((int64_t)1 << 31);
    fp.error = nullptr;  // nobody reads back here; a wait that gives up just ends the kernel early
    rps::set_sgd_scalars(fp, (float)gamma, (float)sigma);
    fp.t_lo = (uint32_t)t;
    fp.t_hi = (uint32_t)(t >> 32);
    fp.descending = (int32_t)(t & 1u);  // as rps_step does: odd steps walk the columns downwards
    fp.inv_n = 1.0f / (float)n;
    rps::set_philox_key(fp, seed);
    if (rps::launch_fused(fp, rps::FusedTuning{}, dtype == RPS_BF16, st->sm_count, stream) != cudaSuccess)
        return RPS_ECUDA;
    return RPS_OK;
}
