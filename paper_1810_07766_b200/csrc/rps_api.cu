// C ABI of the RPS library (see include/rps.h): argument checks, the step
// counter, the window of pre-generated drop masks, copies between dense host
// arrays and the pitched device layout, and per-kernel event timing.
#include "rps.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "rps_device.cuh"
#include "rps_kernels.h"

static_assert(sizeof(rps::StepMasks) == rps::kStepMasksBytes, "mask record layout");

// Extra 128-byte lines appended to every row.  `asked` < 0 = automatic: as many as make the row a whole
// number of kilobytes, so that every row starts on a 1 KB boundary and the row pieces the kernels move (1 to
// 4 KB wide, cut at multiples of their width from the start of the row) are whole DRAM pages in every row
// instead of straddling page boundaries in most of them (measured: up to 3 % of the step).  Rows that all
// start at the same offset modulo a large power of two are no problem on this memory system.
static int64_t rps_row_skew_lines(int64_t lines, int32_t asked)
{
    if (asked >= 0) return asked;
    return (8 - lines % 8) % 8;
}

namespace {

constexpr size_t kDiagBytes = 256;   // two fp64 accumulators, then the kernels' error word, padded
constexpr size_t kErrorOffset = 64;
constexpr int kHostChunks = 8;                       // rps_step_host cuts the columns into at most this many pieces
constexpr int64_t kHostChunkMinBytes = 4 << 20;      // ... of at least this many bytes of x each
thread_local std::string g_create_error;

struct TimedLaunch {
    cudaEvent_t start, stop;
    int kind;  // 0 fused, 1 mask
};

}  // namespace

struct rps_handle {
    int n = 0;
    int64_t d = 0;
    double p = 0.0;
    float gamma = 0.0f;
    float sigma = 0.0f;
    uint64_t seed = 0;
    rps_options opt{};
    // binding
    bool bound = false;
    void* x = nullptr;
    void* b = nullptr;
    unsigned char* scratch = nullptr;
    cudaStream_t stream = nullptr;
    int device = -1;  // the device that was current at rps_bind: x, b, scratch and the stream belong to it
    int sm_count = 0;
    // run state
    uint64_t t = 0;
    bool window_valid = false;
    uint64_t window_t0 = 0;
    int64_t launches = 0;
    // timing
    bool profiling = false;
    std::vector<TimedLaunch> pending;
    double ms[2] = {0.0, 0.0};
    int64_t timed[2] = {0, 0};
    rps::StepMasks staged{};  // host copy of caller-given masks
    // rps_step_host: copy streams and the events that chain upload -> kernel -> download of each piece
    cudaStream_t up_stream = nullptr, down_stream = nullptr;
    cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
    cudaEvent_t ev_up[kHostChunks] = {}, ev_done[kHostChunks] = {};
    // tracked steps (rps_track)
    double* trace = nullptr;
    int64_t trace_capacity = 0;
    int64_t trace_used = 0;
    std::string error;

    size_t elem() const { return opt.dtype == RPS_BF16 ? 2 : 4; }
    // columns held by this handle: the whole model, or its shard
    int64_t cols() const { return opt.shard_cols > 0 ? opt.shard_cols : d; }
    int64_t pitch() const
    {
        const int64_t per_line = 128 / (int64_t)elem();
        const int64_t lines = (cols() + per_line - 1) / per_line;
        return (lines + rps_row_skew_lines(lines, opt.row_skew_lines)) * per_line;
    }
    double* diag_acc() const { return reinterpret_cast<double*>(scratch); }
    int32_t* error_word() const { return reinterpret_cast<int32_t*>(scratch + kErrorOffset); }
    rps::FusedTuning tuning() const
    {
        rps::FusedTuning tune{};
        tune.kernel = opt.kernel;
        tune.workers_per_lane = opt.workers_per_lane;
        tune.stages = opt.stages;
        tune.consumer_warps = opt.consumer_warps;
        tune.copy_mode = opt.copy_mode;
        tune.slice_bytes = opt.slice_bytes;
        tune.store_mode = opt.store_mode;
        tune.wait_limit_ms = opt.wait_limit_ms;
        tune.withhold_copies = opt.withhold_copies;
        tune.traversal = opt.traversal;
        tune.l2_policy = opt.l2_policy;
        tune.launch_overlap = opt.launch_overlap;
        tune.team_warps = opt.team_warps;
        tune.early_targets = opt.early_targets;
        tune.fuse_steps = opt.fuse_steps;
        return tune;
    }
    rps::StepMasks* window() const { return reinterpret_cast<rps::StepMasks*>(scratch + kDiagBytes); }
    rps::StepMasks* probe() const { return window() + opt.mask_window; }
    rps::StepMasks* forced() const { return window() + opt.mask_window + 1; }
    size_t scratch_bytes() const { return kDiagBytes + (size_t)(opt.mask_window + 2) * sizeof(rps::StepMasks); }
};

namespace {

int fail(rps_handle* h, int code, const std::string& why)
{
    if (h) h->error = why;
    return code;
}

int cuda_fail(rps_handle* h, const char* what, cudaError_t err)
{
    return fail(h, RPS_ECUDA, std::string(what) + ": " + cudaGetErrorString(err));
}

#define RPS_CUDA(h, call)                                         \
    do {                                                          \
        cudaError_t err__ = (call);                               \
        if (err__ != cudaSuccess) return cuda_fail(h, #call, err__); \
    } while (0)

int need_bound(rps_handle* h)
{
    if (!h) return RPS_EINVAL;
    if (!h->bound) return fail(h, RPS_ESTATE, "rps_bind has not been called");
    // kernels are launched on, and attributes set for, the CURRENT device: it has to be the handle's
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != h->device)
        return fail(h, RPS_ESTATE, "the device the handle was bound on is not the current device");
    return RPS_OK;
}

int flush_timing(rps_handle* h)
{
    if (h->pending.empty()) return RPS_OK;
    RPS_CUDA(h, cudaStreamSynchronize(h->stream));
    for (TimedLaunch& tl : h->pending) {
        float ms = 0.0f;
        cudaError_t err = cudaEventElapsedTime(&ms, tl.start, tl.stop);
        cudaEventDestroy(tl.start);
        cudaEventDestroy(tl.stop);
        if (err != cudaSuccess) {
            h->pending.clear();
            return cuda_fail(h, "cudaEventElapsedTime", err);
        }
        h->ms[tl.kind] += ms;
        h->timed[tl.kind] += 1;
    }
    h->pending.clear();
    return RPS_OK;
}

// Runs `launch` on the stream; when profiling, brackets it with events.
template <typename Launch>
int timed_launch(rps_handle* h, int kind, Launch launch)
{
    TimedLaunch tl{nullptr, nullptr, kind};
    if (h->profiling) {
        if (h->pending.size() >= 2048) {
            int rc = flush_timing(h);
            if (rc != RPS_OK) return rc;
        }
        RPS_CUDA(h, cudaEventCreate(&tl.start));
        RPS_CUDA(h, cudaEventCreate(&tl.stop));
        RPS_CUDA(h, cudaEventRecord(tl.start, h->stream));
    }
    cudaError_t err = launch();
    if (err != cudaSuccess) return cuda_fail(h, kind == 0 ? "fused step kernel launch" : "mask kernel launch", err);
    h->launches += 1;
    if (h->profiling) {
        RPS_CUDA(h, cudaEventRecord(tl.stop, h->stream));
        h->pending.push_back(tl);
    }
    return RPS_OK;
}

int generate_masks(rps_handle* h, rps::StepMasks* out, uint64_t t0, int steps)
{
    rps::MaskParams prm{};
    prm.out = out;
    prm.t0 = t0;
    prm.drop_threshold = (uint64_t)std::floor(h->p * 4294967296.0);
    prm.key0 = (uint32_t)h->seed;
    prm.key1 = (uint32_t)(h->seed >> 32);
    prm.n = h->n;
    prm.self_delivery = h->opt.self_delivery;
    prm.assign_perm = h->opt.assign == RPS_ASSIGN_PERM;
    return timed_launch(h, 1, [&] { return rps::launch_masks(prm, steps, h->stream); });
}

// The fused kernels' parameters for step h->t on columns [begin, begin + cols) of this handle's arrays.
rps::FusedParams fused_params(rps_handle* h, const rps::StepMasks* masks, int64_t begin, int64_t cols)
{
    rps::FusedParams prm{};
    prm.x = static_cast<char*>(h->x) + (size_t)begin * h->elem();
    prm.b = static_cast<const char*>(h->b) + (size_t)begin * h->elem();
    prm.masks = masks;
    prm.pitch = h->pitch();
    prm.d = cols;
    prm.col_offset = (h->opt.shard_cols > 0 ? h->opt.shard_begin : 0) + begin;
    prm.cols_in_row = h->pitch() - begin;
    prm.block_cols = (h->d + h->n - 1) / h->n;
    prm.n = h->n;
    prm.narrow = h->d < ((int64_t)1 << 31);
    prm.error = h->error_word();
    prm.average_gradients = h->opt.average == RPS_AVERAGE_GRADIENTS;
    prm.inv_n = 1.0f / (float)h->n;
    prm.descending = h->opt.traversal == 0 && (h->t & 1u) != 0;
    const bool tracked = h->trace != nullptr && h->trace_used < h->trace_capacity;
    prm.trace = tracked ? h->trace + 2 * h->trace_used : nullptr;
    rps::set_sgd_scalars(prm, h->gamma, h->sigma);
    prm.t_lo = (uint32_t)h->t;
    prm.t_hi = (uint32_t)(h->t >> 32);
    rps::set_philox_key(prm, h->seed);
    return prm;
}

// Launches the fused kernel of step h->t on columns [begin, begin + cols) of this handle's arrays (a
// multiple-of-64 begin), without advancing the step: a step may be issued in several pieces.
int launch_fused_window(rps_handle* h, const rps::StepMasks* masks, int64_t begin, int64_t cols)
{
    const rps::FusedParams prm = fused_params(h, masks, begin, cols);
    return timed_launch(h, 0, [&] {
        return rps::launch_fused(prm, h->tuning(), h->opt.dtype == RPS_BF16, h->sm_count, h->stream);
    });
}

void advance_step(rps_handle* h)
{
    if (h->trace != nullptr && h->trace_used < h->trace_capacity) h->trace_used += 1;
    h->t += 1;
}

// The mask record of step h->t, generating the next window of records when the step is outside the current one.
int masks_of_step(rps_handle* h, const rps::StepMasks** out)
{
    const uint64_t window = (uint64_t)h->opt.mask_window;
    if (!h->window_valid || h->t < h->window_t0 || h->t - h->window_t0 >= window) {
        int rc = generate_masks(h, h->window(), h->t, (int)window);
        if (rc != RPS_OK) return rc;
        h->window_valid = true;
        h->window_t0 = h->t;
    }
    *out = h->window() + (h->t - h->window_t0);
    return RPS_OK;
}

int run_fused(rps_handle* h, const rps::StepMasks* masks)
{
    int rc = launch_fused_window(h, masks, 0, h->cols());
    if (rc == RPS_OK) advance_step(h);
    return rc;
}

int copy_rows(rps_handle* h, void* dst, size_t dst_pitch_bytes, const void* src, size_t src_pitch_bytes,
              cudaMemcpyKind kind)
{
    const size_t row_bytes = (size_t)h->cols() * h->elem();
    if (dst_pitch_bytes < ((size_t)1 << 31) && src_pitch_bytes < ((size_t)1 << 31)) {
        RPS_CUDA(h, cudaMemcpy2DAsync(dst, dst_pitch_bytes, src, src_pitch_bytes, row_bytes, (size_t)h->n, kind,
                                      h->stream));
        return RPS_OK;
    }
    // rows longer than the 2-D copy's pitch limit: one copy per worker
    for (int i = 0; i < h->n; ++i)
        RPS_CUDA(h, cudaMemcpyAsync(static_cast<char*>(dst) + (size_t)i * dst_pitch_bytes,
                                    static_cast<const char*>(src) + (size_t)i * src_pitch_bytes, row_bytes, kind,
                                    h->stream));
    return RPS_OK;
}

int upload(rps_handle* h, void* dev, const void* host)
{
    return copy_rows(h, dev, (size_t)h->pitch() * h->elem(), host, (size_t)h->cols() * h->elem(), cudaMemcpyHostToDevice);
}

int download(rps_handle* h, void* host, const void* dev)
{
    return copy_rows(h, host, (size_t)h->cols() * h->elem(), dev, (size_t)h->pitch() * h->elem(), cudaMemcpyDeviceToHost);
}

// Drains the stream and reports a kernel that gave up on a bounded wait.
int finish(rps_handle* h)
{
    int32_t word = 0;
    RPS_CUDA(h, cudaMemcpyAsync(&word, h->error_word(), sizeof word, cudaMemcpyDeviceToHost, h->stream));
    RPS_CUDA(h, cudaStreamSynchronize(h->stream));
    if (word != 0)
        return fail(h, RPS_ECUDA, word == 1 ? "the fused kernel's producer gave up waiting for a free stage"
                                            : "the fused kernel's consumers gave up waiting for data");
    return RPS_OK;
}

}  // namespace

extern "C" {

int rps_default_options(rps_options* opt)
{
    if (!opt) return RPS_EINVAL;
    opt->dtype = RPS_F32;
    opt->assign = RPS_ASSIGN_FIXED;
    opt->self_delivery = 1;
    opt->mask_window = 32;
    opt->sigma = 0.0;
    opt->row_skew_lines = -1;
    opt->kernel = 0;
    opt->workers_per_lane = 0;
    opt->stages = 0;
    opt->consumer_warps = 0;
    opt->copy_mode = 0;
    opt->slice_bytes = 0;
    opt->store_mode = 0;
    opt->wait_limit_ms = 0;
    opt->withhold_copies = 0;
    opt->average = RPS_AVERAGE_MODELS;
    opt->traversal = 0;
    opt->l2_policy = 0;
    opt->launch_overlap = 0;
    opt->shard_begin = 0;
    opt->shard_cols = 0;
    opt->block_steps = 0;
    opt->team_warps = 0;
    opt->early_targets = 0;
    opt->fuse_steps = 0;
    return RPS_OK;
}

int rps_create(int n, int64_t d, double p, double gamma, uint64_t seed, rps_handle** out)
{
    if (!out) {
        g_create_error = "out is NULL";
        return RPS_EINVAL;
    }
    *out = nullptr;
    if (n < 1 || n > RPS_MAX_WORKERS) {
        g_create_error = "n must be in 1..64";
        return RPS_EINVAL;
    }
    if (d < 1 || d >= ((int64_t)1 << 34)) {
        g_create_error = "d must be in 1..2^34-1";
        return RPS_EINVAL;
    }
    if (!(p >= 0.0 && p <= 1.0)) {
        g_create_error = "p must be in [0, 1]";
        return RPS_EINVAL;
    }
    if (!std::isfinite(gamma)) {
        g_create_error = "gamma must be finite";
        return RPS_EINVAL;
    }
    rps_handle* h = new (std::nothrow) rps_handle();
    if (!h) {
        g_create_error = "out of host memory";
        return RPS_ENOMEM;
    }
    h->n = n;
    h->d = d;
    h->p = p;
    h->gamma = (float)gamma;
    h->seed = seed;
    rps_default_options(&h->opt);
    *out = h;
    return RPS_OK;
}

int rps_destroy(rps_handle* h)
{
    if (!h) return RPS_OK;
    for (TimedLaunch& tl : h->pending) {
        cudaEventDestroy(tl.start);
        cudaEventDestroy(tl.stop);
    }
    if (h->up_stream) {
        cudaStreamSynchronize(h->up_stream);
        cudaStreamDestroy(h->up_stream);
    }
    if (h->down_stream) {
        cudaStreamSynchronize(h->down_stream);
        cudaStreamDestroy(h->down_stream);
    }
    if (h->ev_begin) cudaEventDestroy(h->ev_begin);
    if (h->ev_end) cudaEventDestroy(h->ev_end);
    for (int k = 0; k < kHostChunks; ++k) {
        if (h->ev_up[k]) cudaEventDestroy(h->ev_up[k]);
        if (h->ev_done[k]) cudaEventDestroy(h->ev_done[k]);
    }
    delete h;
    return RPS_OK;
}

int rps_configure(rps_handle* h, const rps_options* opt)
{
    if (!h) return RPS_EINVAL;
    if (!opt) return fail(h, RPS_EINVAL, "options are NULL");
    if (h->bound) return fail(h, RPS_ESTATE, "options cannot change after rps_bind");
    if (opt->dtype != RPS_F32 && opt->dtype != RPS_BF16) return fail(h, RPS_EINVAL, "unknown dtype");
    if (opt->assign != RPS_ASSIGN_FIXED && opt->assign != RPS_ASSIGN_PERM) return fail(h, RPS_EINVAL, "unknown assign");
    if (opt->self_delivery != 0 && opt->self_delivery != 1) return fail(h, RPS_EINVAL, "self_delivery must be 0 or 1");
    if (opt->mask_window < 1 || opt->mask_window > 256) return fail(h, RPS_EINVAL, "mask_window must be in 1..256");
    if (!std::isfinite(opt->sigma) || opt->sigma < 0.0) return fail(h, RPS_EINVAL, "sigma must be finite and >= 0");
    if (opt->row_skew_lines < -1 || opt->row_skew_lines > 4096)
        return fail(h, RPS_EINVAL, "row_skew_lines must be -1 (auto) or 0..4096");
    if (opt->kernel < 0 || opt->kernel > 4) return fail(h, RPS_EINVAL, "kernel must be 0 (auto) or 1..4");
    if (opt->workers_per_lane != 0 && opt->workers_per_lane != 2 && opt->workers_per_lane != 4 &&
        opt->workers_per_lane != 8)
        return fail(h, RPS_EINVAL, "workers_per_lane must be 0 (auto), 2, 4 or 8");
    if (opt->stages != 0 && (opt->stages < 2 || opt->stages > 8)) return fail(h, RPS_EINVAL, "stages must be 0 or 2..8");
    if (opt->consumer_warps < 0 || opt->consumer_warps > 32)
        return fail(h, RPS_EINVAL, "consumer_warps must be 0 (auto) or 1..32");
    if (opt->slice_bytes != 0 && opt->slice_bytes != 8 && opt->slice_bytes != 16)
        return fail(h, RPS_EINVAL, "slice_bytes must be 0 (auto), 8 or 16");
    if (opt->average != RPS_AVERAGE_MODELS && opt->average != RPS_AVERAGE_GRADIENTS)
        return fail(h, RPS_EINVAL, "unknown average");
    if (opt->wait_limit_ms < 0 || opt->wait_limit_ms > 10000)
        return fail(h, RPS_EINVAL, "wait_limit_ms must be 0 (default) or 1..10000");
    if (opt->withhold_copies != 0 && opt->withhold_copies != 1)
        return fail(h, RPS_EINVAL, "withhold_copies must be 0 or 1");
    if (opt->store_mode < 0 || opt->store_mode > 3) return fail(h, RPS_EINVAL, "store_mode must be 0 (auto) or 1..3");
    if (opt->copy_mode < 0 || opt->copy_mode > 2) return fail(h, RPS_EINVAL, "copy_mode must be 0 (auto), 1 or 2");
    if (opt->traversal != 0 && opt->traversal != 1) return fail(h, RPS_EINVAL, "traversal must be 0 or 1");
    if (opt->l2_policy < 0 || opt->l2_policy > 2) return fail(h, RPS_EINVAL, "l2_policy must be 0 (auto), 1 or 2");
    if (opt->launch_overlap < 0 || opt->launch_overlap > 2)
        return fail(h, RPS_EINVAL, "launch_overlap must be 0 (auto), 1 or 2");
    if (opt->shard_cols < 0 || opt->shard_begin < 0)
        return fail(h, RPS_EINVAL, "shard_begin and shard_cols must not be negative");
    if (opt->shard_cols == 0 && opt->shard_begin != 0) return fail(h, RPS_EINVAL, "shard_begin without shard_cols");
    if (opt->shard_cols > 0 && (opt->shard_begin % 64 != 0 || opt->shard_begin > h->d - opt->shard_cols))
        return fail(h, RPS_EINVAL, "a shard starts at a multiple of 64 and ends inside the model");
    if (opt->block_steps < 0 || opt->block_steps > opt->mask_window)
        return fail(h, RPS_EINVAL, "block_steps must be in 0..mask_window");
    if (opt->team_warps < 0 || opt->team_warps > 16)
        return fail(h, RPS_EINVAL, "team_warps must be 0 (auto) or 1..16");
    if (opt->early_targets < 0 || opt->early_targets > 2)
        return fail(h, RPS_EINVAL, "early_targets must be 0 (auto), 1 or 2");
    if (opt->fuse_steps < 0 || opt->fuse_steps > 2) return fail(h, RPS_EINVAL, "fuse_steps must be 0 (auto), 1 or 2");
    h->opt = *opt;
    h->sigma = (float)opt->sigma;
    return RPS_OK;
}

int64_t rps_pitch(const rps_handle* h) { return h ? h->pitch() : (int64_t)RPS_EINVAL; }

size_t rps_scratch_bytes(const rps_handle* h) { return h ? h->scratch_bytes() : 0; }

int rps_bind(rps_handle* h, void* x_dev, void* b_dev, int64_t pitch, void* scratch_dev, size_t scratch_bytes,
             void* cuda_stream)
{
    if (!h) return RPS_EINVAL;
    if (!x_dev || !b_dev || !scratch_dev) return fail(h, RPS_EINVAL, "a device pointer is NULL");
    if (((uintptr_t)x_dev | (uintptr_t)b_dev) % 128 != 0) return fail(h, RPS_EINVAL, "x and b must be 128-byte aligned");
    if ((uintptr_t)scratch_dev % 256 != 0) return fail(h, RPS_EINVAL, "scratch must be 256-byte aligned");
    if (pitch != h->pitch()) return fail(h, RPS_EINVAL, "pitch must equal rps_pitch()");
    if (scratch_bytes < h->scratch_bytes()) return fail(h, RPS_EINVAL, "scratch is smaller than rps_scratch_bytes()");
    int dev = 0;
    RPS_CUDA(h, cudaGetDevice(&dev));
    RPS_CUDA(h, cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, dev));
    h->device = dev;
    h->x = x_dev;
    h->b = b_dev;
    h->scratch = static_cast<unsigned char*>(scratch_dev);
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    h->bound = true;
    h->window_valid = false;
    RPS_CUDA(h, cudaMemsetAsync(h->error_word(), 0, sizeof(int32_t), h->stream));
    return RPS_OK;
}

int rps_set_targets(rps_handle* h, const void* b_host)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!b_host) return fail(h, RPS_EINVAL, "b_host is NULL");
    return upload(h, h->b, b_host);
}

int rps_write(rps_handle* h, const void* x_host)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!x_host) return fail(h, RPS_EINVAL, "x_host is NULL");
    return upload(h, h->x, x_host);
}

int rps_set_step(rps_handle* h, uint64_t t)
{
    if (!h) return RPS_EINVAL;
    h->t = t;
    return RPS_OK;
}

int rps_get_step(const rps_handle* h, uint64_t* t)
{
    if (!h || !t) return RPS_EINVAL;
    *t = h->t;
    return RPS_OK;
}

int rps_step(rps_handle* h)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    const rps::StepMasks* masks = nullptr;
    if ((rc = masks_of_step(h, &masks)) != RPS_OK) return rc;
    return run_fused(h, masks);
}

int rps_step_n(rps_handle* h, int64_t T)
{
    if (h && T < 0) return fail(h, RPS_EINVAL, "T is negative");
    if (h && h->bound && h->opt.block_steps > 1 && h->opt.average == RPS_AVERAGE_MODELS) {
        // temporal blocking: as many steps per launch as asked for and as the window of masks holds (a lone
        // left-over step goes through the same kernel, so that the lane shape never changes within a run)
        int64_t done = 0;
        while (done < T) {
            const bool tracked = h->trace != nullptr && h->trace_used < h->trace_capacity;
            const rps::StepMasks* masks = nullptr;
            int rc = masks_of_step(h, &masks);
            if (rc != RPS_OK) return rc;
            int64_t chunk = (int64_t)h->opt.mask_window - (int64_t)(h->t - h->window_t0);
            if (chunk > h->opt.block_steps) chunk = h->opt.block_steps;
            if (chunk > T - done) chunk = T - done;
            if (tracked) {  // tracked steps run singly, in the same lane shape (4 workers per lane)
                if ((rc = run_fused(h, masks)) != RPS_OK) return rc;
                done += 1;
                continue;
            }
            rps::FusedParams prm = fused_params(h, masks, 0, h->cols());
            rc = timed_launch(h, 0, [&] {
                return rps::launch_fused_blocked(prm, (int)chunk, h->opt.dtype == RPS_BF16, h->sm_count, h->stream);
            });
            if (rc != RPS_OK) return rc;
            h->t += (uint64_t)chunk;
            done += chunk;
        }
        return RPS_OK;
    }
    if (h && h->bound && h->opt.fuse_steps != 1) {
        // as many steps per launch as the window of masks holds, where the kernel that serves this handle's steps can
        // go from step to step inside one launch (a tracked step, or a kernel that cannot, runs singly)
        int64_t done = 0;
        while (done < T) {
            int rc = need_bound(h);
            if (rc != RPS_OK) return rc;
            const rps::StepMasks* masks = nullptr;
            if ((rc = masks_of_step(h, &masks)) != RPS_OK) return rc;
            rps::FusedParams prm = fused_params(h, masks, 0, h->cols());
            int64_t chunk = (int64_t)h->opt.mask_window - (int64_t)(h->t - h->window_t0);
            if (chunk > T - done) chunk = T - done;
            if (chunk < 2 || !rps::fused_steps_supported(prm, h->tuning(), h->opt.dtype == RPS_BF16, h->sm_count)) {
                if ((rc = run_fused(h, masks)) != RPS_OK) return rc;
                done += 1;
                continue;
            }
            rc = timed_launch(h, 0, [&] {
                return rps::launch_fused_steps(prm, h->tuning(), (int)chunk, h->opt.dtype == RPS_BF16, h->sm_count,
                                               h->stream);
            });
            if (rc != RPS_OK) return rc;
            h->t += (uint64_t)chunk;
            done += chunk;
        }
        return RPS_OK;
    }
    for (int64_t k = 0; k < T; ++k) {
        int rc = rps_step(h);
        if (rc != RPS_OK) return rc;
    }
    return h ? RPS_OK : RPS_EINVAL;
}

int rps_step_forced(rps_handle* h, const uint64_t* up, const uint64_t* down)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!up || !down) return fail(h, RPS_EINVAL, "a mask array is NULL");
    const uint64_t valid = h->n == 64 ? ~(uint64_t)0 : (((uint64_t)1 << h->n) - 1);
    std::memset(&h->staged, 0, sizeof h->staged);
    for (int j = 0; j < h->n; ++j) {
        if ((up[j] | down[j]) & ~valid) return fail(h, RPS_EINVAL, "a mask has a bit set for a worker >= n");
        int cnt = 0;
        for (int i = 0; i < h->n; ++i) cnt += (int)((up[j] >> i) & 1);
        h->staged.up[j] = up[j];
        h->staged.down[j] = cnt > 0 ? down[j] : 0;
        h->staged.cnt[j] = cnt;
        h->staged.server[j] = j;
        h->staged.inv_cnt[j] = cnt > 0 ? 1.0f / (float)cnt : 0.0f;
    }
    // `staged` is pageable, so the copy has left it when the call returns; on the device the
    // copy is ordered after the previous step's kernel by the stream
    RPS_CUDA(h, cudaMemcpyAsync(h->forced(), &h->staged, sizeof h->staged, cudaMemcpyHostToDevice, h->stream));
    return run_fused(h, h->forced());
}

int rps_step_host(rps_handle* h, void* x_host, const void* b_host)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!x_host) return fail(h, RPS_EINVAL, "x_host is NULL");
    // Columns never interact, so the step is issued in pieces: piece k is uploaded on one copy stream,
    // stepped on the bound stream and downloaded on another copy stream, and the upload of piece k + 1
    // runs while piece k is on its way back (PCIe carries both directions at once).
    const int64_t cols = h->cols();
    const int64_t row_bytes = cols * (int64_t)h->elem();
    int pieces = (int)(row_bytes * h->n / kHostChunkMinBytes);
    if (pieces > kHostChunks) pieces = kHostChunks;
    if (pieces < 2 || h->pitch() >= ((int64_t)1 << 31)) {
        if ((rc = upload(h, h->x, x_host)) != RPS_OK) return rc;
        if (b_host && (rc = upload(h, h->b, b_host)) != RPS_OK) return rc;
        if ((rc = rps_step(h)) != RPS_OK) return rc;
        if ((rc = download(h, x_host, h->x)) != RPS_OK) return rc;
        return finish(h);
    }
    if (h->up_stream == nullptr) {
        RPS_CUDA(h, cudaStreamCreateWithFlags(&h->up_stream, cudaStreamNonBlocking));
        RPS_CUDA(h, cudaStreamCreateWithFlags(&h->down_stream, cudaStreamNonBlocking));
        RPS_CUDA(h, cudaEventCreateWithFlags(&h->ev_begin, cudaEventDisableTiming));
        RPS_CUDA(h, cudaEventCreateWithFlags(&h->ev_end, cudaEventDisableTiming));
        for (int k = 0; k < kHostChunks; ++k) {
            RPS_CUDA(h, cudaEventCreateWithFlags(&h->ev_up[k], cudaEventDisableTiming));
            RPS_CUDA(h, cudaEventCreateWithFlags(&h->ev_done[k], cudaEventDisableTiming));
        }
    }
    const rps::StepMasks* masks = nullptr;
    if ((rc = masks_of_step(h, &masks)) != RPS_OK) return rc;
    // the uploads overwrite what earlier work on the bound stream may still be using
    RPS_CUDA(h, cudaEventRecord(h->ev_begin, h->stream));
    RPS_CUDA(h, cudaStreamWaitEvent(h->up_stream, h->ev_begin, 0));
    RPS_CUDA(h, cudaStreamWaitEvent(h->down_stream, h->ev_begin, 0));
    const size_t es = h->elem();
    const size_t dev_pitch = (size_t)h->pitch() * es, host_pitch = (size_t)cols * es;
    const int64_t units = (cols + 63) / 64;  // pieces start at multiples of 64 columns
    for (int k = 0; k < pieces; ++k) {
        const int64_t begin = units * k / pieces * 64;
        const int64_t end = k + 1 == pieces ? cols : units * (k + 1) / pieces * 64;
        if (end <= begin) continue;
        const size_t width = (size_t)(end - begin) * es, at = (size_t)begin * es;
        RPS_CUDA(h, cudaMemcpy2DAsync(static_cast<char*>(h->x) + at, dev_pitch, static_cast<const char*>(x_host) + at,
                                      host_pitch, width, (size_t)h->n, cudaMemcpyHostToDevice, h->up_stream));
        if (b_host)
            RPS_CUDA(h, cudaMemcpy2DAsync(static_cast<char*>(h->b) + at, dev_pitch,
                                          static_cast<const char*>(b_host) + at, host_pitch, width, (size_t)h->n,
                                          cudaMemcpyHostToDevice, h->up_stream));
        RPS_CUDA(h, cudaEventRecord(h->ev_up[k], h->up_stream));
        RPS_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_up[k], 0));
        if ((rc = launch_fused_window(h, masks, begin, end - begin)) != RPS_OK) return rc;
        RPS_CUDA(h, cudaEventRecord(h->ev_done[k], h->stream));
        RPS_CUDA(h, cudaStreamWaitEvent(h->down_stream, h->ev_done[k], 0));
        RPS_CUDA(h, cudaMemcpy2DAsync(static_cast<char*>(x_host) + at, host_pitch, static_cast<const char*>(h->x) + at,
                                      dev_pitch, width, (size_t)h->n, cudaMemcpyDeviceToHost, h->down_stream));
    }
    advance_step(h);
    RPS_CUDA(h, cudaEventRecord(h->ev_end, h->down_stream));
    RPS_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_end, 0));
    return finish(h);
}

int rps_read(rps_handle* h, void* x_host_out)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!x_host_out) return fail(h, RPS_EINVAL, "x_host_out is NULL");
    if ((rc = download(h, x_host_out, h->x)) != RPS_OK) return rc;
    return finish(h);
}

int rps_read_masks(rps_handle* h, uint64_t t, uint64_t* up, uint64_t* down, int32_t* count, int32_t* server)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (!up || !down || !count) return fail(h, RPS_EINVAL, "an output array is NULL");
    if ((rc = generate_masks(h, h->probe(), t, 1)) != RPS_OK) return rc;
    rps::StepMasks host;
    RPS_CUDA(h, cudaMemcpyAsync(&host, h->probe(), sizeof host, cudaMemcpyDeviceToHost, h->stream));
    RPS_CUDA(h, cudaStreamSynchronize(h->stream));
    for (int j = 0; j < h->n; ++j) {
        up[j] = host.up[j];
        down[j] = host.down[j];
        count[j] = host.cnt[j];
        if (server) server[j] = host.server[j];
    }
    return RPS_OK;
}

int rps_diag(rps_handle* h, double* dist2_to_opt, double* consensus)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    RPS_CUDA(h, cudaMemsetAsync(h->diag_acc(), 0, 2 * sizeof(double), h->stream));
    rps::DiagParams prm{};
    prm.x = h->x;
    prm.b = h->b;
    prm.out = h->diag_acc();
    prm.pitch = h->pitch();
    prm.d = h->cols();  // a shard reports its own columns' part of both sums
    prm.n = h->n;
    cudaError_t err = rps::launch_diag(prm, h->opt.dtype == RPS_BF16, h->sm_count, h->stream);
    if (err != cudaSuccess) return cuda_fail(h, "diagnostic kernel launch", err);
    double host[2] = {0.0, 0.0};
    RPS_CUDA(h, cudaMemcpyAsync(host, h->diag_acc(), sizeof host, cudaMemcpyDeviceToHost, h->stream));
    RPS_CUDA(h, cudaStreamSynchronize(h->stream));
    if (dist2_to_opt) *dist2_to_opt = host[0];
    if (consensus) *consensus = host[1];
    return RPS_OK;
}

int rps_estimate_alpha(rps_handle* h, uint64_t t0, int64_t steps, double* alpha1, double* alpha2)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (h->n < 2) return fail(h, RPS_EINVAL, "alpha needs at least 2 workers");
    if (steps < 1 || !alpha1 || !alpha2) return fail(h, RPS_EINVAL, "steps must be positive and the outputs non-NULL");
    RPS_CUDA(h, cudaMemsetAsync(h->diag_acc(), 0, 2 * sizeof(double), h->stream));
    h->window_valid = false;  // the window of pre-generated masks is reused as sample storage
    const int64_t window = h->opt.mask_window;
    for (int64_t done = 0; done < steps; done += window) {
        const int chunk = (int)(steps - done < window ? steps - done : window);
        rc = generate_masks(h, h->window(), t0 + (uint64_t)done, chunk);
        if (rc != RPS_OK) return rc;
        rps::AlphaParams prm{h->window(), h->diag_acc(), h->n};
        cudaError_t err = rps::launch_alpha(prm, chunk, h->stream);
        if (err != cudaSuccess) return cuda_fail(h, "alpha kernel launch", err);
        h->launches += 1;
    }
    double host[2] = {0.0, 0.0};
    RPS_CUDA(h, cudaMemcpyAsync(host, h->diag_acc(), sizeof host, cudaMemcpyDeviceToHost, h->stream));
    RPS_CUDA(h, cudaStreamSynchronize(h->stream));
    const double samples = (double)steps * (double)h->n;
    *alpha1 = host[0] / samples;
    *alpha2 = host[1] / samples;
    return RPS_OK;
}

int rps_track(rps_handle* h, double* trace_dev, int64_t capacity)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (capacity < 0) return fail(h, RPS_EINVAL, "capacity is negative");
    if (capacity > ((int64_t)1 << 40)) return fail(h, RPS_EINVAL, "capacity is larger than 2^40 steps");
    if ((uintptr_t)trace_dev % 16 != 0) return fail(h, RPS_EINVAL, "trace_dev must be 16-byte aligned");
    h->trace = nullptr;
    h->trace_capacity = 0;
    h->trace_used = 0;
    if (trace_dev == nullptr || capacity == 0) return RPS_OK;
    RPS_CUDA(h, cudaMemsetAsync(trace_dev, 0, (size_t)capacity * 2 * sizeof(double), h->stream));
    h->trace = trace_dev;
    h->trace_capacity = capacity;
    return RPS_OK;
}

int rps_read_trace(rps_handle* h, double* trace_host_out, int64_t max_entries, int64_t* entries)
{
    int rc = need_bound(h);
    if (rc != RPS_OK) return rc;
    if (h->trace == nullptr) return fail(h, RPS_ESTATE, "tracking is off (rps_track)");
    if (!trace_host_out || !entries || max_entries < 0) return fail(h, RPS_EINVAL, "bad output arguments");
    const int64_t count = h->trace_used < max_entries ? h->trace_used : max_entries;
    if (count > 0)
        RPS_CUDA(h, cudaMemcpyAsync(trace_host_out, h->trace, (size_t)count * 2 * sizeof(double),
                                    cudaMemcpyDeviceToHost, h->stream));
    rc = finish(h);
    if (rc != RPS_OK) return rc;
    *entries = count;
    return RPS_OK;
}

int rps_profile(rps_handle* h, int enable)
{
    if (!h) return RPS_EINVAL;
    if (!enable) {
        int rc = flush_timing(h);
        h->profiling = false;
        return rc;
    }
    h->profiling = true;
    return RPS_OK;
}

int rps_profile_read(rps_handle* h, double* fused_ms, int64_t* fused_launches, double* mask_ms, int64_t* mask_launches)
{
    if (!h) return RPS_EINVAL;
    int rc = flush_timing(h);
    if (rc != RPS_OK) return rc;
    if (fused_ms) *fused_ms = h->ms[0];
    if (fused_launches) *fused_launches = h->timed[0];
    if (mask_ms) *mask_ms = h->ms[1];
    if (mask_launches) *mask_launches = h->timed[1];
    h->ms[0] = h->ms[1] = 0.0;
    h->timed[0] = h->timed[1] = 0;
    return RPS_OK;
}

int64_t rps_launch_count(const rps_handle* h) { return h ? h->launches : 0; }

const char* rps_last_error(const rps_handle* h) { return h ? h->error.c_str() : g_create_error.c_str(); }

const char* rps_version(void) { return "0.1"; }

}  // extern "C"
