/*
 * rps.h: C ABI of the RPS synchronisation step on one NVIDIA B200 (sm_100a).
 *
 * The library simulates, on one GPU, the unreliable parameter-server step of
 * centralized SGD from "Distributed Learning over Unreliable Networks"
 * (Algorithm 1, "RPS"): n workers each hold a full replica x^(i) of a model of
 * d parameters; the model is cut into n blocks, block j being averaged by one
 * worker (its server); every worker->server and server->worker message is lost
 * independently with probability p (Section 3).
 *
 * General rules
 *   - Every function returns RPS_OK (0) or a negative rps_status; nothing throws
 *     or aborts.  rps_last_error() gives a readable reason for the last failure
 *     on that handle.
 *   - "host" pointers are ordinary (preferably pinned) CPU memory, "device"
 *     pointers are CUDA global memory of the current device.  The library never
 *     allocates or frees device memory: the caller lends it x, b and a small
 *     scratch buffer with rps_bind() and keeps ownership.
 *   - Work is enqueued on the CUDA stream given to rps_bind(); calls that return
 *     data to the host synchronise that stream first.
 *   - A handle is not thread-safe; distinct handles are independent: they may be
 *     used from different host threads at the same time and bound on different
 *     devices of one process.  A handle belongs to the device that was current at
 *     rps_bind(); every later call that touches the device must be made with that
 *     device current (RPS_ESTATE otherwise).
 *   - Dense host arrays are row-major [n][d] in the replica type (float, or
 *     bfloat16 bit patterns in uint16_t).  On the device a row occupies
 *     rps_pitch() elements (d rounded up so that every row starts on a 1 KB
 *     boundary, or as row_skew_lines says); columns d..pitch-1 are padding that
 *     belongs to the library: it reads it, may zero the few padding columns that
 *     share a 16-byte unit with column d-1, and leaves the rest as it found it.
 */
#ifndef RPS_H
#define RPS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rps_handle rps_handle;

typedef enum rps_status {
    RPS_OK = 0,
    RPS_EINVAL = -1, /* bad argument (range, NULL, alignment, size)          */
    RPS_ESTATE = -2, /* call not allowed in the handle's current state      */
    RPS_ECUDA = -3,  /* a CUDA runtime call or kernel launch reported an error */
    RPS_ENOMEM = -4, /* host allocation failed                               */
    RPS_ELIMIT = -5  /* a size exceeds a fixed capacity built into the library */
} rps_status;

enum { RPS_MAX_WORKERS = 64 };

/* Replica storage type.  Arithmetic is always fp32 (bf16 replicas are widened
 * on load, accumulated in fp32, and rounded to nearest-even on store).        */
typedef enum rps_dtype { RPS_F32 = 0, RPS_BF16 = 1 } rps_dtype;

/* Who averages block j at step t.
 * RPS_ASSIGN_FIXED: worker j, every step (the simplification of Section 4.1).
 * RPS_ASSIGN_PERM:  a uniformly random permutation drawn afresh every step, as
 *                   Algorithm 1 states ("choose one worker b_t^(i) without
 *                   replacement") and as the lemmas of the supplement assume. */
typedef enum rps_assign { RPS_ASSIGN_FIXED = 0, RPS_ASSIGN_PERM = 1 } rps_assign;

/* What the workers exchange.
 * RPS_AVERAGE_MODELS:    the models v after the local SGD step: the RPS algorithm (Algorithm 1).
 * RPS_AVERAGE_GRADIENTS: the stochastic gradients, over the same unreliable Reduce-Scatter / All-Gather
 *                        (Section 5, "Comparison with Gradient Averaging"): the server of block j averages
 *                        the gradients that arrived; a worker that receives the average applies it,
 *                        x <- x - gamma * gtilde, any other worker applies its own gradient.  A drop then
 *                        leaves a difference between replicas that never decays, which is the paper's
 *                        argument for averaging models. */
typedef enum rps_average { RPS_AVERAGE_MODELS = 0, RPS_AVERAGE_GRADIENTS = 1 } rps_average;

typedef struct rps_options {
    int32_t dtype;         /* rps_dtype, default RPS_F32                                   */
    int32_t assign;        /* rps_assign, default RPS_ASSIGN_FIXED                         */
    int32_t self_delivery; /* 1 (default): a server's own copy never crosses the network,
                              so it is always part of the average and the server always has
                              the average (proof of Lemma 7).  0: all 2n messages of a block
                              can be lost; a block whose server received nothing is not
                              broadcast and every worker keeps v for it.                   */
    int32_t mask_window;   /* drop masks are generated this many steps at a time (1..256,
                              default 32); does not change any result                     */
    double sigma;          /* std-dev of the Gaussian gradient noise, default 0           */
    /* Shape of the fused kernel; 0 = the library's choice.  None of these changes what is
     * computed beyond the order of the fp32 additions inside the masked average.           */
    int32_t row_skew_lines;   /* extra 128-byte lines of padding per device row after d has been
                                 rounded up to a whole line; -1 = automatic: as many as make the
                                 row a whole number of kilobytes (the kernels' row pieces are then
                                 whole DRAM pages in every row)                               */
    int32_t kernel;           /* 1: lanes load their slices directly from global memory;
                                 2: slices are staged through shared memory by bulk
                                 asynchronous copies issued by a producer warp;
                                 3: the same staging with no producer warp: all 16 warps of a
                                 CTA compute, each taking the next slice of the next tile from a
                                 counter, and the last warp to have read a stage refills it (built for bf16 replicas
                                 with more than 4 workers, untracked steps; any other step runs
                                 as kernel 2);
                                 4: workers streamed: a lane owns one 16-byte slice of columns and
                                 walks all n workers in order, two at a time, adding each v to the
                                 running sum and storing it at once where the return message is
                                 lost; the average is rounded once and stored to every receiver.
                                 Teams of warps share shared-memory rings of a few rows that they
                                 refill themselves; a team reads whole 2 KB pieces of rows and a warp
                                 writes whole 512-byte pieces.  Gradient averaging sums the
                                 updates instead and reads a tile's rows of x a second time for
                                 the receivers (n >= 2, blocks of at least 16 bytes, tracked
                                 steps in model averaging only; any other step runs as kernel
                                 2 or 3).
                                 0: kernel 1 for models too short to give every SM a tile.  Else
                                 kernel 4 where n is not a power of two (kernels 2 and 3 pad their
                                 lane groups to the next one and take as long as that many workers
                                 would), for bf16 replicas of fewer than 8 or more than 32 workers
                                 and for tracked bf16 steps; gradient averaging on bf16 replicas
                                 takes kernel 4 only below 5 workers and, from 9 on, where n is at
                                 most four fifths of the next power of two.  Else kernel 3 for
                                 bf16 replicas (5 workers or more, untracked) and kernel 2 for the
                                 rest (fp32 with 4, 8, 16, 32, 64 workers; 2 workers run as kernel 4
                                 in model averaging, 4 workers when tracked).  An option that
                                 shapes kernel 2 alone (workers_per_lane, copy_mode, slice_bytes)
                                 keeps kernels 3 and 4 out of the choice.                      */
    int32_t workers_per_lane; /* 2, 4 or 8 workers' slices held in registers by one lane      */
    int32_t stages;           /* depth of the shared-memory ring(s) of kernels 2, 3 and 4 (2..8) */
    int32_t consumer_warps;   /* compute warps per CTA of kernel 2 (1..24; shapes that need
                                 many registers are clamped lower) and of kernel 4 (1..32)   */
    int32_t copy_mode;        /* kernel 2 fills a stage with 1: one bulk copy per row,
                                 2: two-dimensional TMA boxes covering all n rows            */
    int32_t slice_bytes;      /* kernel 2, bf16 replicas: bytes of a row handled by one lane,
                                 16 or 8 (8 = more, lighter warps per tile)                  */
    int32_t store_mode;       /* kernels 2 and 3 write results 1: from registers, 16 bytes per
                                 lane, 2: through an output tile in shared memory with TMA tensor
                                 stores, 3: in place in the stage, with TMA tensor stores from
                                 there (kernel 2: by a store warp; kernel 3: by the last warp of
                                 a team to have written).  Kernel 4: 1 from registers, 2 the
                                 average through a 512-byte slot in shared memory and one bulk
                                 copy per receiving row                                        */
    int32_t wait_limit_ms;    /* kernel 2: every wait of a warp on data or on a free stage gives
                                 up after this many milliseconds (0 = 2000); the next
                                 synchronising call then returns RPS_ECUDA                   */
    int32_t withhold_copies;  /* kernel 2, test aid for that time-out path: 1 = the producer warp
                                 issues no copies, so the compute warps' waits run out, x is
                                 left unchanged and the error is reported; 0 otherwise       */
    int32_t average;          /* rps_average, default RPS_AVERAGE_MODELS                        */
    /* How consecutive steps share the L2 cache; neither changes any result. */
    int32_t traversal;        /* 0 (default): even steps walk the columns upwards, odd steps
                                 downwards, so a step starts on the part of x and b that the step
                                 before it touched last and that is still in L2; 1: always upwards */
    int32_t l2_policy;        /* kernel 2: 1 = plain loads; 2 = the targets b are loaded with the
                                 L2 evict-first hint, which leaves the cache to the lines of x
                                 (a retained line of x saves a read and a write-back, one of b
                                 only a read); 0 = the library's choice                        */
    int32_t launch_overlap;   /* all kernels: 2 = the fused kernel is launched with programmatic stream
                                 serialization: its CTAs may be placed and set up while the kernel
                                 before it in the stream drains, and wait (griddepcontrol.wait) for
                                 that kernel to complete before they read anything it may have
                                 written; 1 = plain launches; 0 = the library's choice          */
    /* Column shard.  Columns never interact (block j of every worker meets only block j of the
     * others, and masks and noise are pure functions of (seed, t, block, worker, column)), so a
     * model can be cut by columns over several handles, on one GPU or on several, with no
     * exchange between them: each handle holds columns [shard_begin, shard_begin + shard_cols)
     * of all n workers and produces bit for bit what a handle holding the whole model produces
     * for those columns.  The device and host arrays of a shard handle are [n][shard_cols]
     * (pitch from rps_pitch); d of rps_create stays the size of the whole model, which fixes the
     * blocks.  shard_cols = 0 (default): the whole model.  shard_begin must be a multiple of 64. */
    int64_t shard_begin;
    int64_t shard_cols;
    /* Temporal blocking of rps_step_n.  With the quadratic objective of this library the gradient of
     * a column needs only that column, so up to block_steps consecutive steps (2..mask_window) can be
     * applied to a slice of x while it sits in registers: x and b are read once and x written once per
     * block_steps steps, each step with its own masks and noise and with x rounded to the replica
     * type as a store would.  The result equals that of single steps in the lane shape with 4 workers per lane
     * bit for bit.  This is not the paper's setting (there a model's forward and backward pass sits
     * between two synchronisations), so it is off by default (0 or 1); it applies to rps_step_n only,
     * and only to untracked model averaging.                                                         */
    int32_t block_steps;
    int32_t team_warps;       /* kernel 3: warp slices per tile, 1..16 (0 = the library's choice: 8, or
                                 fewer where the ring would otherwise be too shallow); kernel 4: warps
                                 per team, 1, 2 or 4 (0 = 4): a team's row piece is team_warps x 512 bytes */
    int32_t early_targets;    /* kernels 2 and 4 under launch_overlap = 2: 2 = the copies of the targets b
                                 for a CTA's first stages are issued BEFORE the CTA waits for the kernel
                                 ahead of it in the stream, so they arrive while that kernel drains; only
                                 the copies of x wait.  This relies on b not being written by that
                                 kernel: no kernel of this library writes b, and the library's own
                                 uploads (rps_set_targets, rps_step_host) are copies, which a kernel
                                 launch never overtakes.  A caller whose OWN kernel writes b on the bound
                                 stream directly before a step must set 1 (every copy waits) or put a
                                 stream synchronisation or an event between the two.  0 = the library's
                                 choice (2 for kernel 2, 1 for kernel 4).                          */
    int32_t fuse_steps;       /* rps_step_n: 2 = consecutive untracked steps are issued as ONE launch of the
                                 fused kernel (up to the steps left in the window of masks) where the
                                 kernel that serves this handle can go from step to step by itself
                                 (kernel 4: a team of warps works on the same tiles in every step, and a
                                 column's next step needs only that column's last step, so a team sees
                                 its own stores done, fences, and goes on; no launch boundary, no wait
                                 for the rest of the GPU).  Results are bit for bit those of single
                                 steps.  1 = one launch per step.  0 = the library's choice (2).     */
} rps_options;

/*
 * rps_create: inputs of Algorithm 1 and of the channel model of Section 3.
 *   n      number of workers = parameter servers = blocks, 1..RPS_MAX_WORKERS
 *   d      model size, 1 <= d < 2^34
 *   p      message drop probability, 0 <= p <= 1; a message is lost iff a 32-bit
 *          Philox4x32-10 draw is below floor(p * 2^32)
 *   gamma  learning rate (finite); rounded to float once, here
 *   seed   key of every random stream (masks, server draw, gradient noise)
 * The new handle starts at step t = 0 with default options; *out is owned by
 * the library until rps_destroy().  Errors: RPS_EINVAL, RPS_ENOMEM.
 */
int rps_create(int n, int64_t d, double p, double gamma, uint64_t seed, rps_handle** out);

/* Frees the handle (NULL is allowed).  Does not touch the caller's buffers.  */
int rps_destroy(rps_handle* h);

/* Fills *opt with the defaults listed above. */
int rps_default_options(rps_options* opt);

/* Sets the options; allowed only before rps_bind() (else RPS_ESTATE).        */
int rps_configure(rps_handle* h, const rps_options* opt);

/* Row pitch, in elements, that x and b must have on the device.              */
int64_t rps_pitch(const rps_handle* h);

/* Bytes of device scratch (drop masks of mask_window steps) rps_bind() wants. */
size_t rps_scratch_bytes(const rps_handle* h);

/*
 * rps_bind: lends the device buffers.
 *   x_dev, b_dev  [n][pitch] replicas and targets, 128-byte aligned, caller-owned,
 *                 borrowed until rps_destroy() or the next rps_bind()
 *   pitch         must equal rps_pitch(h)
 *   scratch_dev   >= rps_scratch_bytes(h) bytes, 256-byte aligned
 *   cuda_stream   a cudaStream_t (NULL = the default stream)
 * Errors: RPS_EINVAL on NULL, misalignment, wrong pitch or short scratch.
 */
int rps_bind(rps_handle* h, void* x_dev, void* b_dev, int64_t pitch, void* scratch_dev, size_t scratch_bytes,
             void* cuda_stream);

/* Copies dense host [n][d] targets b_i of the objective f_i(x) = 0.5*||x - b_i||^2
 * (worker i's local objective f_i of Eq. 1) to the device.  Asynchronous with
 * respect to the host only if b_host is pinned.                               */
int rps_set_targets(rps_handle* h, const void* b_host);

/* Overwrites all replicas from a dense host [n][d] array (Algorithm 1 starts all
 * workers from the same value; any state is accepted).                        */
int rps_write(rps_handle* h, const void* x_host);

/* Step counter t of the next rps_step (the first step is t = 0).  Because every
 * random stream is a pure function of (seed, t, ...), rps_write + rps_set_step
 * resume a run exactly.                                                       */
int rps_set_step(rps_handle* h, uint64_t t);
int rps_get_step(const rps_handle* h, uint64_t* t);

/*
 * rps_step: one iteration of Algorithm 1 for all workers, enqueued on the stream:
 *   v^(i)      = x^(i) - gamma * ((x^(i) - b_i) + sigma * xi_t^(i))      local SGD step
 *   vtilde^(j) = 1/|N^(j)| * sum_{k in N^(j)} v^(k,j)                    Reduce-Scatter
 *   x^(i,j)    = vtilde^(j) if worker i received it, else v^(i,j)        All-Gather
 * with N^(j) the workers whose block j reached its server (Section 4.1).  The
 * drop masks of step t come from the mask kernel (generated mask_window steps at
 * a time), the rest is one fused kernel that reads x and b once and writes x
 * once.  Asynchronous; launch errors are returned, execution errors surface at
 * the next synchronising call.  Needs rps_bind() (else RPS_ESTATE).
 */
int rps_step(rps_handle* h);

/*
 * rps_step_n: T consecutive steps (the loop over t of Algorithm 1), with the results of T calls of
 * rps_step bit for bit.  Where the kernel that serves the handle allows it (rps_options.fuse_steps),
 * consecutive untracked steps go out as one launch per window of masks: x and b are still read once
 * and x written once PER STEP, only the launch boundaries between the steps are gone.  (Several steps per
 * PASS over x and b, which changes the traffic, is rps_options.block_steps.)  T < 0: RPS_EINVAL.
 */
int rps_step_n(rps_handle* h, int64_t T);

/*
 * rps_step_forced: the same fused kernel with drop masks given by the caller
 * instead of sampled: bit i of up[j] = worker i's block j reached its server,
 * bit i of down[j] = worker i received the averaged block j (host arrays of n
 * words, used as given; a block with up[j] == 0 is not broadcast).  Advances t.
 * Lets a test enumerate the outcomes behind W_t^(j) of Eq. 3.
 */
int rps_step_forced(rps_handle* h, const uint64_t* up, const uint64_t* down);

/*
 * rps_step_host: one step with host-resident state.  Copies dense host [n][d]
 * x_host (and b_host unless NULL, in which case the resident targets are used)
 * to the device, runs rps_step, copies the new replicas back into x_host and
 * synchronises.  Pinned host memory makes the copies fast; pageable works.
 * Because columns never interact, a large model goes through in up to 8 pieces of
 * columns: the upload of one piece overlaps the step and the download of the piece
 * before it (two internal copy streams and a few events, created on the first call
 * and released by rps_destroy; no device memory).  The result is that of rps_step.
 */
int rps_step_host(rps_handle* h, void* x_host, const void* b_host);

/* Synchronises and copies the replicas to a dense host [n][d] array.          */
int rps_read(rps_handle* h, void* x_host_out);

/*
 * rps_read_masks: runs the device mask generator for step t (any t; does not
 * disturb the run) and returns, for each block j: up[j], down[j] as above,
 * count[j] = |N^(j)|, server[j] = the worker that averages block j.  Host arrays
 * of n entries; server may be NULL.
 */
int rps_read_masks(rps_handle* h, uint64_t t, uint64_t* up, uint64_t* down, int32_t* count, int32_t* server);

/*
 * rps_diag: off the hot path.  dist2_to_opt = ||xbar - mean_i b_i||^2 (squared
 * distance of the averaged model to the optimum of the quadratic objective) and
 * consensus = sum_i ||x^(i) - xbar||^2 (the quantity bounded by Lemma 3).
 * Synchronises.  Either output may be NULL.
 */
int rps_diag(rps_handle* h, double* dist2_to_opt, double* consensus);

/*
 * rps_estimate_alpha: Monte-Carlo estimate of the constants of Eqs. (4) and (5),
 *   E[W W^T] = alpha_1 I + (1 - alpha_1) A_n,   E[W A_n W^T] = alpha_2 I + (1 - alpha_2) A_n,
 * (W = W_t^(j) of Eq. 3, A_n = 1 1^T / n), which Figures 2 and 3 plot and whose difference beta
 * sets the rate of Theorem 1.  Runs the mask generator for steps t0 .. t0+steps-1 of this handle's
 * streams (n, p, seed, assign, self_delivery) and averages, over the n blocks of every step, the
 * value (mean diagonal) - (mean off-diagonal) of W W^T and of W A_n W^T, computed on the device from
 * the counts of arrivals and receivers.  Does not touch x, b or the step counter.  Synchronises.
 * RPS_EINVAL for n < 2 (no off-diagonal entries) or steps < 1.
 */
int rps_estimate_alpha(rps_handle* h, uint64_t t0, int64_t steps, double* alpha1, double* alpha2);

/*
 * rps_track: the same two quantities as rps_diag, as a by-product of the fused pass itself (no extra
 * read of x or b): the step measures what it leaves behind from the values it holds in registers,
 * so a run can follow the distance to the optimum (Section 5 plots convergence against the optimum;
 * Lemma 3 bounds the consensus error) at every step.
 *   trace_dev : device array of 2 * capacity doubles, 16-byte aligned, owned by the caller, who keeps
 *               it alive until tracking is switched off or the handle destroyed.  Cleared here
 *               (asynchronously, on the bound stream).
 *   capacity  : number of steps to record; later steps run untracked.
 * The k-th step enqueued after this call (k = 0 .. capacity-1; rps_step, rps_step_n, rps_step_forced,
 * rps_step_host alike) adds into trace_dev[2k] the value ||xbar - mean_i b_i||^2 and into
 * trace_dev[2k+1] the value sum_i ||x^(i) - xbar||^2 of the state x_{t+1} it produces (for bf16
 * replicas: of the rounded values it stores).  fp32 arithmetic relative to a per-column pivot
 * within a tile of columns, fp64 across tiles; the order of the fp64 additions is not fixed, so the
 * last bits vary from run to run.  trace_dev == NULL or capacity == 0 switches tracking off.
 * Errors: RPS_ESTATE before rps_bind, RPS_EINVAL for a negative capacity or a misaligned pointer.
 */
int rps_track(rps_handle* h, double* trace_dev, int64_t capacity);

/*
 * rps_read_trace: synchronises and copies the entries recorded so far (at most max_entries) to
 * trace_host_out as pairs {dist2_to_opt, consensus}; *entries receives how many pairs were
 * written.  RPS_ESTATE when tracking is off.
 */
int rps_read_trace(rps_handle* h, double* trace_host_out, int64_t max_entries, int64_t* entries);

/*
 * Per-kernel device timing.  rps_profile(h, 1) makes every later kernel launch of
 * this handle be bracketed by CUDA events on the bound stream; rps_profile_read
 * synchronises and returns the summed device time and launch count of the fused
 * step kernel and of the mask kernel since profiling was switched on, then
 * resets them.  rps_profile(h, 0) switches it off.
 */
int rps_profile(rps_handle* h, int enable);
int rps_profile_read(rps_handle* h, double* fused_ms, int64_t* fused_launches, double* mask_ms,
                     int64_t* mask_launches);

/*
 * rps_step_static: one step of the same method with no handle, no rps_bind() and
 * no scratch buffer from the caller.  (The paper has no counterpart: this entry
 * point exists for the sake of callers, not of the algorithm.)
 *
 * Who needs it: code that cannot call cudaMalloc or any allocating routine where
 * it runs.  Examples are a plug-in living inside another framework's fixed
 * memory pool, a control loop that may not block on the driver's allocator, or a
 * host that hands out device buffers and forbids further allocation.  Such a
 * caller already owns x and b; the only other device memory a step needs is the
 * record of that step's drop masks, which here lives in a fixed 1792-byte array
 * compiled into the library (room for RPS_MAX_WORKERS workers).  Every GPU that
 * loads the library carries that array until the process exits.
 *
 *   n, d, p, gamma, seed   as for rps_create; n > RPS_MAX_WORKERS returns RPS_ELIMIT
 *                          because the built-in mask record cannot hold more workers
 *   dtype                  rps_dtype of x_dev and b_dev
 *   x_dev                  device [n][pitch] replicas, 128-byte aligned; input and output
 *   b_dev                  device [n][pitch] targets, 128-byte aligned; input
 *   pitch                  row pitch in elements: >= d and a multiple of 32 (fp32) or 64 (bf16)
 *   sigma                  std-dev of the gradient noise, >= 0
 *   t                      step counter; the caller advances it (0, 1, 2, ...)
 *   cuda_stream            cudaStream_t the two kernels are enqueued on (NULL = default)
 *
 * Fixed assignment and self-delivery, as in the default options.  Calls with the
 * same arguments give the same replicas as rps_step() on a handle at step t.
 * The call allocates nothing on the device and frees nothing.  Its first call on
 * a device looks up the array's device address and the SM count (once per
 * device, with that device current); make that first call outside any stream
 * capture.  All calls on a device share the one array, which keeps whatever the
 * previous call left in it; each call rewrites the part it reads, so nothing
 * needs clearing, but two calls that overlap on the GPU (different streams, or
 * different host threads on different streams) race on it: keep them on one
 * stream or order them with events.  Returns RPS_OK, RPS_EINVAL, RPS_ELIMIT or
 * RPS_ECUDA; asynchronous like rps_step().  One difference from the handle path:
 * there is no error word here for a kernel to write, so a bounded wait inside the
 * fused kernel that gives up (which rps_read() on a handle reports as RPS_ECUDA)
 * ends that kernel early WITHOUT any report, with x partly updated.  Callers that
 * need that report use a handle.
 */
int rps_step_static(int n, int64_t d, int dtype, void* x_dev, const void* b_dev, int64_t pitch, double p,
                    double gamma, double sigma, uint64_t seed, uint64_t t, void* cuda_stream);

/* Kernels launched by this handle since creation (both kinds).               */
int64_t rps_launch_count(const rps_handle* h);

/* Reason for the last failure on h ("" if none); valid until the next call.
 * With h == NULL: reason for the last failed rps_create on this thread.       */
const char* rps_last_error(const rps_handle* h);

/* Library version, "major.minor". */
const char* rps_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RPS_H */
