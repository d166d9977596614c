// Fused RPS step, streamed workers (sm_100a).
//
// The AG step gives every worker that receives block j the SAME value (Section 4.1: x <- the average if
// the return message arrived, else the worker's own v), so a worker's v has to outlive the running sum only
// if its return message is lost (a fraction p of the workers).  This form is built on that:
//
//   * A lane owns one 16-byte slice of columns (4 floats / 8 bf16) and walks ALL n workers in index order,
//     two at a time (one noise draw serves a worker pair).  For each worker it forms v, adds it to the
//     running sum of its columns where the up bit is set, and stores v AT ONCE where the down bit is clear.
//     After the last worker the average is formed, rounded and packed ONCE, and stored to every receiver's
//     row.  Nothing like v[workers][columns] stays live: no select, no shuffle, summation in worker order
//     (the order of the plain definition), about half the registers of the lane-group forms.
//   * A warp therefore covers 32 slices = 512 contiguous bytes of every row it touches, in loads and in
//     stores alike (the lane-group forms store 64-byte pieces at n = 64), and the shared memory a warp needs
//     does not grow with n: what is staged is a worker pair, not a tile of all workers.
//   * Warps work in teams of team_warps neighbours.  A team owns a ring in shared memory whose stage holds
//     one or two worker pairs of the team's tile: ROWS rows x (team_warps x 512 bytes) of x and of b, fetched by
//     two TMA box copies (the arrays are described to the unit in 8-byte units, so one box spans up to 2 KB of a
//     row; with rows that start on 1 KB boundaries every row piece is a whole number of DRAM pages).  A warp
//     works through its part of a stage and counts itself off; the warp that counts last refills the stage with
//     the rows that come `stages` stages later (of the same tile or of the team's next one).  Nobody waits for
//     a free stage; the only wait is the bounded one for a stage's copies to land.  Teams take the tiles in
//     fixed turns, so every warp knows the whole sequence of stages in advance.
//   * The arithmetic runs two columns at a time in the packed fp32 forms (fma / mul / add .f32x2): one issue
//     slot, two IEEE operations, the same bits as the scalar forms of the other kernels.
//   * Tracked steps (DIAG) need little more than the walk: every receiver holds the same value, so only the
//     keepers have a deviation from it, and their rows are read back when the tile's average is known.
//   * One launch can run several consecutive steps (rps_step_n): a team has the same tiles in every step and a
//     column's next step needs only that column's last step, so a team goes on to the next step by itself once
//     its own stores are done and fenced.  There is no launch boundary between the steps and no wait for the
//     rest of the GPU; odd steps walk the team's tiles backwards, onto what is still in L2.
//
//   * Gradient averaging (GRAD) sums the updates v - x instead, and a receiver's new value x + (average update)
//     needs its own x after the last worker: the tile's rows of x go through the ring a second time, last rows
//     first (what was read last is still in L2), and each receiver's row is finished then.  Keepers are stored
//     in the first pass as always.
//
// A lane whose slice straddles two blocks or the end of the row (at most n such lanes per step) takes a
// per-column branch with the same arithmetic, so a column's result does not depend on where it lies.
//
// Every mbarrier wait is bounded; a warp that gives up records a code in *prm.error, sees the copies that may
// still be in flight land (bounded again) and leaves; its team mates run into their own limits.
#include "rps_device.cuh"
#include "rps_tma.cuh"

namespace rps {

namespace {

constexpr int kStreamMaxWarps = 32;
constexpr int kStreamMaxStages = 8;
constexpr int kStreamDefaultStages = 3;
constexpr int kStreamDefaultStoreMode = 1;            // 1: 16-byte stores from registers; 2: bulk copies from shared memory
constexpr int kStreamMaxTeamWarps = 4;                // a team's row piece is one TMA box: at most 256 8-byte units
constexpr uint32_t kPieceBytes = 512;                 // of one row per warp: 32 lanes x 16 bytes
// shared-memory header: a line per team (barriers, counters), then the tracked steps' sums
constexpr uint32_t kTeamLineBytes = 128;              // [8] mbarriers, [8] int counters of warps done with a stage, the step barrier
constexpr uint32_t kStepBarOffset = kStreamMaxStages * (8 + 4);  // in a team's line
constexpr uint32_t kTrackOffset = kStreamMaxWarps * kTeamLineBytes;  // tracked steps: 2 doubles, a counter
constexpr uint32_t kStreamHeaderBytes = kTrackOffset + 128;
static_assert(kStreamHeaderBytes % 128 == 0, "stages start on 128-byte boundaries");
static_assert(kStepBarOffset + 8 <= kTeamLineBytes && kStepBarOffset % 8 == 0, "a team's barriers and counters fit its line");
static_assert(kStreamMaxTeamWarps * kPieceBytes / 8 <= 256, "a team's row piece is one box");

struct StreamShape {
    int32_t tiles;            // team tiles in the row
    int32_t stages;           // depth of every team's ring
    int32_t team_warps;       // warps per team: a tile is team_warps x 32 slices wide
    int32_t teams;            // teams per CTA
    int32_t withhold_copies;  // test aid: nothing is ever copied, so that the waits run out
    int32_t steps;            // consecutive steps this launch runs, each with the mask record that follows the last one's
    int32_t alternate;        // 1: in odd steps a team takes ITS tiles from the last to the first (FusedTuning::traversal = 0)
    int32_t bulk_stores;      // 1: the average leaves through shared memory and bulk copies (see the kernel)
    int32_t early_targets;    // 1: the first stages' copies of b are issued before the wait for the kernel ahead in the stream
    uint32_t out_offset;      // of the warps' output slots from the start of the rings
    uint64_t wait_limit_ns;
};

// Tracked steps (distance of the averaged model to the optimum, consensus error; see Tracker in rps_device.cuh),
// in the streamed form.  Every receiver of a block holds the same stored value P, so with P as the pivot only
// the workers that keep their own v (down bit clear, a fraction p of them) have a deviation.  The walk itself
// carries only the sum of the targets (two columns at a time, with the step: local_sgd_pair_packed).  When a tile's
// average has been stored the lane reads its keepers' rows back (its own stores of a moment ago) and forms
//   D = sum over keepers (v_k - P),  Q = sum over keepers (v_k - P)^2          (v_k as stored),
//   mean x = P + D / n,   consensus = Q - D^2 / n.   Nothing large is squared and subtracted.
// With no receiver at all every worker is a keeper and worker 0's stored value is the pivot.

// One column's contribution to (|| mean x - mean b ||^2, consensus error) from the keepers' deviations from the
// pivot: their sum and the sum of their squares.
__device__ __forceinline__ void close_tracked_column(float bsum, float pivot, float dev_sum, float dev_sq, float inv_n,
                                                     float& dist2, float& cons)
{
    const float gap = fmaf(dev_sum - bsum, inv_n, pivot);  // mean x - mean b of this column
    dist2 = fmaf(gap, gap, dist2);
    cons += fmaf(-dev_sum * inv_n, dev_sum, dev_sq);
}

// The two steps of a lane whose slice is cut by a block boundary or by the end of the row, per column:
// columns [0, cut) of the slice belong to block j, columns [cut, VEC) to block j + 1, columns from live_n on
// do not exist.  Same arithmetic as the regular path (predicated add in worker order, one multiplication).
// Out of line and on copies of the caller's registers: this is rare.
// `v` is what the sum takes and `own` what a keeper stores: the same values in model averaging, the update and
// x + the update in gradient averaging.
template <typename T, int VEC>
__device__ __noinline__ void irregular_pair(float (&sum)[VEC], const float (&v)[2][VEC], const float (&own)[2][VEC],
                                            int k, int j, int j_next, int cut, int live_n, uint64_t valid,
                                            const uint64_t* s_up, const uint64_t* s_down, T* dst, int64_t pitch)
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int w = k + h;
        const uint32_t up_lo = (uint32_t)(s_up[j] >> w) & 1u, up_hi = (uint32_t)(s_up[j_next] >> w) & 1u;
        const uint32_t keep_lo = (uint32_t)((~s_down[j] & valid) >> w) & 1u;
        const uint32_t keep_hi = (uint32_t)((~s_down[j_next] & valid) >> w) & 1u;
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const bool live = e < live_n, hi = e >= cut;
            add_if(sum[e], v[h][e], live ? (hi ? up_hi : up_lo) : 0u);
            const bool kept = live && (hi ? keep_hi : keep_lo);
            if (kept) dst[(int64_t)w * pitch + e] = RowVec<T, VEC>::narrow(own[h][e]);
        }
    }
}

template <typename T, int VEC, bool DIAG>
__device__ __noinline__ void irregular_receivers(const float (&sum)[VEC], int n, int j, int j_next, int cut,
                                                 int live_n, const uint64_t* s_down, const float* s_inv, T* dst,
                                                 int64_t pitch, const float (&target_sum)[VEC], float inv_n,
                                                 float* dist2, float* cons)
{
    T avg[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) avg[e] = RowVec<T, VEC>::narrow(sum[e] * (e >= cut ? s_inv[j_next] : s_inv[j]));
    const uint64_t down_lo = s_down[j], down_hi = s_down[j_next];
#pragma unroll 1
    for (int i = 0; i < n; ++i) {
        const bool lo = (down_lo >> i) & 1u, hi = (down_hi >> i) & 1u;
#pragma unroll
        for (int e = 0; e < VEC; ++e)
            if (e < live_n && (e >= cut ? hi : lo)) dst[(int64_t)i * pitch + e] = avg[e];
    }
    if (DIAG) {
        // the keepers' rows as this lane stored them, against what the receivers hold
        const uint64_t valid = n >= 64 ? ~(uint64_t)0 : (((uint64_t)1 << n) - 1);
        float dd = 0.0f, q = 0.0f;
#pragma unroll
        for (int e = 0; e < VEC; ++e)
            if (e < live_n) {
                const uint64_t down = (e >= cut ? down_hi : down_lo) & valid;
                const float pivot = down != 0 ? (float)avg[e] : (float)dst[e];
                float dev_sum = 0.0f, dev_sq = 0.0f;
                for (uint64_t rest = ~down & valid; rest != 0; rest &= rest - 1) {
                    const int i = __ffsll((long long)rest) - 1;
                    const float dev = (float)dst[(int64_t)i * pitch + e] - pivot;
                    dev_sum += dev;
                    dev_sq = fmaf(dev, dev, dev_sq);
                }
                close_tracked_column(target_sum[e], pivot, dev_sum, dev_sq, inv_n, dd, q);
            }
        *dist2 = dd, *cons = q;
    }
}

// 16 bytes of a row from VEC / 2 column pairs, rounded to T (nearest even).
template <typename T, int VEC>
__device__ __forceinline__ uint4 pack_pairs(const Float2 (&v)[VEC / 2])
{
    uint32_t w[4];
    if (sizeof(T) == 4) {
#pragma unroll
        for (int m = 0; m < 2; ++m) {
            float lo, hi;
            unpack2(v[m % (VEC / 2)], lo, hi);
            w[2 * m] = __float_as_uint(lo), w[2 * m + 1] = __float_as_uint(hi);
        }
    } else {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            float lo, hi;
            unpack2(v[m % (VEC / 2)], lo, hi);
            const __nv_bfloat162 pair = __floats2bfloat162_rn(lo, hi);
            w[m] = *reinterpret_cast<const uint32_t*>(&pair);
        }
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// 16 bytes of a row as VEC / 2 column pairs in fp32.
template <typename T, int VEC>
__device__ __forceinline__ void unpack_pairs(const uint4 raw, Float2 (&x)[VEC / 2])
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    if (sizeof(T) == 4) {
#pragma unroll
        for (int m = 0; m < 2; ++m) x[m % (VEC / 2)] = pack2(w[2 * m], w[2 * m + 1]);
    } else {
#pragma unroll
        for (int m = 0; m < 4; ++m) x[m % (VEC / 2)] = pack2(w[m] << 16, w[m] & 0xFFFF0000u);
    }
}

// Gradient averaging, second pass, a lane whose slice is cut by a block boundary or the end of the row: worker w
// takes x + (average update) in the columns whose block's average reached it.
template <typename T, int VEC>
__device__ __noinline__ void irregular_update_row(const uint4 raw_x, const float (&avg)[VEC], int w, int j, int j_next,
                                                  int cut, int live_n, const uint64_t* s_down, T* row)
{
    float x[VEC];
    RowVec<T, VEC>::unpack(raw_x, x);
    const bool lo = (s_down[j] >> w) & 1u, hi = (s_down[j_next] >> w) & 1u;
#pragma unroll
    for (int e = 0; e < VEC; ++e)
        if (e < live_n && (e >= cut ? hi : lo)) row[e] = RowVec<T, VEC>::narrow(x[e] + avg[e]);
}

// Waits for the phase with the given parity: one cheap test first (the data has usually landed long ago), then
// the bounded wait.
__device__ __forceinline__ bool stream_wait(uint32_t bar, uint32_t parity, uint64_t limit_ns)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    return mbar_wait(bar, parity, limit_ns);
}

template <typename T, int VEC, int MAXW, int ROWS, bool DIAG, bool GRAD>
__global__ void __launch_bounds__(MAXW * 32, 1)
    rps_fused_stream_kernel(const __grid_constant__ FusedParams prm, const StreamShape shape,
                            const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_b)
{
    constexpr int WARP_COLS = 32 * VEC;
    static_assert(ROWS == 2 || ROWS == 4, "a stage holds one or two worker pairs");
    static_assert(!(DIAG && GRAD), "tracked steps are model averaging");
    extern __shared__ __align__(128) unsigned char smem[];
    const int n = prm.n;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int team = warp / shape.team_warps, member = warp - team * shape.team_warps;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + team * kTeamLineBytes);         // [stages] the rows have landed
    int* done = reinterpret_cast<int*>(smem + team * kTeamLineBytes + kStreamMaxStages * 8);  // [stages] warps done with them
    uint64_t* step_bar = reinterpret_cast<uint64_t*>(smem + team * kTeamLineBytes + kStepBarOffset);  // between two steps
    // tracked steps: the CTA's pair of sums and the count of warps that have added theirs
    double* track_pair = reinterpret_cast<double*>(smem + kTrackOffset);
    int* track_arrivals = reinterpret_cast<int*>(smem + kTrackOffset + 16);
    // a stage: ROWS rows of x, then ROWS rows of b, each row the team's piece (team_warps x 512 bytes)
    const uint32_t row_bytes = (uint32_t)shape.team_warps * kPieceBytes;
    const uint32_t array_bytes = ROWS * row_bytes;
    const uint32_t stage_bytes = 2 * array_bytes;
    unsigned char* ring = smem + kStreamHeaderBytes + (size_t)team * shape.stages * stage_bytes;
    const uint32_t ring_addr = smem_addr(ring);
    const int team_cols = shape.team_warps * WARP_COLS;
    const int32_t units_per_tile = (int32_t)(row_bytes / 8);  // 8-byte units of one row of a tile

    // tiles of this team: turns g, g + teams_total, ...
    const int teams_total = (int)gridDim.x * shape.teams;
    const int g = (int)blockIdx.x * shape.teams + team;
    const int my_tiles = g < shape.tiles ? (shape.tiles - g + teams_total - 1) / teams_total : 0;
    // Gradient averaging goes through a tile's rows twice: a receiver's new value x + (average update) needs its
    // own x once all workers have been seen, so the rows of x come round again (from L2, mostly) in a second pass.
    const int pass_chunks = (n + ROWS - 1) / ROWS;
    const int chunks_per_tile = GRAD ? 2 * pass_chunks : pass_chunks;
    const uint32_t total = (uint32_t)my_tiles * (uint32_t)chunks_per_tile;  // stages' worth of rows this team goes through per step
    const uint64_t t_first = ((uint64_t)prm.t_hi << 32) | prm.t_lo;
    auto walks_down = [&](int step) { return shape.alternate != 0 && ((t_first + (uint64_t)step) & 1u) != 0; };
    // The team's tile number `local` of a step: the same set of tiles in every step (a team depends on nobody else's
    // stores from one step to the next), walked upwards or downwards, so that a step starts on the tiles the step
    // before it touched last, which are still in L2.
    auto tile_of = [&](int local, bool down) { return g + (down ? my_tiles - 1 - local : local) * teams_total; };

    if (member == 0 && lane == 0) {
        for (int s = 0; s < shape.stages; ++s) {
            mbar_init(smem_addr(&full[s]), 1);
            done[s] = 0;
        }
        mbar_init(smem_addr(step_bar), (uint32_t)shape.team_warps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        if (DIAG) {
            track_pair[0] = 0.0;
            track_pair[1] = 0.0;
            *track_arrivals = 0;
        }
    }
    // Copies rows [ROWS * chunk, ROWS * chunk + ROWS) of the team's tile number `local` into `stage` (which must be
    // free): one thread, one box per array (the replicas, the targets, or both); `expect` announces the bytes of
    // BOTH to the stage's barrier.  Boxes arrive whole (rows past n and columns past the pitch as zeros), so the
    // byte count is fixed.  The maps count columns in 8-byte units.
    auto issue = [&](int stage, bool down, int local, int chunk, bool with_x, bool with_b, bool expect) {
        if (shape.withhold_copies) return;
        const int tile = tile_of(local, down);
        const uint32_t bar = smem_addr(&full[stage]);
        const uint32_t dst = ring_addr + (uint32_t)stage * stage_bytes;
        // The second pass of gradient averaging takes the replicas only, from the last rows to the first: what the
        // first pass read last is read again first, while it is still in L2.  The targets of that form are loaded
        // with the evict-first hint, so that they do not push the replicas out meanwhile.
        const bool again = GRAD && chunk >= pass_chunks;
        const int first_row = ROWS * (again ? 2 * pass_chunks - 1 - chunk : chunk);
        if (expect) mbar_arrive_expect_tx(bar, again ? array_bytes : stage_bytes);
        if (with_x) tma_load_box(dst, &map_x, tile * units_per_tile, first_row, bar);
        if (with_b && !again) {
            if (GRAD) tma_load_box(dst + array_bytes, &map_b, tile * units_per_tile, first_row, bar, l2_evict_first_policy());
            else tma_load_box(dst + array_bytes, &map_b, tile * units_per_tile, first_row, bar);
        }
    };
    // the stages a step starts with, filled by the team's first thread: the ring goes on from `stage`
    auto first_fills = [&](int stage, bool down, bool with_x, bool with_b, bool expect) {
        if (member != 0 || lane != 0) return;
        int local = 0, chunk = 0;
        for (int s = 0; s < shape.stages && (uint32_t)s < total; ++s) {
            issue(stage, down, local, chunk, with_x, with_b, expect);
            if (++stage == shape.stages) stage = 0;
            if (++chunk == chunks_per_tile) chunk = 0, ++local;
        }
    };
    // With programmatic stream serialization this CTA may have been placed while the kernel before it in
    // the stream was still draining: let the next kernel do the same, then wait for the one before to
    // complete before reading anything it may have written.  Both are no-ops in a plain launch.  The targets
    // are not written by a step: the copies of b for the first stages go out before the wait (early_targets)
    // and arrive while that kernel drains; only the copies of x wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();  // the barriers are initialised; the only CTA-wide barrier
    if (shape.early_targets) first_fills(0, walks_down(0), false, true, true);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    first_fills(0, walks_down(0), true, !shape.early_targets, !shape.early_targets);

    T* __restrict__ xg = static_cast<T*>(prm.x);
    const uint64_t valid = n >= 64 ? ~(uint64_t)0 : (((uint64_t)1 << n) - 1);
    const PackedScalars scalars(prm);
    // bulk stores: two 512-byte slots per warp, used in turn by the warp's tiles
    unsigned char* out_slots = smem + kStreamHeaderBytes + shape.out_offset + (size_t)warp * 2 * kPieceBytes;
    const unsigned char* my_ring = ring + member * kPieceBytes + lane * 16;
    int stage = 0;
    uint32_t phase = 0;
    Tracker<VEC, 2, 1> tracker;  // this lane's sums over its tiles, and the hand-over to the CTA's pair
    // Several steps in one launch: a team's tiles are the same in every step, and a column's next step needs
    // only that column's last step, so a team goes from step to step on its own.  Between two steps it sees
    // its stores done and ordered ahead of the unit's next reads (below); no other team is waited for.
    for (int step = 0; step < shape.steps; ++step) {
    const bool down_step = walks_down(step);
    const uint64_t t_now = t_first + (uint64_t)step;
    const uint32_t t_lo = (uint32_t)t_now, t_hi = (uint32_t)(t_now >> 32);
    const StepMasks* rec = prm.masks + step;  // this step's drop masks
    const uint64_t* s_up = rec->up;
    const uint64_t* s_down = rec->down;
    const float* s_inv = rec->inv_cnt;
    // where the filling stands: every warp keeps the count (the warp that frees a stage refills it)
    int fill_local = 0, fill_chunk = 0;
    for (int s = 0; s < shape.stages; ++s)
        if (++fill_chunk == chunks_per_tile) fill_chunk = 0, ++fill_local;
    uint32_t q = 0;
    // Waits (bounded) for the ring's current stage to have landed.
    auto await_stage = [&]() -> bool {
        if (__all_sync(0xFFFFFFFFu, stream_wait(smem_addr(&full[stage]), phase, shape.wait_limit_ns))) return true;
        // Something this warp waited for never came: say so, and see the copies that may have been issued
        // into the team's ring land (bounded) before this warp's part of the shared memory is given up.
        report_timeout(prm, 2);
        if (!shape.withhold_copies && lane == 0) {
            for (int s = 1; s < shape.stages && q + (uint32_t)s < total; ++s) {
                if (++stage == shape.stages) stage = 0, phase ^= 1u;
                if (!mbar_wait(smem_addr(&full[stage]), phase, shape.wait_limit_ns)) break;
            }
        }
        if (shape.bulk_stores && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        return false;
    };
    // This warp is done with the stage (its values have been used, so its reads have completed).  The last
    // warp of the team to say so refills the stage with the rows that come `stages` stages later.
    auto release_stage = [&]() {
        __syncwarp();
        if (lane == 0) {
            bool last = true;
            if (shape.team_warps > 1) {
                uint32_t before;
                asm volatile("atom.relaxed.cta.shared::cta.add.u32 %0, [%1], 1;"
                             : "=r"(before) : "r"(smem_addr(&done[stage])) : "memory");
                last = before == (uint32_t)shape.team_warps - 1u;
                if (last) done[stage] = 0;  // seen by the stage's next readers through the barrier the refill completes
            }
            if (last && q + (uint32_t)shape.stages < total) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // reads before the unit's writes
                issue(stage, down_step, fill_local, fill_chunk, true, true, true);
            }
        }
        if (++fill_chunk == chunks_per_tile) fill_chunk = 0, ++fill_local;
        if (++stage == shape.stages) stage = 0, phase ^= 1u;
        ++q;
    };
    for (int local = 0; local < my_tiles; ++local) {
        // ---- a new tile: this lane's columns, the masks of their block, an empty sum
        const int tile = tile_of(local, down_step);
        const int64_t c = (int64_t)tile * team_cols + member * WARP_COLS + lane * VEC;
        T* dst = xg + c;
        const int64_t left = prm.d - c;
        const int live_n = left >= VEC ? VEC : (left > 0 ? (int)left : 0);
        uint64_t up = 0, down = 0, keep = 0;  // a lane past the end of the row adds nothing and stores nothing
        float inv = 0.0f;
        int j = 0, j_next = 0, cut = VEC;
        if (live_n > 0) {
            j = block_of(c, prm);
            j_next = j + 1 < n ? j + 1 : j;
            const int64_t in_block = (int64_t)(j + 1) * prm.block_cols - prm.col_offset - c;
            cut = in_block >= VEC ? VEC : (int)in_block;
            up = s_up[j], down = s_down[j], inv = s_inv[j];
            keep = ~down & valid;
        }
        const bool regular = live_n == 0 || (live_n == VEC && cut == VEC);
        // the whole warp inside one block and inside the row: every lane's masks are the same words
        const bool warp_whole = __all_sync(0xFFFFFFFFu, live_n == VEC && cut == VEC) &&
                                __all_sync(0xFFFFFFFFu, j == __shfl_sync(0xFFFFFFFFu, j, 0));
        Float2 sum[VEC / 2];
#pragma unroll
        for (int m = 0; m < VEC / 2; ++m) sum[m] = 0ull;  // (+0, +0)
        Float2 target_sum[VEC / 2];  // tracked: the sum of the targets, two columns at a time
        if (DIAG) {
#pragma unroll
            for (int m = 0; m < VEC / 2; ++m) target_sum[m] = 0ull;
        }

        for (int chunk = 0; chunk < pass_chunks; ++chunk) {
            if (!await_stage()) return;
            const unsigned char* src = my_ring + (size_t)stage * stage_bytes;
#pragma unroll
            for (int half = 0; half < ROWS / 2; ++half) {
                const int k = ROWS * chunk + 2 * half;  // the pair's first worker
                if (ROWS == 4 && k >= n) break;         // the last stage of a tile may hold one pair only
                uint4 raw_x[2], raw_b[2];
                raw_x[0] = *reinterpret_cast<const uint4*>(src + (2 * half) * row_bytes);
                raw_x[1] = *reinterpret_cast<const uint4*>(src + (2 * half + 1) * row_bytes);
                raw_b[0] = *reinterpret_cast<const uint4*>(src + array_bytes + (2 * half) * row_bytes);
                raw_b[1] = *reinterpret_cast<const uint4*>(src + array_bytes + (2 * half + 1) * row_bytes);
                Float2 v[2][VEC / 2];
                local_sgd_pair_packed<T, VEC, DIAG, GRAD>(raw_x, raw_b, v, c, k, prm, scalars, t_lo, t_hi, target_sum);
                if (regular) {
                    const uint32_t arrived = (uint32_t)(up >> k), kept = (uint32_t)(keep >> k) & 3u;
                    // RS: the running sum over the workers whose copy arrived, in worker order
#pragma unroll
                    for (int m = 0; m < VEC / 2; ++m) add2_if(sum[m], v[0][m], arrived & 1u);
#pragma unroll
                    for (int m = 0; m < VEC / 2; ++m) add2_if(sum[m], v[1][m], arrived & 2u);
                    // AG, the workers whose return message is lost: they keep v, which can go out now
                    if (kept) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            if (!((kept >> h) & 1u)) continue;
                            if (GRAD) {  // v holds the update: the worker keeps x + its own
                                Float2 x2[VEC / 2];
                                unpack_pairs<T, VEC>(raw_x[h], x2);
#pragma unroll
                                for (int m = 0; m < VEC / 2; ++m) v[h][m] = add2(x2[m], v[h][m]);
                            }
                            const uint4 packed_v = pack_pairs<T, VEC>(v[h]);
                            __stcs(reinterpret_cast<uint4*>(dst + (int64_t)(k + h) * prm.pitch), packed_v);
                        }
                    }
                } else {
                    float sum_copy[VEC], v_copy[2][VEC];
#pragma unroll
                    for (int m = 0; m < VEC / 2; ++m) {
                        unpack2(sum[m], sum_copy[2 * m], sum_copy[2 * m + 1]);
                        unpack2(v[0][m], v_copy[0][2 * m], v_copy[0][2 * m + 1]);
                        unpack2(v[1][m], v_copy[1][2 * m], v_copy[1][2 * m + 1]);
                    }
                    if (GRAD) {
                        float own_copy[2][VEC];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            RowVec<T, VEC>::unpack(raw_x[h], own_copy[h]);
#pragma unroll
                            for (int e = 0; e < VEC; ++e) own_copy[h][e] += v_copy[h][e];
                        }
                        irregular_pair<T, VEC>(sum_copy, v_copy, own_copy, k, j, j_next, cut, live_n, valid, s_up, s_down,
                                               dst, prm.pitch);
                    } else {
                        irregular_pair<T, VEC>(sum_copy, v_copy, v_copy, k, j, j_next, cut, live_n, valid, s_up, s_down,
                                               dst, prm.pitch);
                    }
#pragma unroll
                    for (int m = 0; m < VEC / 2; ++m) sum[m] = pack2(sum_copy[2 * m], sum_copy[2 * m + 1]);
                }
            }
            release_stage();
        }

        if (GRAD) {
            // ---- AG of gradient averaging: the average UPDATE of the lane's columns, then the rows of x once
            // more: worker k takes x_k + that average where the return message arrived.
            Float2 avg[VEC / 2];
            if (regular) {
                const Float2 inv2 = pack2(inv, inv);
#pragma unroll
                for (int m = 0; m < VEC / 2; ++m) avg[m] = mul2(sum[m], inv2);
            } else {
                const float inv_next = s_inv[j_next];
#pragma unroll
                for (int m = 0; m < VEC / 2; ++m) {
                    float lo, hi;
                    unpack2(sum[m], lo, hi);
                    avg[m] = pack2(lo * (2 * m >= cut ? inv_next : inv), hi * (2 * m + 1 >= cut ? inv_next : inv));
                }
            }
            for (int chunk = 0; chunk < pass_chunks; ++chunk) {
                if (!await_stage()) return;
                const unsigned char* src = my_ring + (size_t)stage * stage_bytes;
#pragma unroll
                for (int r = 0; r < ROWS; ++r) {
                    const int k = ROWS * (pass_chunks - 1 - chunk) + r;  // the rows come back last chunk first
                    if (k >= n) break;
                    if (regular) {
                        if (!((down >> k) & 1u)) continue;
                        Float2 x2[VEC / 2];
                        unpack_pairs<T, VEC>(*reinterpret_cast<const uint4*>(src + r * row_bytes), x2);
#pragma unroll
                        for (int m = 0; m < VEC / 2; ++m) x2[m] = add2(x2[m], avg[m]);
                        __stcs(reinterpret_cast<uint4*>(dst + (int64_t)k * prm.pitch), pack_pairs<T, VEC>(x2));
                    } else {
                        float avg_copy[VEC];
#pragma unroll
                        for (int m = 0; m < VEC / 2; ++m) unpack2(avg[m], avg_copy[2 * m], avg_copy[2 * m + 1]);
                        irregular_update_row<T, VEC>(*reinterpret_cast<const uint4*>(src + r * row_bytes), avg_copy, k, j,
                                                     j_next, cut, live_n, s_down, dst + (int64_t)k * prm.pitch);
                    }
                }
                release_stage();
            }
            continue;
        }
        // ---- AG, the receivers: one average, rounded and packed once, to every row whose down bit is set
        if (regular) {
            const Float2 inv2 = pack2(inv, inv);
            Float2 avg[VEC / 2];
#pragma unroll
            for (int m = 0; m < VEC / 2; ++m) avg[m] = mul2(sum[m], inv2);
            const uint4 packed = pack_pairs<T, VEC>(avg);
            if (warp_whole && shape.bulk_stores) {
                // The warp's 512 bytes of averages go to one of its two slots in shared memory, and one thread
                // sends the slot to every receiver's row with an asynchronous bulk copy: the rows are written by
                // the copy unit, 512 bytes at a time, while the warp is already at its next tile.  A slot is
                // reused two tiles later, once the copies that read it have done so.
                unsigned char* slot = out_slots + (local & 1) * kPieceBytes;
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                __syncwarp();
                *reinterpret_cast<uint4*>(slot + lane * 16) = packed;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // visible to the copy unit
                __syncwarp();
                if (lane == 0) {
                    const uint32_t src = smem_addr(slot);
                    uint64_t rest = down;
                    const T* row = dst;  // lane 0 holds the warp's first column
#pragma unroll 4
                    for (int i = 0; i < n; ++i, row += prm.pitch, rest >>= 1)
                        if (rest & 1u)
                            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(row), "r"(src),
                                         "n"(kPieceBytes)
                                         : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            } else {
                uint64_t rest = down;
                T* row = dst;
#pragma unroll 4
                for (int i = 0; i < n; ++i, row += prm.pitch, rest >>= 1)
                    if (rest & 1u) __stcs(reinterpret_cast<uint4*>(row), packed);
            }
            if (DIAG && live_n == VEC) {
                // the keepers' rows as this lane stored them a moment ago, against what the receivers hold
                float pivot[VEC], targets[VEC], dev_sum[VEC], dev_sq[VEC], dd = 0.0f, qq = 0.0f;
                if (down != 0) RowVec<T, VEC>::unpack(packed, pivot);
                else RowVec<T, VEC>::unpack(__ldcg(reinterpret_cast<const uint4*>(dst)), pivot);
#pragma unroll
                for (int e = 0; e < VEC; ++e) dev_sum[e] = dev_sq[e] = 0.0f;
                for (uint64_t rest = keep; rest != 0; rest &= rest - 1) {
                    const int i = __ffsll((long long)rest) - 1;
                    float kept_v[VEC];
                    RowVec<T, VEC>::unpack(__ldcg(reinterpret_cast<const uint4*>(dst + (int64_t)i * prm.pitch)), kept_v);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) {
                        const float dev = kept_v[e] - pivot[e];
                        dev_sum[e] += dev;
                        dev_sq[e] = fmaf(dev, dev, dev_sq[e]);
                    }
                }
#pragma unroll
                for (int m = 0; m < VEC / 2; ++m) unpack2(target_sum[m], targets[2 * m], targets[2 * m + 1]);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    close_tracked_column(targets[e], pivot[e], dev_sum[e], dev_sq[e], prm.inv_n, dd, qq);
                tracker.dist2 += (double)dd;
                tracker.cons += (double)qq;
            }
        } else {
            float sum_copy[VEC], dd = 0.0f, qq = 0.0f;
#pragma unroll
            for (int m = 0; m < VEC / 2; ++m) unpack2(sum[m], sum_copy[2 * m], sum_copy[2 * m + 1]);
            float targets[VEC];  // (of the columns that exist: the others hold whatever the padding held)
#pragma unroll
            for (int m = 0; m < VEC / 2; ++m) {
                if (DIAG) unpack2(target_sum[m], targets[2 * m], targets[2 * m + 1]);
                else targets[2 * m] = targets[2 * m + 1] = 0.0f;
            }
            irregular_receivers<T, VEC, DIAG>(sum_copy, n, j, j_next, cut, live_n, s_down, s_inv, dst, prm.pitch,
                                              targets, prm.inv_n, &dd, &qq);
            if (DIAG) {
                tracker.dist2 += (double)dd;
                tracker.cons += (double)qq;
            }
        }
    }
    if (step + 1 < shape.steps) {
        // ---- between two steps.  The next step reads, through the TMA unit, what this team's warps have just
        // stored: every lane sees its own stores done (bulk copies first, then a fence over global memory), the
        // team meets on its barrier (bounded like every other wait), and the thread that starts the next step's
        // copies orders them behind all that with a proxy fence.  The ring has run empty by itself (nothing
        // is refilled past the end of a step), so the team's pipeline restarts: a few microseconds per step and
        // team, at a different time for every team, instead of a launch boundary for the whole GPU.
        if (shape.bulk_stores && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        __threadfence();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(step_bar));
        if (!__all_sync(0xFFFFFFFFu, stream_wait(smem_addr(step_bar), (uint32_t)step & 1u, shape.wait_limit_ns))) {
            report_timeout(prm, 3);
            return;
        }
        if (member == 0 && lane == 0) asm volatile("fence.proxy.async;" ::: "memory");
        first_fills(stage, walks_down(step + 1), true, true, true);
    }
    }
    if (DIAG) tracker.flush(track_pair, track_arrivals, (int)(blockDim.x >> 5), prm.trace);
    // the bulk copies issued by this thread still read this CTA's shared memory: see them through
    if (shape.bulk_stores && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Describes one [n][pitch] array to the TMA unit in 8-byte units (so that a box may span 2 KB of a row whatever
// the replica type), with boxes of `rows` rows x team_warps x 512 bytes.  Row starts, the pitch and the part of a
// row that may be read are multiples of 128 bytes.
bool encode_row_boxes(CUtensorMap* map, const void* base, size_t elem, const FusedParams& prm, int team_warps, int rows)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)prm.cols_in_row * elem / 8, (cuuint64_t)prm.n};
    const cuuint64_t strides[1] = {(cuuint64_t)prm.pitch * elem};  // bytes between rows
    const cuuint32_t box[2] = {(cuuint32_t)team_warps * (kPieceBytes / 8), (cuuint32_t)rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, int VEC, int MAXW, int ROWS, bool DIAG = false, bool GRAD = false>
cudaError_t launch_stream_as(const FusedParams& prm, const FusedTuning& tune, int warps, int team_warps, int steps,
                             int sm_count, cudaStream_t stream)
{
    auto kernel = rps_fused_stream_kernel<T, VEC, MAXW, ROWS, DIAG, GRAD>;
    static LaunchState state;
    size_t smem_limit = 0;
    cudaError_t err = smem_limit_of_device(state, &smem_limit);
    if (err != cudaSuccess) return err;
    constexpr int warp_cols = 32 * VEC;
    StreamShape shape{};
    shape.team_warps = team_warps;
    shape.teams = warps / team_warps;
    shape.stages = tune.stages > 0 ? tune.stages : kStreamDefaultStages;
    if (shape.stages > kStreamMaxStages) shape.stages = kStreamMaxStages;
    shape.bulk_stores = !GRAD && (tune.store_mode != 0 ? tune.store_mode : kStreamDefaultStoreMode) == 2;
    // the rings, then (bulk stores) two 512-byte output slots per warp
    auto ring_bytes = [&] {
        return (size_t)shape.teams * team_warps * (shape.stages * (2 * ROWS * kPieceBytes) + (shape.bulk_stores ? 2 * kPieceBytes : 0));
    };
    while (shape.stages > 2 && kStreamHeaderBytes + ring_bytes() > smem_limit) --shape.stages;
    while (shape.teams > 1 && kStreamHeaderBytes + ring_bytes() > smem_limit) --shape.teams;
    if (kStreamHeaderBytes + ring_bytes() > smem_limit) return cudaErrorInvalidConfiguration;
    shape.out_offset = (uint32_t)((size_t)shape.teams * team_warps * shape.stages * (2 * ROWS * kPieceBytes));
    const int64_t team_cols = (int64_t)team_warps * warp_cols;
    shape.tiles = (int32_t)((prm.d + team_cols - 1) / team_cols);
    shape.wait_limit_ns = tune.wait_limit_ms > 0 ? (uint64_t)tune.wait_limit_ms * 1000000ull : kDefaultWaitLimitNs;
    shape.withhold_copies = tune.withhold_copies;
    shape.steps = steps;
    shape.alternate = tune.traversal == 0;
    // early copies of the targets: built and bit-identical, but worth nothing here (cfg5: 1.036 ms per step with
    // them, 1.024 without, three alternating pairs on one box); the staged kernel gains 0.7 % on the smallest model
    shape.early_targets = tune.early_targets == 2;
    const uint32_t smem_bytes = kStreamHeaderBytes + (uint32_t)ring_bytes();
    if ((err = grant_smem(state, kernel, smem_bytes)) != cudaSuccess) return err;
    alignas(64) CUtensorMap map_x, map_b;
    // boxes of ROWS workers x one team's row piece; loads may read up to the pitch (padding arrives and is ignored)
    if (!encode_row_boxes(&map_x, prm.x, sizeof(T), prm, team_warps, ROWS) ||
        !encode_row_boxes(&map_b, prm.b, sizeof(T), prm, team_warps, ROWS))
        return cudaErrorInvalidValue;
    // Persistent CTAs, one per SM; the teams take the tiles in fixed turns, so the step lasts as long as
    // the team with the most tiles.  A few SMs fewer can even that out: take the grid, from the SM count
    // down to 7/8 of it, that loses the least to the last, partly filled round of turns.
    int64_t grid = sm_count;
    if (grid * shape.teams > shape.tiles) grid = (shape.tiles + shape.teams - 1) / shape.teams;
    if (grid < 1) grid = 1;
    if (grid == sm_count) {
        double best = 0.0;
        for (int64_t cand = sm_count; cand >= sm_count - sm_count / 8 && cand >= 1; --cand) {
            const int64_t teams_total = cand * shape.teams;
            const int64_t rounds = (shape.tiles + teams_total - 1) / teams_total;
            const double busy = (double)shape.tiles / (double)(rounds * shape.teams * sm_count);  // of all SMs' time
            if (busy > best + 1e-9) best = busy, grid = cand;
        }
    }
    cudaLaunchConfig_t config = {};
    config.gridDim = dim3((unsigned)grid);
    config.blockDim = dim3((unsigned)(shape.teams * team_warps) * 32);
    config.dynamicSmemBytes = smem_bytes;
    config.stream = stream;
    cudaLaunchAttribute attribute[1];
    attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attribute[0].val.programmaticStreamSerializationAllowed = 1;
    config.attrs = attribute;
    config.numAttrs = tune.launch_overlap == 1 ? 0 : 1;
    return cudaLaunchKernelEx(&config, kernel, prm, shape, map_x, map_b);
}

template <typename T, int VEC, int ROWS>
cudaError_t launch_stream_for_warps(const FusedParams& prm, const FusedTuning& tune, int steps, int sm_count,
                                    cudaStream_t stream)
{
    // the register file is shared out by launch bound: 32 warps of 64 registers, 24 of 80, 20 of 96, 16 of 128
    // defaults from sweeps on B200 (n = 64, bf16): 5 teams of 4 warps (whose rings of 16 KB stages are two stages deep:
    // a third does not fit in shared memory, and made no difference where it did); 16 warps leave issue slots idle,
    // 24 and more lose more to the memory system than they gain
    int warps = tune.consumer_warps > 0 ? tune.consumer_warps : 20;
    if (warps > kStreamMaxWarps) warps = kStreamMaxWarps;
    int team_warps = tune.team_warps == 0 || tune.team_warps >= 4 ? 4 : (tune.team_warps >= 2 ? 2 : 1);
    while (team_warps > warps) team_warps /= 2;
    warps -= warps % team_warps;  // whole teams
    if (warps <= 16) return launch_stream_as<T, VEC, 16, ROWS>(prm, tune, warps, team_warps, steps, sm_count, stream);
    if (warps <= 20) return launch_stream_as<T, VEC, 20, ROWS>(prm, tune, warps, team_warps, steps, sm_count, stream);
    if (warps <= 24) return launch_stream_as<T, VEC, 24, ROWS>(prm, tune, warps, team_warps, steps, sm_count, stream);
    return launch_stream_as<T, VEC, 32, ROWS>(prm, tune, warps, team_warps, steps, sm_count, stream);
}

// Tracked steps: stages of two worker pairs, 20 warps like the plain step (the walk carries only the sum of the
// targets on top of it; bf16, n = 64: 1.11 ms per launch against 1.16 with 16 warps).
template <typename T, int VEC>
cudaError_t launch_stream_tracked(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    int warps = tune.consumer_warps > 0 ? tune.consumer_warps : 20;
    if (warps > 20) warps = 20;
    int team_warps = tune.team_warps == 0 || tune.team_warps >= 4 ? 4 : (tune.team_warps >= 2 ? 2 : 1);
    while (team_warps > warps) team_warps /= 2;
    warps -= warps % team_warps;
    if (warps <= 16) return launch_stream_as<T, VEC, 16, 4, true>(prm, tune, warps, team_warps, 1, sm_count, stream);
    return launch_stream_as<T, VEC, 20, 4, true>(prm, tune, warps, team_warps, 1, sm_count, stream);
}

// Gradient averaging: stages of two worker pairs, 16 or 20 warps.
template <typename T, int VEC>
cudaError_t launch_stream_gradients(const FusedParams& prm, const FusedTuning& tune, int steps, int sm_count,
                                    cudaStream_t stream)
{
    int warps = tune.consumer_warps > 0 ? tune.consumer_warps : 20;
    if (warps > 20) warps = 20;
    int team_warps = tune.team_warps == 0 || tune.team_warps >= 4 ? 4 : (tune.team_warps >= 2 ? 2 : 1);
    while (team_warps > warps) team_warps /= 2;
    warps -= warps % team_warps;
    if (warps <= 16)
        return launch_stream_as<T, VEC, 16, 4, false, true>(prm, tune, warps, team_warps, steps, sm_count, stream);
    return launch_stream_as<T, VEC, 20, 4, false, true>(prm, tune, warps, team_warps, steps, sm_count, stream);
}

}  // namespace

bool stream_kernel_covers(const FusedParams& prm, bool bf16)
{
    // at least one worker pair, blocks at least as wide as a lane's slice (a slice then meets at most two
    // blocks); TMA coordinates are 32-bit.  Tracked steps are model averaging.
    return prm.n >= 2 && !(prm.average_gradients && prm.trace != nullptr) && prm.block_cols >= (bf16 ? 8 : 4) &&
           prm.pitch < ((int64_t)1 << 31);
}

cudaError_t launch_fused_stream(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                                cudaStream_t stream, int steps)
{
    if (!stream_kernel_covers(prm, bf16) || steps < 1) return cudaErrorInvalidConfiguration;
    if (prm.trace != nullptr) {
        if (steps != 1) return cudaErrorInvalidConfiguration;  // tracked steps run one per launch
        return bf16 ? launch_stream_tracked<__nv_bfloat16, 8>(prm, tune, sm_count, stream)
                    : launch_stream_tracked<float, 4>(prm, tune, sm_count, stream);
    }
    if (prm.average_gradients)
        return bf16 ? launch_stream_gradients<__nv_bfloat16, 8>(prm, tune, steps, sm_count, stream)
                    : launch_stream_gradients<float, 4>(prm, tune, steps, sm_count, stream);
    // rows per stage: two worker pairs, unless one pair is asked for (workers_per_lane = 2)
    const bool one_pair = tune.workers_per_lane == 2 || prm.n <= 2;
    if (bf16)
        return one_pair ? launch_stream_for_warps<__nv_bfloat16, 8, 2>(prm, tune, steps, sm_count, stream)
                        : launch_stream_for_warps<__nv_bfloat16, 8, 4>(prm, tune, steps, sm_count, stream);
    return one_pair ? launch_stream_for_warps<float, 4, 2>(prm, tune, steps, sm_count, stream)
                    : launch_stream_for_warps<float, 4, 4>(prm, tune, steps, sm_count, stream);
}

}  // namespace rps
