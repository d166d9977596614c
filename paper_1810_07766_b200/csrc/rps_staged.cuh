// Fused RPS step, staged form (sm_100a): the row slices of x and b travel from
// HBM into a shared-memory ring with TMA tensor copies (cp.async.bulk.tensor.2d)
// that complete on mbarriers, issued by one producer thread per CTA; the other
// warps only compute.  The bytes in flight are set by the ring (stages x tile),
// not by how many registers the compute warps can spare, so the copy engine
// keeps HBM busy while the warps run Philox and Box-Muller.
//
// One tile = tile_cols consecutive columns of all n workers of both arrays.
// Two ways of filling a stage.  (a) Boxes: x and b are described to the TMA unit
// as 2-D tensors [n][pitch]; one copy brings a box of all n rows x box_cols
// columns (box_cols <= 256 elements), so a stage is filled by a handful of
// instructions whatever n is and the unit itself walks the rows; columns past
// the row pitch arrive as zeros.  (b) Rows: one 1-D bulk copy per row and array,
// issued by the 32 lanes of the producer warp; fewer, longer copies when n is
// small.
// Consumer warp w of a CTA owns columns [w * WARP_COLS, (w+1) * WARP_COLS) of
// the tile and maps its lanes to (worker group, 16-byte column slice) exactly as
// the direct kernel does; the arithmetic is the same code (rps_device.cuh).
// Results leave either straight from registers with 16-byte streaming stores,
// or, where a lane group would write less than a full line per row (many
// workers), through a double-buffered tile in shared memory and TMA tensor
// stores of whole boxes (clipped at column d by the tensor map).
//
// Every wait on an mbarrier is bounded (2 s of %globaltimer by default); a wait
// that gives up records a code in *prm.error and the warp stops working.
//
// This header holds the kernel template and its host-side planning; the translation units that
// include it each build one group of instantiations (plain, gradient averaging, tracked).
#pragma once

#include <cuda.h>

#include "rps_kernels.h"

#include "rps_device.cuh"
#include "rps_tma.cuh"

namespace rps {

namespace {

constexpr int kMaxStages = 8;
constexpr int kMaxConsumerWarps = 16;
constexpr int kMaxBoxCols = 256;  // a TMA box is at most 256 elements wide
constexpr uint32_t kSmemHeaderBytes = 128 + 2 * kMaxWorkers * 8 + kMaxWorkers * 4 + 128;  // barriers, mask copy, flags
constexpr uint32_t kAbortFlagOffset = kSmemHeaderBytes - 128;
constexpr int kOutBuffers = 2;
constexpr int kDefaultL2Policy = 1;
constexpr int kDefaultLaunchOverlap = 2;
constexpr int kDefaultEarlyTargets = 2;
static_assert(kSmemHeaderBytes % 128 == 0, "tile data must start on a 128-byte boundary");

struct StagedShape {
    int64_t tiles;
    int32_t stages;
    int32_t consumer_warps;
    int32_t tile_cols;
    int32_t use_boxes;     // 1: 2-D tensor copies of whole boxes; 0: one 1-D bulk copy per row
    int32_t box_cols;      // columns per TMA box; a tile is boxes_per_tile boxes side by side
    int32_t boxes_per_tile;
    uint32_t row_bytes;    // bytes of one row of one box
    uint32_t box_tx_bytes; // bytes one box copy delivers: n rows
    uint32_t box_bytes;    // the same rounded up to 128: boxes start on 128-byte boundaries
    uint32_t array_bytes;  // all boxes of one array
    uint32_t stage_bytes;  // both arrays, rounded up to 128
    // how results leave: 1 straight from registers; 2 through a double-buffered output tile in shared
    // memory and TMA tensor stores issued by a compute thread; 3 written back in place over the x half of
    // the stage and stored from there by a dedicated store warp, which then frees the stage
    int32_t store_mode;
    int32_t out_box_cols;
    int32_t out_boxes_per_tile;
    uint32_t out_row_bytes;   // out_box_cols elements
    uint32_t out_box_bytes;   // n rows, rounded up to 128
    uint32_t out_bytes;       // one output buffer: all boxes of a tile
    uint32_t out_offset;      // of the first output buffer, from the start of the ring
    uint64_t wait_limit_ns;   // how long a wait on an mbarrier may last before the warp gives up
    int32_t withhold_copies;  // test aid: the producer issues nothing, so that the waits run out
    // 1: the tiles are taken from the last to the first.  Odd steps run this way, so that a step starts
    // on the columns the step before it touched last, which are still in L2 (and still dirty there).
    int32_t descending;
    int32_t evict_first_targets;  // 1: b is loaded with the L2 evict-first hint
    // 1: the producer issues the copies of b for its first `stages` tiles BEFORE it waits for the kernel ahead of
    // it in the stream (programmatic launch): the targets are not written by a step, so they can arrive while
    // that kernel drains.  Only the copies of x wait.
    int32_t early_targets;

    __device__ __forceinline__ int64_t tile_of_turn(int64_t turn) const { return descending ? tiles - 1 - turn : turn; }
};

// Eight workers per lane need more registers than 17 warps leave: that shape runs with at most 12 consumer
// warps, or 20 in the narrow bf16 form (8-byte slices: half the raw registers, half the shared memory per warp).
constexpr int max_consumer_warps(int wpt, int vec, int elem)
{
    return wpt >= 8 ? ((elem == 2 && vec == 4) ? 20 : 12) : kMaxConsumerWarps;
}

template <typename T, int VEC, int WPT, int G, bool GRAD, bool DIAG>
__global__ void __launch_bounds__((max_consumer_warps(WPT, VEC, (int)sizeof(T)) + 2) * 32, 1)
    rps_fused_staged_kernel(const FusedParams prm, const StagedShape shape, const __grid_constant__ CUtensorMap map_x,
                            const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_out)
{
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);           // [kMaxStages] data has landed
    uint64_t* empty = reinterpret_cast<uint64_t*>(smem + 64);     // [kMaxStages] consumers are done
    uint64_t* s_up = reinterpret_cast<uint64_t*>(smem + 128);     // copy of this step's masks
    uint64_t* s_down = s_up + kMaxWorkers;
    float* s_inv = reinterpret_cast<float*>(s_down + kMaxWorkers);
    unsigned char* ring = smem + kSmemHeaderBytes;

    const int n = prm.n;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int consumer_warps = shape.consumer_warps;

    if (threadIdx.x == 0) {
        for (int s = 0; s < shape.stages; ++s) {
            mbar_init(smem_addr(&full[s]), 1);
            // a stage is handed back by every compute warp, or (in-place results) by the store warp alone
            mbar_init(smem_addr(&empty[s]), shape.store_mode == 3 ? 1u : (uint32_t)consumer_warps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    constexpr uint32_t elem = (uint32_t)sizeof(T);
    // Launched with programmatic stream serialization this CTA may have been placed while the kernel before
    // it in the stream was still draining.  Let the kernel after this one do the same, then wait for the one
    // before to complete (its writes visible) before reading anything it may have written: the masks here, x
    // in the producer.  Both are no-ops in a plain launch.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Copies of one tile into its stage, by the producer warp: the targets, the replicas, or both; `expect`
    // announces the bytes of BOTH to the stage's barrier (once per tile, before its first copy).
    auto copy_tile = [&](int stage, int64_t tile, bool with_x, bool with_b, bool expect) {
        const unsigned char* x_bytes = static_cast<const unsigned char*>(prm.x);
        const unsigned char* b_bytes = static_cast<const unsigned char*>(prm.b);
        const uint64_t targets_policy = l2_evict_first_policy();
        const int64_t c0 = tile * shape.tile_cols;
        const uint32_t bar = smem_addr(&full[stage]);
        const uint32_t dst = smem_addr(ring) + (uint32_t)stage * shape.stage_bytes;
        if (shape.use_boxes) {
            // one thread, a few copies: the TMA unit walks the n rows of each box itself.  Boxes are
            // always delivered whole (zeros past the pitch), so the byte count is fixed.
            if (lane == 0) {
                if (expect) mbar_arrive_expect_tx(bar, 2u * (uint32_t)shape.boxes_per_tile * shape.box_tx_bytes);
                for (int k = 0; k < shape.boxes_per_tile; ++k) {
                    const int32_t col = (int32_t)c0 + k * shape.box_cols;
                    if (with_x) tma_load_box(dst + (uint32_t)k * shape.box_bytes, &map_x, col, 0, bar);
                    if (with_b) {
                        if (shape.evict_first_targets)
                            tma_load_box(dst + shape.array_bytes + (uint32_t)k * shape.box_bytes, &map_b, col, 0, bar,
                                         targets_policy);
                        else
                            tma_load_box(dst + shape.array_bytes + (uint32_t)k * shape.box_bytes, &map_b, col, 0, bar);
                    }
                }
            }
        } else {
            // one bulk copy per row and array, spread over the lanes; the last tile stops at the pitch
            const int64_t cols_left = prm.cols_in_row - c0;
            const uint32_t cols = (uint32_t)(cols_left < shape.tile_cols ? cols_left : shape.tile_cols);
            const uint32_t bytes = cols * elem;
            if (expect && lane == 0) mbar_arrive_expect_tx(bar, 2u * (uint32_t)n * bytes);
            __syncwarp();
            for (int i = lane; i < n; i += 32) {
                const int64_t at = ((int64_t)i * prm.pitch + c0) * elem;
                if (with_x) bulk_load_row(dst + (uint32_t)i * shape.row_bytes, x_bytes + at, bytes, bar);
                if (with_b) {
                    if (shape.evict_first_targets)
                        bulk_load_row(dst + shape.array_bytes + (uint32_t)i * shape.row_bytes, b_bytes + at, bytes, bar,
                                      targets_policy);
                    else
                        bulk_load_row(dst + shape.array_bytes + (uint32_t)i * shape.row_bytes, b_bytes + at, bytes, bar);
                }
            }
        }
    };
    // the targets of the producer's first tiles, ahead of the wait (see StagedShape::early_targets)
    int early_tiles = 0;
    if (shape.early_targets && !shape.withhold_copies) {
        __syncthreads();  // the barriers are initialised
        if (warp == consumer_warps) {
            if (shape.use_boxes && lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
            for (int64_t turn = blockIdx.x; turn < shape.tiles && early_tiles < shape.stages; turn += gridDim.x) {
                copy_tile(early_tiles, shape.tile_of_turn(turn), false, true, true);
                ++early_tiles;
            }
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kAbortFlagOffset);
    if (threadIdx.x == 0) *abort_flag = 0;
    // tracked steps: the CTA's pair of sums and the count of warps that have added theirs
    int* track_arrivals = reinterpret_cast<int*>(smem + kAbortFlagOffset + 8);
    double* track_pair = reinterpret_cast<double*>(smem + kAbortFlagOffset + 16);
    if (DIAG && threadIdx.x == 0) {
        track_pair[0] = 0.0;
        track_pair[1] = 0.0;
        *track_arrivals = 0;
    }
    for (int j = threadIdx.x; j < kMaxWorkers; j += blockDim.x) {
        const bool used = j < n;
        s_up[j] = used ? prm.masks->up[j] : 0;
        s_down[j] = used ? prm.masks->down[j] : 0;
        s_inv[j] = used ? prm.masks->inv_cnt[j] : 0.0f;
    }
    __syncthreads();
    // no CTA-wide barrier below this line: the producer warp runs ahead and leaves first

    if (warp == consumer_warps) {
        // ---------------- producer warp: keeps the ring full
        if (shape.withhold_copies) return;
        if (shape.use_boxes && lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        }
        int stage = 0;
        uint32_t phase = 0;
        int64_t issued = 0;
        bool ok = true;
        for (int64_t turn = blockIdx.x; turn < shape.tiles; turn += gridDim.x) {
            const int64_t tile = shape.tile_of_turn(turn);
            // a fresh barrier counts as "previous phase complete", so the first lap does not wait
            if (!mbar_wait(smem_addr(&empty[stage]), phase ^ 1u, shape.wait_limit_ns)) {
                ok = false;
                break;
            }
            // the targets of the first tiles are on their way already, and their bytes announced
            const bool early = issued < early_tiles;
            copy_tile(stage, tile, true, !early, !early);
            ++issued;
            if (++stage == shape.stages) {
                stage = 0;
                phase ^= 1u;
            }
        }
        if (!ok) {
            report_timeout(prm, 1);
            // copies already issued still target this CTA's shared memory: see them land before leaving
            const int64_t back = issued < shape.stages ? issued : shape.stages;
            for (int64_t k = 0; k < back; ++k) {
                if (--stage < 0) {
                    stage = shape.stages - 1;
                    phase ^= 1u;
                }
                if (!mbar_wait(smem_addr(&full[stage]), phase, shape.wait_limit_ns)) break;
            }
        }
        return;
    }

    const uint32_t consumer_threads = (uint32_t)consumer_warps * 32u;
    if (warp == consumer_warps + 1) {
        // ---------------- store warp (in-place results only): when every compute warp has put its results
        // of a tile back into the stage, send the x half of the stage to global memory and free the stage
        if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out) : "memory");
        int stage = 0;
        bool dead = false;
        for (int64_t turn = blockIdx.x; turn < shape.tiles; turn += gridDim.x) {
            const int64_t tile = shape.tile_of_turn(turn);
            asm volatile("bar.sync %0, %1;" ::"r"(1 + stage), "r"(consumer_threads + 32u) : "memory");
            if (*abort_flag) dead = true;
            if (lane == 0 && !dead) {
                const int32_t c0 = (int32_t)(tile * shape.tile_cols);
                const uint32_t src = smem_addr(ring) + (uint32_t)stage * shape.stage_bytes;
                for (int k = 0; k < shape.boxes_per_tile; ++k) {
                    const int32_t col = c0 + k * shape.box_cols;
                    if (col < prm.d) tma_store_box(&map_out, col, 0, src + (uint32_t)k * shape.box_bytes);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the unit has read the stage
                mbar_arrive(smem_addr(&empty[stage]));
            }
            if (++stage == shape.stages) stage = 0;
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        return;
    }

    // ---------------- consumers
    T* __restrict__ xg = static_cast<T*>(prm.x);
    const MaskView masks{s_up, s_down, s_inv};
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;
    // where this lane's slice sits inside a stage: box, then column inside the box
    const int col_in_tile = warp * WARP_COLS + sub * VEC;
    const uint32_t lane_off =
        (uint32_t)(col_in_tile / shape.box_cols) * shape.box_bytes + (uint32_t)(col_in_tile % shape.box_cols) * elem;
    const bool out_tiles = shape.store_mode == 2, in_place = shape.store_mode == 3;
    // the stage is read a second time after the average when updates rather than models are averaged
    const bool hold_stage = in_place || GRAD;
    const uint32_t lane_out_off = out_tiles ? (uint32_t)(col_in_tile / shape.out_box_cols) * shape.out_box_bytes +
                                                  (uint32_t)(col_in_tile % shape.out_box_cols) * elem
                                            : 0u;
    const bool store_leader = threadIdx.x == 0;  // issues the tensor stores of mode 2
    if (out_tiles && store_leader) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out) : "memory");
    int stage = 0, out_slot = 0;
    uint32_t phase = 0;
    // A warp whose wait gave up stops working but keeps meeting the other compute warps at the
    // per-tile barrier below, so that nobody is left waiting for it.
    bool dead = false;
    BlockCursor cursor;
    Tracker<VEC, WPT, G> tracker;
    const uint32_t present = Tracker<VEC, WPT, G>::present_workers(w_first, n);
    for (int64_t turn = blockIdx.x; turn < shape.tiles; turn += gridDim.x) {
        const int64_t tile = shape.tile_of_turn(turn);
        if (!dead && !__all_sync(0xFFFFFFFFu, mbar_wait(smem_addr(&full[stage]), phase, shape.wait_limit_ns))) {
            report_timeout(prm, 2);
            *abort_flag = 1;
            dead = true;
            if (shape.store_mode == 1) return;  // no barrier to keep: leave
        }
        if (!dead) {
            const int64_t c = tile * shape.tile_cols + warp * WARP_COLS + sub * VEC;
            const bool col_live = c < prm.d;
            unsigned char* base = ring + (size_t)stage * shape.stage_bytes + lane_off;

            float v[WPT][VEC];
            {
                using Raw = typename RowVec<T, VEC>::Raw;
                Raw raw_x[WPT], raw_b[WPT];
#pragma unroll
                for (int w = 0; w < WPT; ++w) {
                    // workers past n read the last real row: their values are masked out (their mask bits
                    // are 0) and never stored, so no lane needs a zero-filled stand-in
                    const int row = w_first + w < n ? w_first + w : n - 1;
                    raw_x[w] = *reinterpret_cast<const Raw*>(base + (size_t)row * shape.row_bytes);
                    raw_b[w] = *reinterpret_cast<const Raw*>(base + shape.array_bytes + (size_t)row * shape.row_bytes);
                }
                if (!hold_stage) {
                    // this warp has read everything it needs from the stage: hand it back to the producer
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_addr(&empty[stage]));
                }
                if (DIAG) {
                    float bv[WPT][VEC];
#pragma unroll
                    for (int w = 0; w < WPT; ++w) RowVec<T, VEC>::unpack(raw_b[w], bv[w]);
                    tracker.targets(bv, present);
                }
                local_sgd_raw<T, VEC, WPT, GRAD>(raw_x, raw_b, v, c, w_first, prm);
            }
            const uint32_t live_bits = average_and_select<VEC, WPT, G>(v, c, col_live, w_first, masks, cursor, prm);
            if (GRAD) {
                // v holds the update each worker applies (the average one where it arrived): x_{t+1} = x + update
#pragma unroll
                for (int w = 0; w < WPT; ++w) {
                    const int row = w_first + w < n ? w_first + w : n - 1;
                    float xv[VEC];
                    RowVec<T, VEC>::unpack(
                        *reinterpret_cast<const typename RowVec<T, VEC>::Raw*>(base + (size_t)row * shape.row_bytes), xv);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) v[w][e] += xv[e];
                }
                if (!in_place) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_addr(&empty[stage]));
                }
            }
            if (DIAG) {
#pragma unroll
                for (int w = 0; w < WPT; ++w) as_stored<T, VEC>(v[w]);
                tracker.models(v, present, live_bits, prm.inv_n);
            }
            if (in_place) {
                // every lane overwrites exactly the slices of x it read; columns past d are clipped by
                // the tensor store
#pragma unroll
                for (int w = 0; w < WPT; ++w)
                    if (w_first + w < n)
                        *reinterpret_cast<typename RowVec<T, VEC>::Raw*>(base + (size_t)(w_first + w) * shape.row_bytes) =
                            RowVec<T, VEC>::pack(v[w]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // visible to the TMA unit
            } else if (out_tiles) {
                // results go to this tile's output buffer in box layout; columns past d are written
                // here too and clipped by the tensor store
                unsigned char* out = ring + shape.out_offset + (size_t)out_slot * shape.out_bytes + lane_out_off;
#pragma unroll
                for (int w = 0; w < WPT; ++w)
                    if (w_first + w < n)
                        *reinterpret_cast<typename RowVec<T, VEC>::Raw*>(out + (size_t)(w_first + w) * shape.out_row_bytes) =
                            RowVec<T, VEC>::pack(v[w]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // visible to the TMA unit
            } else {
                T* dst = xg + (int64_t)w_first * prm.pitch + c;  // this lane's slice of its first worker's row
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
        if (in_place) {
            // Tell the store warp.  A warp that gave up still takes part, and waits for the meeting to
            // complete: it no longer waits for data, and must not run ahead of the store warp and be counted
            // twice on one barrier.
            if (dead)
                asm volatile("bar.sync %0, %1;" ::"r"(1 + stage), "r"(consumer_threads + 32u) : "memory");
            else
                asm volatile("bar.arrive %0, %1;" ::"r"(1 + stage), "r"(consumer_threads + 32u) : "memory");
        } else if (out_tiles) {
            // One meeting of the compute warps per tile.  Before it the leader sees the previous tile's
            // stores finish reading their buffer, so after it (a) the other buffer is free for the next
            // tile and (b) every warp's results for this tile are in place.
            if (store_leader && !dead) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            asm volatile("bar.sync 1, %0;" ::"r"(consumer_threads) : "memory");
            if (*abort_flag) dead = true;
            if (store_leader && !dead) {
                const int32_t c0 = (int32_t)(tile * shape.tile_cols);
                const uint32_t src = smem_addr(ring) + shape.out_offset + (uint32_t)out_slot * shape.out_bytes;
                for (int k = 0; k < shape.out_boxes_per_tile; ++k) {
                    const int32_t col = c0 + k * shape.out_box_cols;
                    if (col < prm.d) tma_store_box(&map_out, col, 0, src + (uint32_t)k * shape.out_box_bytes);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            out_slot ^= 1;
        }
        if (++stage == shape.stages) {
            stage = 0;
            phase ^= 1u;
        }
    }
    if (DIAG) tracker.flush(track_pair, track_arrivals, consumer_warps, prm.trace);
    // the stores still read this CTA's shared memory: see them through before the CTA retires
    if (out_tiles && store_leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

struct Plan {
    int32_t threads;
    uint32_t smem_bytes;
    StagedShape shape;
};

// Shapes the tile and the ring for one instantiation with the given number of compute warps; false if
// a ring of 2 stages (plus the output buffers) does not fit in shared memory.
bool shape_for(const FusedParams& prm, const FusedTuning& tune, int vec, int g, size_t elem, size_t smem_limit,
               int warps, int default_store_mode, Plan* out)
{
    const int warp_cols = (32 / g) * vec;
    StagedShape& sh = out->shape;
    sh.consumer_warps = warps;
    sh.tile_cols = warps * warp_cols;
    // the widest box (<= 256 elements) that tiles the tile exactly; warp_cols always does
    int box_cols = warp_cols;
    for (int k = 1; k <= warps; ++k)
        if (warps % k == 0 && k * warp_cols <= kMaxBoxCols) box_cols = k * warp_cols;
    // 2-D boxes when many rows would otherwise mean many small copies, or when asked for
    // Results: 16-byte stores from registers, or TMA tensor stores from shared memory: from a separate
    // double-buffered output tile (2), or in place from the stage by a store warp (3) where shared memory
    // is too scarce for output tiles (8 workers per lane).  In place needs the box layout.
    const int store_mode = tune.store_mode != 0 ? tune.store_mode : default_store_mode;
    int mode = store_mode == 3 ? 2 : (tune.copy_mode != 0 ? tune.copy_mode : (prm.n > 16 ? 2 : 1));
    // Lane groups of 16 lanes on fp32 replicas (a warp is 8 columns wide: 2 or 4 workers per lane with more than 16
    // or 32 workers, shapes only an explicit workers_per_lane reaches in plain steps) gave wrong sums in the first
    // tiles of a CTA when their stages were filled by box copies and handed back before the results were stored;
    // filled by row copies, or held until the store warp has sent them (in place), they are right.  The cause is
    // not understood, so these shapes take row copies whatever was asked for.
    if (g == 16 && elem == 4 && store_mode != 3) mode = 1;
    sh.use_boxes = mode == 2;
    if (sh.use_boxes) {
        sh.box_cols = box_cols;
        sh.boxes_per_tile = sh.tile_cols / sh.box_cols;
        sh.row_bytes = (uint32_t)(sh.box_cols * elem);
    } else {
        // rows lie side by side, each shifted by 16 bytes (4 banks) against the one before
        sh.box_cols = sh.tile_cols;
        sh.boxes_per_tile = 1;
        sh.row_bytes = (uint32_t)(sh.tile_cols * elem) + 16u;
    }
    sh.box_tx_bytes = (uint32_t)prm.n * sh.row_bytes;
    sh.box_bytes = (sh.box_tx_bytes + 127u) / 128u * 128u;
    sh.array_bytes = (uint32_t)sh.boxes_per_tile * sh.box_bytes;
    sh.stage_bytes = (2u * sh.array_bytes + 127u) / 128u * 128u;
    sh.tiles = (prm.d + sh.tile_cols - 1) / sh.tile_cols;
    sh.store_mode = store_mode;
    sh.out_box_cols = box_cols;
    sh.out_boxes_per_tile = sh.tile_cols / sh.out_box_cols;
    sh.out_row_bytes = (uint32_t)(sh.out_box_cols * elem);
    sh.out_box_bytes = ((uint32_t)prm.n * sh.out_row_bytes + 127u) / 128u * 128u;
    sh.out_bytes = (uint32_t)sh.out_boxes_per_tile * sh.out_box_bytes;
    const size_t out_total = store_mode == 2 ? (size_t)kOutBuffers * sh.out_bytes : 0;
    int stages = tune.stages > 0 ? tune.stages : 2;
    if (stages > kMaxStages) stages = kMaxStages;
    while (stages > 2 && kSmemHeaderBytes + (size_t)stages * sh.stage_bytes + out_total > smem_limit) --stages;
    if (stages < 2 || kSmemHeaderBytes + (size_t)stages * sh.stage_bytes + out_total > smem_limit) return false;
    sh.stages = stages;
    sh.wait_limit_ns = tune.wait_limit_ms > 0 ? (uint64_t)tune.wait_limit_ms * 1000000ull : kDefaultWaitLimitNs;
    sh.withhold_copies = tune.withhold_copies;
    sh.descending = prm.descending;
    sh.evict_first_targets = (tune.l2_policy != 0 ? tune.l2_policy : kDefaultL2Policy) == 2;
    sh.early_targets = (tune.early_targets != 0 ? tune.early_targets : kDefaultEarlyTargets) == 2;
    sh.out_offset = (uint32_t)stages * sh.stage_bytes;
    out->threads = (warps + (store_mode == 3 ? 2 : 1)) * 32;
    out->smem_bytes = kSmemHeaderBytes + (uint32_t)stages * sh.stage_bytes + (uint32_t)out_total;
    return true;
}

// The plan with as many compute warps as asked for (or the default) that still fits in shared memory.
bool make_plan(const FusedParams& prm, const FusedTuning& tune, int vec, int wpt, int g, size_t elem,
               size_t smem_limit, Plan* out)
{
    // Defaults from sweeps on B200.  A lane holding 2 or 4 workers: 16 light compute warps and a separate
    // output tile (the ring is small).  A lane holding 8 workers: 12 heavier warps, and no room for output
    // tiles: fp32 results go back in place through the store warp, bf16 results (half the bytes per
    // replica-param, bound by instruction issue rather than by HBM) leave straight from registers.
    int warps = tune.consumer_warps > 0 ? tune.consumer_warps : (wpt >= 8 ? 12 : 16);
    if (warps > max_consumer_warps(wpt, vec, (int)elem)) warps = max_consumer_warps(wpt, vec, (int)elem);
    const int default_store_mode = wpt >= 8 ? (elem == 2 ? 1 : 3) : 2;
    for (; warps >= 1; --warps)
        if (shape_for(prm, tune, vec, g, elem, smem_limit, warps, default_store_mode, out)) return true;
    return false;
}


template <typename T, int VEC, int WPT, int G, bool GRAD = false, bool DIAG = false>
cudaError_t launch_staged_as(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    auto kernel = rps_fused_staged_kernel<T, VEC, WPT, G, GRAD, DIAG>;
    static LaunchState state;  // of this instantiation, per device
    size_t smem_limit = 0;
    cudaError_t err = smem_limit_of_device(state, &smem_limit);
    if (err != cudaSuccess) return err;
    Plan plan;
    if (!make_plan(prm, tune, VEC, WPT, G, sizeof(T), smem_limit, &plan)) return cudaErrorInvalidConfiguration;
    constexpr bool bf16 = sizeof(T) == 2;
    alignas(64) CUtensorMap map_x, map_b, map_out;
    const int map_box_cols = plan.shape.use_boxes ? plan.shape.box_cols : 16;  // unused by 1-D copies, but valid
    if (!encode_rows(&map_x, prm.x, bf16, prm, map_box_cols, prm.cols_in_row) ||
        !encode_rows(&map_b, prm.b, bf16, prm, map_box_cols, prm.cols_in_row) ||
        !encode_rows(&map_out, prm.x, bf16, prm, plan.shape.out_box_cols, prm.d))
        return cudaErrorInvalidValue;
    if ((err = grant_smem(state, kernel, plan.smem_bytes)) != cudaSuccess) return err;
    int occ_per_sm = 1;
    if ((err = resident_ctas_per_sm(state, kernel, plan.threads, plan.smem_bytes, &occ_per_sm)) != cudaSuccess) return err;
    // persistent CTAs: a whole number of resident CTAs per SM, each striding over the tiles
    int64_t grid = (int64_t)sm_count * occ_per_sm;
    if (grid > plan.shape.tiles) grid = plan.shape.tiles;
    if (grid < 1) grid = 1;
    if ((tune.launch_overlap != 0 ? tune.launch_overlap : kDefaultLaunchOverlap) == 2) {
        cudaLaunchConfig_t config = {};
        config.gridDim = dim3((unsigned)grid);
        config.blockDim = dim3((unsigned)plan.threads);
        config.dynamicSmemBytes = plan.smem_bytes;
        config.stream = stream;
        cudaLaunchAttribute attribute[1];
        attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attribute[0].val.programmaticStreamSerializationAllowed = 1;
        config.attrs = attribute;
        config.numAttrs = 1;
        return cudaLaunchKernelEx(&config, kernel, prm, plan.shape, map_x, map_b, map_out);
    }
    kernel<<<(unsigned)grid, plan.threads, plan.smem_bytes, stream>>>(prm, plan.shape, map_x, map_b, map_out);
    return cudaGetLastError();
}

// The one family of lane shapes (4 workers per lane, 2 for n <= 2) in which the optional forms of the
// step (gradient averaging, tracking) are built.
template <typename T, int VEC, bool GRAD, bool DIAG>
cudaError_t launch_staged_light(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    const int n = prm.n;
    if (n <= 2) return launch_staged_as<T, VEC, 2, 1, GRAD, DIAG>(prm, tune, sm_count, stream);
    if (n <= 4) return launch_staged_as<T, VEC, 4, 1, GRAD, DIAG>(prm, tune, sm_count, stream);
    if (n <= 8) return launch_staged_as<T, VEC, 4, 2, GRAD, DIAG>(prm, tune, sm_count, stream);
    if (n <= 16) return launch_staged_as<T, VEC, 4, 4, GRAD, DIAG>(prm, tune, sm_count, stream);
    if (n <= 32) return launch_staged_as<T, VEC, 4, 8, GRAD, DIAG>(prm, tune, sm_count, stream);
    return launch_staged_as<T, VEC, 4, 16, GRAD, DIAG>(prm, tune, sm_count, stream);
}

}  // namespace

}  // namespace rps
