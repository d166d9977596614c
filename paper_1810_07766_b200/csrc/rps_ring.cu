// Fused RPS step, self-refilling ring (sm_100a).  The shape for replicas whose step is bound by
// instruction issue rather than by HBM (bf16: half the bytes for the same arithmetic per replica-param).
//
// What such a step needs is as many compute warps as the register file holds, and the register file is
// handed out by warp scheduler: 16 warps of 128 registers fill it, a 17th warp (a producer) would cut every
// warp to 96.  So here every warp computes and nobody only produces:
//
//   * A tile is team_warps x WARP_COLS columns of all n rows of x and b, cut into team_warps slices of
//     WARP_COLS columns, one warp's work each.  Tile L of the CTA lives in stage L mod stages of a
//     shared-memory ring filled by TMA box copies (cp.async.bulk.tensor.2d, completion on the stage's
//     mbarrier).  Tiles of 8 slices (64 KB at n = 64) instead of 16 are what lets a ring of three stages fit
//     beside 16 compute warps.
//   * A warp that is free takes the next slice of the next tile from one counter: no warp is tied to a tile
//     or to a position in it, so 16 warps share tiles of any number of slices evenly, about 16 / team_warps
//     tiles are in work at a time, and a warp that fell behind holds nobody up.
//   * A warp copies its slices of the stage to registers and counts itself off on the stage's counter
//     (a shared-memory atomic).  The warp that counts last knows the stage is free: it resets the
//     counter and issues the copies of the tile that comes `stages` tiles later, then goes on computing.
//     No thread ever waits for a free stage; the only waits are the bounded ones for a tile's copies to be
//     issued (a counter per stage) and to land (the stage's mbarrier).
//
//   * Results leave either straight from registers with 16-byte streaming stores, or in place: x and b then
//     have rings of their own; a b tile is handed back as soon as it has been read, the results are written
//     over the x tile they came from, and the last warp to have written its part of a tile sends the tile out with
//     TMA tensor stores of whole boxes (whole 512-byte pieces of rows instead of the 64 bytes a lane group
//     covers at n = 64), sees the unit finish reading it and refills the stage.
//
// The arithmetic is rps_device.cuh's, the lane mapping the staged kernel's.
#include "rps_device.cuh"
#include "rps_tma.cuh"

namespace rps {

namespace {

constexpr int kRingMaxStages = 8;
constexpr int kRingDefaultStoreMode = 1;  // 1 stores from registers, 3 in place + TMA tensor stores
constexpr int kRingWarps = 16;  // 16 warps x 32 lanes x 128 registers = the whole register file
// two sets (x ring, b ring) of: landed-data barriers, counters of warps done with a stage, counts of fills issued
constexpr uint32_t kRingSyncBytes = 2 * kRingMaxStages * (8 + 4 + 4) + 4 * kRingWarps * 4;  // + the output tiles' counters, the tile counters
constexpr uint32_t kRingHeaderBytes = kRingSyncBytes + 2 * kMaxWorkers * 8 + kMaxWorkers * 4 + 128;  // + masks, flags
constexpr uint32_t kRingFlagOffset = kRingHeaderBytes - 128;
static_assert(kRingSyncBytes % 128 == 0 && kRingHeaderBytes % 128 == 0, "tile data must start on a 128-byte boundary");

struct RingShape {
    int64_t tiles;
    int32_t x_stages;       // depth of the ring of x tiles
    int32_t b_stages;       // depth of the ring of b tiles (the same, and filled together, unless results go back in place)
    int32_t team_warps;     // warp slices per tile
    int32_t teams;          // tiles in work at a time: warps of the CTA / team_warps, rounded up
    int32_t tile_cols;      // team_warps x WARP_COLS
    int32_t box_cols;       // columns per TMA box (<= 256); a tile is boxes_per_tile boxes side by side
    int32_t boxes_per_tile;
    uint32_t row_bytes;     // bytes of one row of one box
    uint32_t box_tx_bytes;  // bytes one box copy delivers: n rows
    uint32_t box_bytes;     // the same rounded up to 128
    uint32_t array_bytes;   // one tile of one array: all its boxes
    uint32_t b_ring_offset; // of the b ring from the start of the x ring
    uint32_t out_offset;    // of the teams' output tiles from the start of the x ring (store_mode 2)
    // 1: results leave from registers with 16-byte stores.  2: through one of `teams` output tiles in shared
    // memory and TMA tensor stores of whole boxes.  In both a tile's x and b share one barrier and one
    // counter and are handed back as soon as they have been read.  3: results are written back over the x
    // tile and leave as TMA tensor stores from there; the b tile is handed back as soon as it has been read,
    // the x tile after its store.
    int32_t store_mode;
    uint64_t wait_limit_ns;
    int32_t withhold_copies;  // test aid: nothing is ever copied, so that the waits run out
    int32_t descending;       // 1: the tiles are taken from the last to the first (odd steps)

    __device__ __forceinline__ int64_t tile_of_turn(int64_t turn) const { return descending ? tiles - 1 - turn : turn; }
};

// One ring's bookkeeping in shared memory.
struct RingSync {
    uint64_t* full;       // [stages] mbarrier: the tile's copies have landed
    int* done;            // [stages] warps that are done with the stage (team_warps of them free it)
    volatile int* fills;  // [stages] fills issued so far
};

__device__ __forceinline__ uint32_t count_off(int* counter)
{
    uint32_t old;
    asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(smem_addr(counter)) : "memory");
    return old;
}

// Waits until *counter >= want; gives up after limit_ns.
__device__ __forceinline__ bool wait_for_count(const volatile int* counter, int want, uint64_t limit_ns)
{
    if (*counter >= want) return true;
    const uint64_t start = global_timer_ns();
#pragma unroll 1
    for (;;) {
        if (*counter >= want) return true;
        if (global_timer_ns() - start > limit_ns) return false;
        __nanosleep(64);
    }
}

// Where a warp stands in a ring: stage, parity and number of the fill it waits for next.
struct RingCursor {
    int stage;
    uint32_t phase;
    int fill_no;
    __device__ __forceinline__ RingCursor(uint32_t local, uint32_t stages)
        : stage((int)(local % stages)), phase((local / stages) & 1u), fill_no((int)(local / stages) + 1)
    {
    }
    // A parity wait can only tell a phase from the one before it, and the tile that had this stage last may
    // still be with a slower warp: first see that this tile's fill has been issued (which happens only after the
    // earlier tile was done with), then wait for it to land.
    __device__ __forceinline__ bool wait(const RingSync& ring, uint64_t limit_ns) const
    {
        return wait_for_count(&ring.fills[stage], fill_no, limit_ns) &&
               mbar_wait(smem_addr(&ring.full[stage]), phase, limit_ns);
    }
};

template <typename T, int VEC, int WPT, int G, bool GRAD>
__global__ void __launch_bounds__(kRingWarps * 32, 1)
    rps_fused_ring_kernel(const FusedParams prm, const RingShape shape, const __grid_constant__ CUtensorMap map_x,
                          const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_out)
{
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    constexpr uint32_t elem = (uint32_t)sizeof(T);
    using Raw = typename RowVec<T, VEC>::Raw;
    extern __shared__ __align__(128) unsigned char smem[];
    const RingSync xs{reinterpret_cast<uint64_t*>(smem), reinterpret_cast<int*>(smem + 128),
                      reinterpret_cast<volatile int*>(smem + 192)};
    const RingSync bs{reinterpret_cast<uint64_t*>(smem + 64), reinterpret_cast<int*>(smem + 160),
                      reinterpret_cast<volatile int*>(smem + 224)};
    uint64_t* s_up = reinterpret_cast<uint64_t*>(smem + kRingSyncBytes);  // copy of this step's masks
    uint64_t* s_down = s_up + kMaxWorkers;
    float* s_inv = reinterpret_cast<float*>(s_down + kMaxWorkers);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kRingFlagOffset);
    unsigned char* x_ring = smem + kRingHeaderBytes;
    unsigned char* b_ring = x_ring + shape.b_ring_offset;
    int* out_done = reinterpret_cast<int*>(smem + 256);                    // [teams] warps that have written their results
    volatile int* out_free = reinterpret_cast<volatile int*>(smem + 320);  // [teams] stores that have left the output tile
    int* next_item = reinterpret_cast<int*>(smem + 384);                   // next (tile, slice) of the CTA that no warp has taken

    const int n = prm.n;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const bool in_place = shape.store_mode == 3, out_tiles = shape.store_mode == 2;
    // tiles of this CTA: turns blockIdx.x, blockIdx.x + gridDim.x, ...
    const int64_t my_tiles =
        (int64_t)blockIdx.x < shape.tiles ? (shape.tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kRingMaxStages; ++s) {
            mbar_init(smem_addr(&xs.full[s]), 1);
            mbar_init(smem_addr(&bs.full[s]), 1);
            xs.done[s] = bs.done[s] = 0;
            xs.fills[s] = bs.fills[s] = 0;
        }
        for (int k = 0; k < kRingWarps; ++k) out_done[k] = out_free[k] = 0;
        *next_item = 0;
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
        if (in_place || out_tiles) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_out) : "memory");
    }
    // With programmatic stream serialization this CTA may have been placed while the kernel before it in
    // the stream was still draining: let the next kernel do the same, then wait for the one before to
    // complete before reading anything from global memory.  Both are no-ops in a plain launch.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int j = threadIdx.x; j < kMaxWorkers; j += blockDim.x) {
        const bool used = j < n;
        s_up[j] = used ? prm.masks->up[j] : 0;
        s_down[j] = used ? prm.masks->down[j] : 0;
        s_inv[j] = used ? prm.masks->inv_cnt[j] : 0.0f;
    }
    __syncthreads();  // the only CTA-wide barrier

    // Issues the copies of the CTA's tile `local`: of x (with_x) and/or b (with_b) into their stages.  Called
    // by one thread once the stage is free.  Without in-place results a tile's x and b arrive together on the
    // b ring's barrier.  Boxes always arrive whole (zeros past the pitch), so the byte count is fixed.
    auto fill = [&](int64_t local, bool with_x, bool with_b) {
        const int64_t tile = shape.tile_of_turn((int64_t)blockIdx.x + local * gridDim.x);
        const int32_t c0 = (int32_t)(tile * shape.tile_cols);
        const uint32_t tile_tx = (uint32_t)shape.boxes_per_tile * shape.box_tx_bytes;
        const int sx = (int)(local % shape.x_stages), sb = (int)(local % shape.b_stages);
        const uint32_t x_bar = smem_addr(in_place ? &xs.full[sx] : &bs.full[sb]), b_bar = smem_addr(&bs.full[sb]);
        const uint32_t x_dst = smem_addr(x_ring) + (uint32_t)sx * shape.array_bytes;
        const uint32_t b_dst = smem_addr(b_ring) + (uint32_t)sb * shape.array_bytes;
        if (in_place) {
            if (with_x) {
                xs.fills[sx] = xs.fills[sx] + 1;
                mbar_arrive_expect_tx(x_bar, tile_tx);
            }
            if (with_b) {
                bs.fills[sb] = bs.fills[sb] + 1;
                mbar_arrive_expect_tx(b_bar, tile_tx);
            }
        } else {
            bs.fills[sb] = bs.fills[sb] + 1;
            mbar_arrive_expect_tx(b_bar, 2u * tile_tx);
        }
        for (int k = 0; k < shape.boxes_per_tile; ++k) {
            const int32_t col = c0 + k * shape.box_cols;
            if (with_x) tma_load_box(x_dst + (uint32_t)k * shape.box_bytes, &map_x, col, 0, x_bar);
            if (with_b) tma_load_box(b_dst + (uint32_t)k * shape.box_bytes, &map_b, col, 0, b_bar);
        }
    };
    if (threadIdx.x == 0 && !shape.withhold_copies) {
        const int most = shape.x_stages > shape.b_stages ? shape.x_stages : shape.b_stages;
        for (int64_t local = 0; local < my_tiles && local < most; ++local)
            fill(local, local < shape.x_stages, local < shape.b_stages);
    }

    T* __restrict__ xg = static_cast<T*>(prm.x);
    const MaskView masks{s_up, s_down, s_inv};
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;
    BlockCursor cursor;
    bool stores_pending = false;
    // What a warp does when something it waited for never came: say so, stop the refilling, and see the
    // copies that were issued land and its own stores leave (bounded) before its part of the CTA's shared
    // memory is given up.  Warps that still wait for something this warp will not count itself off on run
    // into their own limit.
    auto give_up = [&](int code) {
        report_timeout(prm, code);
        *abort_flag = 1;
        if (lane != 0) return;
        bool landed = true;
        for (int s = 0; s < kRingMaxStages && landed; ++s) {
            if (xs.fills[s] > 0)
                landed = mbar_wait(smem_addr(&xs.full[s]), (uint32_t)(xs.fills[s] - 1) & 1u, shape.wait_limit_ns);
            if (landed && bs.fills[s] > 0)
                landed = mbar_wait(smem_addr(&bs.full[s]), (uint32_t)(bs.fills[s] - 1) & 1u, shape.wait_limit_ns);
        }
        if (stores_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    };
    for (;;) {
        // the next slice of WARP_COLS columns, of the next tile of the CTA, that no warp has taken
        uint32_t taken = 0;
        if (lane == 0) taken = (uint32_t)atomicAdd(next_item, 1);
        taken = __shfl_sync(0xFFFFFFFFu, taken, 0);
        const int64_t local = taken / (uint32_t)shape.team_warps;
        if (local >= my_tiles) break;
        const int slot = (int)(taken % (uint32_t)shape.team_warps);
        const int col_in_tile = slot * WARP_COLS + sub * VEC;
        const uint32_t lane_off =
            (uint32_t)(col_in_tile / shape.box_cols) * shape.box_bytes + (uint32_t)(col_in_tile % shape.box_cols) * elem;
        const RingCursor at_x((uint32_t)local, (uint32_t)shape.x_stages), at_b((uint32_t)local, (uint32_t)shape.b_stages);
        if (!__all_sync(0xFFFFFFFFu, (!in_place || at_x.wait(xs, shape.wait_limit_ns)) && at_b.wait(bs, shape.wait_limit_ns))) {
            give_up(2);
            return;
        }
        const int64_t tile = shape.tile_of_turn((int64_t)blockIdx.x + local * gridDim.x);
        const int64_t c = tile * shape.tile_cols + col_in_tile;
        const bool col_live = c < prm.d;
        unsigned char* x_base = x_ring + (size_t)at_x.stage * shape.array_bytes + lane_off;
        const unsigned char* b_base = b_ring + (size_t)at_b.stage * shape.array_bytes + lane_off;

        auto hand_back = [&] {
            __syncwarp();
            if (lane == 0 && count_off(&bs.done[at_b.stage]) == (uint32_t)shape.team_warps - 1u) {
                bs.done[at_b.stage] = 0;  // seen by the stage's next readers through the barrier the refill completes
                const int64_t next = local + shape.b_stages;
                if (next < my_tiles && !*abort_flag) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // reads before the unit's writes
                    fill(next, !in_place, true);
                }
            }
        };
        float v[WPT][VEC];
        {
            Raw raw_x[WPT], raw_b[WPT];
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                // workers past n read the last real row: their mask bits are 0 and they are never stored
                const int row = w_first + w < n ? w_first + w : n - 1;
                raw_x[w] = *reinterpret_cast<const Raw*>(x_base + (size_t)row * shape.row_bytes);
                raw_b[w] = *reinterpret_cast<const Raw*>(b_base + (size_t)row * shape.row_bytes);
            }
            // This warp has everything it needs from the tile (from its b half, if results go back in place).
            // The last warp to say so refills the stage with the tile that comes b_stages later.  (Gradient
            // averaging reads x a second time after the average and hands the tile back only then.)
            if (!GRAD) hand_back();
            local_sgd_raw<T, VEC, WPT, GRAD>(raw_x, raw_b, v, c, w_first, prm);
        }
        const uint32_t live_bits = average_and_select<VEC, WPT, G>(v, c, col_live, w_first, masks, cursor, prm);
        if (GRAD) {
            // v holds the update each worker applies (the average one where it arrived): x_{t+1} = x + update
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                const int row = w_first + w < n ? w_first + w : n - 1;
                float xv[VEC];
                RowVec<T, VEC>::unpack(*reinterpret_cast<const Raw*>(x_base + (size_t)row * shape.row_bytes), xv);
#pragma unroll
                for (int e = 0; e < VEC; ++e) v[w][e] += xv[e];
            }
            hand_back();
        }
        if (in_place || out_tiles) {
            unsigned char* out_base = x_base;
            const int out_slot = (int)((uint32_t)local % (uint32_t)shape.teams);
            const int out_turn = (int)((uint32_t)local / (uint32_t)shape.teams);
            if (out_tiles) {
                // tile L goes out through output tile L mod teams, which is free once the store of the tile
                // that had it before has read it
                if (!__all_sync(0xFFFFFFFFu, wait_for_count(&out_free[out_slot], out_turn, shape.wait_limit_ns))) {
                    give_up(3);
                    return;
                }
                out_base = x_ring + shape.out_offset + (size_t)out_slot * shape.array_bytes + lane_off;
            }
            // in place every lane overwrites exactly the slices of x it read; columns past d are clipped by the store
#pragma unroll
            for (int w = 0; w < WPT; ++w)
                if (w_first + w < n)
                    *reinterpret_cast<Raw*>(out_base + (size_t)(w_first + w) * shape.row_bytes) = RowVec<T, VEC>::pack(v[w]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // visible to the TMA unit
            __syncwarp();
            // The last warp to have written its part sends the tile to global memory and sees the unit finish
            // reading it; then the output tile is free for the next tile that uses it, or (in place) the stage is
            // refilled with the x tile that comes x_stages later.
            int* done = in_place ? &xs.done[at_x.stage] : &out_done[out_slot];
            if (lane == 0 && count_off(done) == (uint32_t)shape.team_warps - 1u) {
                *done = 0;
                const int32_t c0 = (int32_t)(tile * shape.tile_cols);
                const uint32_t src = in_place ? smem_addr(x_ring) + (uint32_t)at_x.stage * shape.array_bytes
                                              : smem_addr(x_ring) + shape.out_offset + (uint32_t)out_slot * shape.array_bytes;
                for (int k = 0; k < shape.boxes_per_tile; ++k) {
                    const int32_t col = c0 + k * shape.box_cols;
                    if (col < prm.d) tma_store_box(&map_out, col, 0, src + (uint32_t)k * shape.box_bytes);
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                stores_pending = true;
                if (out_tiles) {
                    __threadfence_block();
                    out_free[out_slot] = out_turn + 1;
                } else {
                    const int64_t next = local + shape.x_stages;
                    if (next < my_tiles && !*abort_flag) fill(next, true, false);
                }
            }
        } else {
            T* dst = xg + (int64_t)w_first * prm.pitch + c;  // this lane's slice of its first worker's row
            if (live_bits == (1u << VEC) - 1u) {
#pragma unroll
                for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                    if (w_first + w < n) __stcs(reinterpret_cast<Raw*>(dst), RowVec<T, VEC>::pack(v[w]));
            } else if (live_bits != 0) {
#pragma unroll
                for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                    if (w_first + w < n) store_ragged<T, VEC>(dst, v[w], live_bits);
            }
        }
    }
    // tensor stores issued by this thread still read this CTA's shared memory: see them through
    if (stores_pending) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// Tiles and ring depths for one instantiation: the number of slices per tile asked for if rings of two
// stages fit, else the largest (from 8 down) whose tiles leave room for as many stages as tiles are in work.
bool plan_ring(const FusedParams& prm, const FusedTuning& tune, int vec, int g, size_t elem, size_t smem_limit,
               RingShape* sh, uint32_t* smem_bytes)
{
    const int warp_cols = (32 / g) * vec;
    int team_warps = tune.team_warps > 0 ? tune.team_warps : 8;
    if (team_warps > kRingWarps) team_warps = kRingWarps;
    const int team_asked = team_warps;
    sh->store_mode = tune.store_mode != 0 ? tune.store_mode : kRingDefaultStoreMode;
    for (; team_warps >= 1; team_warps = team_warps > 8 ? 8 : team_warps / 2) {
        sh->team_warps = team_warps;
        sh->teams = (kRingWarps + team_warps - 1) / team_warps;  // tiles in work at a time, rounded up
        sh->tile_cols = team_warps * warp_cols;
        // the widest box (<= 256 elements) that tiles the tile exactly; warp_cols always does
        int box_cols = warp_cols;
        for (int k = 1; k <= team_warps; ++k)
            if (team_warps % k == 0 && k * warp_cols <= 256) box_cols = k * warp_cols;
        sh->box_cols = box_cols;
        sh->boxes_per_tile = sh->tile_cols / box_cols;
        sh->row_bytes = (uint32_t)(box_cols * elem);
        sh->box_tx_bytes = (uint32_t)prm.n * sh->row_bytes;
        sh->box_bytes = (sh->box_tx_bytes + 127u) / 128u * 128u;
        sh->array_bytes = (uint32_t)sh->boxes_per_tile * sh->box_bytes;
        // shared memory holds `units` tiles of one array; an x tile is held through the arithmetic when
        // results go back in place, a b tile only until it has been read: the odd unit goes to x
        const int out_units = sh->store_mode == 2 ? sh->teams : 0;  // one output tile per tile in work
        const int units = (int)((smem_limit - kRingHeaderBytes) / sh->array_bytes) - out_units;
        int b_stages = units / 2, x_stages = sh->store_mode == 3 ? units - b_stages : b_stages;
        if (tune.stages > 0 && b_stages > tune.stages) b_stages = tune.stages;
        if (tune.stages > 0 && x_stages > tune.stages) x_stages = tune.stages;
        if (b_stages > kRingMaxStages) b_stages = kRingMaxStages;
        if (x_stages > kRingMaxStages) x_stages = kRingMaxStages;
        // a team size that was asked for is kept if rings of two stages fit at all
        const bool asked = tune.team_warps > 0 && team_warps == team_asked;
        const int enough = sh->store_mode == 3 ? sh->teams + 1 : sh->teams;
        if (b_stages >= 2 && (x_stages >= enough || asked || team_warps == 1)) {
            sh->x_stages = x_stages;
            sh->b_stages = b_stages;
            sh->b_ring_offset = (uint32_t)x_stages * sh->array_bytes;
            sh->out_offset = (uint32_t)(x_stages + b_stages) * sh->array_bytes;
            sh->tiles = (prm.d + sh->tile_cols - 1) / sh->tile_cols;
            sh->wait_limit_ns = tune.wait_limit_ms > 0 ? (uint64_t)tune.wait_limit_ms * 1000000ull : kDefaultWaitLimitNs;
            sh->withhold_copies = tune.withhold_copies;
            sh->descending = prm.descending;
            *smem_bytes = kRingHeaderBytes + (uint32_t)(x_stages + b_stages + out_units) * sh->array_bytes;
            return true;
        }
    }
    return false;
}

template <typename T, int VEC, int WPT, int G, bool GRAD = false>
cudaError_t launch_ring_as(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    auto kernel = rps_fused_ring_kernel<T, VEC, WPT, G, GRAD>;
    static LaunchState state;  // of this instantiation, per device
    size_t smem_limit = 0;
    cudaError_t err = smem_limit_of_device(state, &smem_limit);
    if (err != cudaSuccess) return err;
    RingShape shape;
    uint32_t smem_bytes = 0;
    FusedTuning shaped = tune;
    if (GRAD) shaped.store_mode = 1;  // gradient averaging is built with results leaving from registers
    if (!plan_ring(prm, shaped, VEC, G, sizeof(T), smem_limit, &shape, &smem_bytes)) return cudaErrorInvalidConfiguration;
    constexpr bool bf16 = sizeof(T) == 2;
    alignas(64) CUtensorMap map_x, map_b, map_out;
    // loads may read up to the pitch (padding arrives and is ignored); stores end at column d
    if (!encode_rows(&map_x, prm.x, bf16, prm, shape.box_cols, prm.cols_in_row) ||
        !encode_rows(&map_b, prm.b, bf16, prm, shape.box_cols, prm.cols_in_row) ||
        !encode_rows(&map_out, prm.x, bf16, prm, shape.box_cols, prm.d))
        return cudaErrorInvalidValue;
    if ((err = grant_smem(state, kernel, smem_bytes)) != cudaSuccess) return err;
    // persistent CTAs, one per SM (a CTA is the whole register file), each striding over the tiles
    int64_t grid = sm_count;
    if (grid > shape.tiles) grid = shape.tiles;
    if (grid < 1) grid = 1;
    cudaLaunchConfig_t config = {};
    config.gridDim = dim3((unsigned)grid);
    config.blockDim = dim3(kRingWarps * 32);
    config.dynamicSmemBytes = smem_bytes;
    config.stream = stream;
    cudaLaunchAttribute attribute[1];
    attribute[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attribute[0].val.programmaticStreamSerializationAllowed = 1;
    config.attrs = attribute;
    config.numAttrs = tune.launch_overlap == 1 ? 0 : 1;
    return cudaLaunchKernelEx(&config, kernel, prm, shape, map_x, map_b, map_out);
}

}  // namespace

bool ring_kernel_covers(const FusedParams& prm, bool bf16)
{
    // built for bf16 replicas with 8 workers per lane, untracked (models or gradients averaged); TMA coordinates are 32-bit
    return bf16 && prm.n > 4 && prm.trace == nullptr && prm.pitch < ((int64_t)1 << 31);
}

cudaError_t launch_fused_ring(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                              cudaStream_t stream)
{
    if (!ring_kernel_covers(prm, bf16)) return cudaErrorInvalidConfiguration;
    const int n = prm.n;
    if (prm.average_gradients) {
        if (n <= 8) return launch_ring_as<__nv_bfloat16, 8, 8, 1, true>(prm, tune, sm_count, stream);
        if (n <= 16) return launch_ring_as<__nv_bfloat16, 8, 8, 2, true>(prm, tune, sm_count, stream);
        if (n <= 32) return launch_ring_as<__nv_bfloat16, 8, 8, 4, true>(prm, tune, sm_count, stream);
        return launch_ring_as<__nv_bfloat16, 8, 8, 8, true>(prm, tune, sm_count, stream);
    }
    if (n <= 8) return launch_ring_as<__nv_bfloat16, 8, 8, 1>(prm, tune, sm_count, stream);
    if (n <= 16) return launch_ring_as<__nv_bfloat16, 8, 8, 2>(prm, tune, sm_count, stream);
    if (n <= 32) return launch_ring_as<__nv_bfloat16, 8, 8, 4>(prm, tune, sm_count, stream);
    return launch_ring_as<__nv_bfloat16, 8, 8, 8>(prm, tune, sm_count, stream);
}

}  // namespace rps
