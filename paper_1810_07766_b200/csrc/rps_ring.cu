// Fused RPS step, self-refilling ring (sm_100a).  The shape for replicas whose step is bound by
// instruction issue rather than by HBM (bf16: half the bytes for the same arithmetic per replica-param).
//
// What such a step needs is as many compute warps as the register file holds, and the register file is
// handed out by warp scheduler: 16 warps of 128 registers fill it, a 17th warp (a producer) would cut every
// warp to 96.  So here every warp computes and nobody only produces:
//
//   * The 16 warps of a CTA form teams of team_warps warps.  A tile (team_warps x WARP_COLS columns of
//     all n rows of x and b) belongs to one team; the CTA's tiles go to the teams in turn, and tile L
//     of the CTA lives in stage L mod stages of a shared-memory ring filled by TMA box copies
//     (cp.async.bulk.tensor.2d, completion on the stage's mbarrier).  Tiles of 8 warps (64 KB at n = 64)
//     instead of 16 are what lets a ring of three stages fit beside 16 compute warps.
//   * A warp copies its slices of the stage to registers and counts itself off on the stage's counter
//     (a shared-memory atomic).  The warp that counts last knows the stage is free: it resets the
//     counter and issues the copies of the tile that comes `stages` tiles later, then goes on computing.
//     No thread ever waits for a free stage; the only waits are the bounded ones for a tile's copies to be
//     issued (a counter per stage) and to land (the stage's mbarrier).
//
// The arithmetic is rps_device.cuh's, the lane mapping the staged kernel's; results leave straight from
// registers with 16-byte streaming stores.
#include "rps_device.cuh"
#include "rps_tma.cuh"

namespace rps {

namespace {

constexpr int kRingMaxStages = 8;
constexpr int kRingWarps = 16;  // 16 warps x 32 lanes x 128 registers = the whole register file
constexpr uint32_t kRingHeaderBytes = 128 + 2 * kMaxWorkers * 8 + kMaxWorkers * 4 + 128;  // barriers+counters, masks, flags
constexpr uint32_t kRingFlagOffset = kRingHeaderBytes - 128;
static_assert(kRingHeaderBytes % 128 == 0, "tile data must start on a 128-byte boundary");

struct RingShape {
    int64_t tiles;
    int32_t stages;
    int32_t team_warps;     // warps that share a tile
    int32_t teams;          // warps of the CTA / team_warps
    int32_t tile_cols;      // team_warps x WARP_COLS
    int32_t box_cols;       // columns per TMA box (<= 256); a tile is boxes_per_tile boxes side by side
    int32_t boxes_per_tile;
    uint32_t row_bytes;     // bytes of one row of one box
    uint32_t box_tx_bytes;  // bytes one box copy delivers: n rows
    uint32_t box_bytes;     // the same rounded up to 128
    uint32_t array_bytes;   // all boxes of one array
    uint32_t stage_bytes;   // both arrays
    uint64_t wait_limit_ns;
    int32_t withhold_copies;  // test aid: nothing is ever copied, so that the waits run out
    int32_t descending;       // 1: the tiles are taken from the last to the first (odd steps)

    __device__ __forceinline__ int64_t tile_of_turn(int64_t turn) const { return descending ? tiles - 1 - turn : turn; }
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

template <typename T, int VEC, int WPT, int G>
__global__ void __launch_bounds__(kRingWarps * 32, 1)
    rps_fused_ring_kernel(const FusedParams prm, const RingShape shape, const __grid_constant__ CUtensorMap map_x,
                          const __grid_constant__ CUtensorMap map_b)
{
    constexpr int LPG = 32 / G;
    constexpr int WARP_COLS = LPG * VEC;
    constexpr uint32_t elem = (uint32_t)sizeof(T);
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem);                 // [kRingMaxStages] data has landed
    int* readers = reinterpret_cast<int*>(smem + 64);                   // [kRingMaxStages] warps done reading
    volatile int* fills = reinterpret_cast<volatile int*>(smem + 96);   // [kRingMaxStages] fills issued so far
    uint64_t* s_up = reinterpret_cast<uint64_t*>(smem + 128);           // copy of this step's masks
    uint64_t* s_down = s_up + kMaxWorkers;
    float* s_inv = reinterpret_cast<float*>(s_down + kMaxWorkers);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kRingFlagOffset);
    unsigned char* ring = smem + kRingHeaderBytes;

    const int n = prm.n;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int team = warp / shape.team_warps;
    const int warp_in_team = warp - team * shape.team_warps;
    // tiles of this CTA: turns blockIdx.x, blockIdx.x + gridDim.x, ...
    const int64_t my_tiles =
        (int64_t)blockIdx.x < shape.tiles ? (shape.tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < shape.stages; ++s) {
            mbar_init(smem_addr(&full[s]), 1);
            readers[s] = 0;
            fills[s] = 0;
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
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

    // Copies of the CTA's tile `local` into its stage; called by one thread once the stage is free.
    auto fill = [&](int64_t local) {
        const int stage = (int)(local % shape.stages);
        const int64_t tile = shape.tile_of_turn((int64_t)blockIdx.x + local * gridDim.x);
        const int32_t c0 = (int32_t)(tile * shape.tile_cols);
        const uint32_t bar = smem_addr(&full[stage]);
        const uint32_t dst = smem_addr(ring) + (uint32_t)stage * shape.stage_bytes;
        fills[stage] = fills[stage] + 1;
        // boxes always arrive whole (zeros past the pitch), so the byte count is fixed
        mbar_arrive_expect_tx(bar, 2u * (uint32_t)shape.boxes_per_tile * shape.box_tx_bytes);
        for (int k = 0; k < shape.boxes_per_tile; ++k) {
            const int32_t col = c0 + k * shape.box_cols;
            tma_load_box(dst + (uint32_t)k * shape.box_bytes, &map_x, col, 0, bar);
            tma_load_box(dst + shape.array_bytes + (uint32_t)k * shape.box_bytes, &map_b, col, 0, bar);
        }
    };
    if (threadIdx.x == 0 && !shape.withhold_copies)
        for (int64_t local = 0; local < my_tiles && local < shape.stages; ++local) fill(local);

    T* __restrict__ xg = static_cast<T*>(prm.x);
    const MaskView masks{s_up, s_down, s_inv};
    const int sub = lane % LPG;
    const int w_first = (lane / LPG) * WPT;
    const int col_in_tile = warp_in_team * WARP_COLS + sub * VEC;
    const uint32_t lane_off =
        (uint32_t)(col_in_tile / shape.box_cols) * shape.box_bytes + (uint32_t)(col_in_tile % shape.box_cols) * elem;
    int stage = team % shape.stages;
    uint32_t phase = (uint32_t)(team / shape.stages) & 1u;
    BlockCursor cursor;
    for (int64_t local = team; local < my_tiles; local += shape.teams) {
        // A parity wait can only tell a phase from the one before it, and the tile that had this stage last
        // may belong to a slower team: first see that the fill of this tile has been issued (which happens
        // only after that earlier tile was read to the end), then wait for it to land.
        const int fill_no = (int)(local / shape.stages) + 1;
        if (!__all_sync(0xFFFFFFFFu, wait_for_count(&fills[stage], fill_no, shape.wait_limit_ns) &&
                                         mbar_wait(smem_addr(&full[stage]), phase, shape.wait_limit_ns))) {
            // The data never came.  Say so, stop refilling, and see the copies that were issued land (bounded)
            // before this warp's part of the CTA's shared memory is given up.  Warps that still wait for a
            // stage this warp will not count itself off on run into their own limit.
            report_timeout(prm, 2);
            *abort_flag = 1;
            if (lane == 0)
                for (int s = 0; s < shape.stages; ++s)
                    if (fills[s] > 0 && !mbar_wait(smem_addr(&full[s]), (uint32_t)(fills[s] - 1) & 1u, shape.wait_limit_ns))
                        break;
            return;
        }
        const int64_t tile = shape.tile_of_turn((int64_t)blockIdx.x + local * gridDim.x);
        const int64_t c = tile * shape.tile_cols + col_in_tile;
        const bool col_live = c < prm.d;
        const unsigned char* base = ring + (size_t)stage * shape.stage_bytes + lane_off;

        float v[WPT][VEC];
        {
            float xv[WPT][VEC], bv[WPT][VEC];
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                // workers past n read the last real row: their mask bits are 0 and they are never stored
                const int row = w_first + w < n ? w_first + w : n - 1;
                using Raw = typename RowVec<T, VEC>::Raw;
                const Raw raw_x = *reinterpret_cast<const Raw*>(base + (size_t)row * shape.row_bytes);
                const Raw raw_b = *reinterpret_cast<const Raw*>(base + shape.array_bytes + (size_t)row * shape.row_bytes);
                RowVec<T, VEC>::unpack(raw_x, xv[w]);
                RowVec<T, VEC>::unpack(raw_b, bv[w]);
            }
            // This warp has everything it needs from the stage.  The last warp of the team to say so
            // refills the stage with the tile that comes `stages` tiles later.
            __syncwarp();
            if (lane == 0 && count_off(&readers[stage]) == (uint32_t)shape.team_warps - 1u) {
                readers[stage] = 0;  // seen by the next readers through the barrier the refill completes
                const int64_t next = local + shape.stages;
                if (next < my_tiles && !*abort_flag) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // reads before the unit's writes
                    fill(next);
                }
            }
            local_sgd<VEC, WPT, false>(xv, bv, v, c, w_first, prm);
        }
        const uint32_t live_bits = average_and_select<VEC, WPT, G>(v, c, col_live, w_first, masks, cursor, prm);
        T* dst = xg + (int64_t)w_first * prm.pitch + c;  // this lane's slice of its first worker's row
        if (live_bits == (1u << VEC) - 1u) {
#pragma unroll
            for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                if (w_first + w < n) __stcs(reinterpret_cast<typename RowVec<T, VEC>::Raw*>(dst), RowVec<T, VEC>::pack(v[w]));
        } else if (live_bits != 0) {
#pragma unroll
            for (int w = 0; w < WPT; ++w, dst += prm.pitch)
                if (w_first + w < n) store_ragged<T, VEC>(dst, v[w], live_bits);
        }
        stage += shape.teams;
        while (stage >= shape.stages) {
            stage -= shape.stages;
            phase ^= 1u;
        }
    }
}

// Teams, tiles and ring depth for one instantiation: the team size asked for if a ring of two stages fits,
// else the largest team (from 8 warps down) whose tiles leave room for a ring of at least teams + 1 stages.
bool plan_ring(const FusedParams& prm, const FusedTuning& tune, int vec, int g, size_t elem, size_t smem_limit,
               RingShape* sh, uint32_t* smem_bytes)
{
    const int warp_cols = (32 / g) * vec;
    int team_warps = tune.team_warps > 0 ? tune.team_warps : 8;
    if (team_warps > kRingWarps) team_warps = kRingWarps;
    while (kRingWarps % team_warps != 0) --team_warps;
    const int sh_team_asked = team_warps;
    for (; team_warps >= 1; team_warps /= 2) {
        sh->team_warps = team_warps;
        sh->teams = kRingWarps / team_warps;
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
        sh->stage_bytes = 2u * sh->array_bytes;
        int fit = (int)((smem_limit - kRingHeaderBytes) / sh->stage_bytes);
        if (fit > kRingMaxStages) fit = kRingMaxStages;
        int stages = tune.stages > 0 ? tune.stages : fit;
        if (stages > fit) stages = fit;
        // a team size that was asked for is kept if a ring of two stages fits at all
        const bool asked = tune.team_warps > 0 && team_warps == sh_team_asked;
        if (stages >= sh->teams + 1 || (stages >= 2 && (asked || team_warps == 1))) {
            sh->stages = stages;
            sh->tiles = (prm.d + sh->tile_cols - 1) / sh->tile_cols;
            sh->wait_limit_ns = tune.wait_limit_ms > 0 ? (uint64_t)tune.wait_limit_ms * 1000000ull : kDefaultWaitLimitNs;
            sh->withhold_copies = tune.withhold_copies;
            sh->descending = prm.descending;
            *smem_bytes = kRingHeaderBytes + (uint32_t)stages * sh->stage_bytes;
            return true;
        }
    }
    return false;
}

template <typename T, int VEC, int WPT, int G>
cudaError_t launch_ring_as(const FusedParams& prm, const FusedTuning& tune, int sm_count, cudaStream_t stream)
{
    auto kernel = rps_fused_ring_kernel<T, VEC, WPT, G>;
    static size_t smem_limit = 0;  // opt-in shared memory per CTA of this device
    static uint32_t smem_granted = 0;
    cudaError_t err;
    if (smem_limit == 0) {
        int dev = 0, optin = 0;
        if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
        if ((err = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) != cudaSuccess)
            return err;
        smem_limit = (size_t)optin;
    }
    RingShape shape;
    uint32_t smem_bytes = 0;
    if (!plan_ring(prm, tune, VEC, G, sizeof(T), smem_limit, &shape, &smem_bytes)) return cudaErrorInvalidConfiguration;
    constexpr bool bf16 = sizeof(T) == 2;
    alignas(64) CUtensorMap map_x, map_b;
    if (!encode_rows(&map_x, prm.x, bf16, prm, shape.box_cols, prm.cols_in_row) ||
        !encode_rows(&map_b, prm.b, bf16, prm, shape.box_cols, prm.cols_in_row))
        return cudaErrorInvalidValue;
    if (smem_bytes > smem_granted) {
        if ((err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes)) !=
            cudaSuccess)
            return err;
        smem_granted = smem_bytes;
    }
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
    return cudaLaunchKernelEx(&config, kernel, prm, shape, map_x, map_b);
}

}  // namespace

bool ring_kernel_covers(const FusedParams& prm, bool bf16)
{
    // built for bf16 replicas with 8 workers per lane, plain model averaging, untracked; TMA coordinates are 32-bit
    return bf16 && prm.n > 4 && prm.trace == nullptr && !prm.average_gradients && prm.pitch < ((int64_t)1 << 31);
}

cudaError_t launch_fused_ring(const FusedParams& prm, const FusedTuning& tune, bool bf16, int sm_count,
                              cudaStream_t stream)
{
    if (!ring_kernel_covers(prm, bf16)) return cudaErrorInvalidConfiguration;
    const int n = prm.n;
    if (n <= 8) return launch_ring_as<__nv_bfloat16, 8, 8, 1>(prm, tune, sm_count, stream);
    if (n <= 16) return launch_ring_as<__nv_bfloat16, 8, 8, 2>(prm, tune, sm_count, stream);
    if (n <= 32) return launch_ring_as<__nv_bfloat16, 8, 8, 4>(prm, tune, sm_count, stream);
    return launch_ring_as<__nv_bfloat16, 8, 8, 8>(prm, tune, sm_count, stream);
}

}  // namespace rps
