// Thin wrappers over the sm_100a asynchronous-copy machinery used by the staged kernels: mbarriers
// with bounded waits, bulk and tensor (TMA) copies between global and shared memory, and the host-side
// encoding of a [n][pitch] array as a 2-D tensor map.
#pragma once

#include <cuda.h>

#include "rps_kernels.h"

namespace rps {

namespace {

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(arrivals) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

// How long a wait on an mbarrier lasts before the warp gives up, unless the caller sets another limit.
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;

// One try: the hardware may park the thread for up to `kSuspendHintNs` before answering.
constexpr uint32_t kSuspendHintNs = 1000000u;

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return done != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for the phase with the given parity to complete; gives up after limit_ns.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t limit_ns)
{
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t start = global_timer_ns();
#pragma unroll 1
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - start > limit_ns) return false;
    }
}

// TMA tensor copy global -> shared of one box whose first element is (column, row) of the
// tensor described by `map`; completion is signalled on `bar` as the box's bytes.
__device__ __forceinline__ void tma_load_box(uint32_t dst_smem, const CUtensorMap* map, int32_t column, int32_t row,
                                             uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            dst_smem),
        "l"(map), "r"(column), "r"(row), "r"(bar)
        : "memory");
}

// Bulk asynchronous copy global -> shared of one contiguous run of bytes; completion is signalled
// on `bar`.  Both addresses and the size are multiples of 16.
__device__ __forceinline__ void bulk_load_row(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// The same two copies carrying an L2 cache policy (made by createpolicy).
__device__ __forceinline__ void tma_load_box(uint32_t dst_smem, const CUtensorMap* map, int32_t column, int32_t row,
                                             uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, "
        "%3}], [%4], %5;" ::"r"(dst_smem),
        "l"(map), "r"(column), "r"(row), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ void bulk_load_row(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}

__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}

// TMA tensor store shared -> global of one box; the unit clips what lies outside the tensor (columns >= d).
__device__ __forceinline__ void tma_store_box(const CUtensorMap* map, int32_t column, int32_t row, uint32_t src_smem)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map), "r"(column),
                 "r"(row), "r"(src_smem)
                 : "memory");
}

__device__ __forceinline__ void report_timeout(const FusedParams& prm, int code)
{
    if (prm.error != nullptr) atomicExch(prm.error, code);
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled, fetched from the driver once (the library does not link libcuda).
EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult status;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &status) != cudaSuccess ||
            status != cudaDriverEntryPointSuccess)
            ptr = nullptr;
        return reinterpret_cast<EncodeTiledFn>(ptr);
    }();
    return fn;
}

// Describes one [n][pitch] array to the TMA unit, with boxes of box_rows rows x box_cols columns; `cols` columns
// of every row belong to the tensor (the pitch for loads, d for stores: what lies beyond is not written).
bool encode_boxes(CUtensorMap* map, const void* base, bool bf16, const FusedParams& prm, int box_cols, int box_rows,
                  int64_t cols)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (encode == nullptr) return false;
    const size_t elem = bf16 ? 2 : 4;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)prm.n};
    const cuuint64_t strides[1] = {(cuuint64_t)prm.pitch * elem};  // bytes between rows
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return encode(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                  const_cast<void*>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same with boxes that span all n rows.
bool encode_rows(CUtensorMap* map, const void* base, bool bf16, const FusedParams& prm, int box_cols, int64_t cols)
{
    return encode_boxes(map, base, bf16, prm, box_cols, prm.n, cols);
}

}  // namespace

}  // namespace rps
