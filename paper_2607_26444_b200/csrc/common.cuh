// Internal declarations shared by the kernels and the C-ABI layer (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "strata_moe.h"

namespace strata {

// ---- workspace layout -----------------------------------------------------
// word 0: device status (a strata_status, first error wins)
// word 1: ticket of the layout kernel (returns to 0 after every call)
// bytes [256, ...): per-tile, per-expert counts, int32 [n_tiles, E]
constexpr int kWsHeaderBytes = 256;
constexpr int kLayoutThreads = 1024;   // threads per layout CTA
constexpr int kItemsPerThread = 4;
constexpr int kLayoutTile = kLayoutThreads * kItemsPerThread;   // items per tile
constexpr int kMaxExperts = 1024;
constexpr int kMaxTopK = 32;

struct LayoutGeom {
    int items_per_rank;   // T*K
    int tiles_per_rank;   // ceil(T*K / kLayoutTile); a tile never spans two ranks
    int n_tiles;          // R * tiles_per_rank
};

inline LayoutGeom layout_geom(const strata_moe_shape& s)
{
    LayoutGeom g;
    g.items_per_rank = s.T * s.K;
    g.tiles_per_rank = (g.items_per_rank + kLayoutTile - 1) / kLayoutTile;
    g.n_tiles = s.R * g.tiles_per_rank;
    return g;
}

// Largest grid <= max_ctas in which round-robin dealing gives every CTA the same number of
// units (the last CTA may get fewer): no CTA is left with one extra unit at the tail.
inline long long balanced_grid(long long units, long long max_ctas)
{
    if (units <= 0) return 1;
    if (max_ctas < 1) max_ctas = 1;
    const long long per = (units + max_ctas - 1) / max_ctas;
    return (units + per - 1) / per;
}

// ---- launchers (defined next to their kernels) -----------------------------
cudaError_t launch_layout(const strata_moe_shape& s, const int32_t* ids, const strata_moe_layout_t& L,
                          int* ws_header, int* tile_cnt, cudaStream_t st, int* n_launches);
cudaError_t launch_dispatch_bf16(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv,
                                 size_t capacity_rows, int* status, int n_sm, cudaStream_t st);
cudaError_t launch_dispatch_fp8(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv_q,
                                float* recv_scale, size_t capacity_rows, int* status, int n_sm, cudaStream_t st);
cudaError_t launch_combine(const strata_moe_shape& s, const int32_t* dst_row, const void* y, size_t y_rows,
                           const float* w, void* out, int* status, int n_sm, cudaStream_t st);
cudaError_t configure_kernels(int device);

#ifdef __CUDACC__
// ---- device helpers --------------------------------------------------------
__device__ __forceinline__ void report_status(int* status, int code)
{
    atomicCAS(status, 0, code);   // first error wins
}

__device__ __forceinline__ uint32_t smem_addr(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// mbarrier (shared::cta) ------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within the iteration limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity)
{
    for (uint32_t it = 0; it < (1u << 22); ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// L2 eviction policies ----------------------------------------------------------
__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// Bulk asynchronous copies (the copy engine of the SM; no tensor map, 16-byte granularity).
// global -> this CTA's shared memory, completion counted in bytes on an mbarrier.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar,
                                         uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(smem_addr(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}
// this CTA's shared memory -> global, tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_addr(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_s2g_hint(void* gdst, const void* smem_src, uint32_t bytes, uint64_t policy)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(gdst),
                 "r"(smem_addr(smem_src)), "r"(bytes), "l"(policy)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// generic-proxy writes to shared memory become visible to the async proxy
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// streaming 16-byte global accesses ------------------------------------------------
__device__ __forceinline__ uint4 ld_stream16(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
#endif  // __CUDACC__

}  // namespace strata
