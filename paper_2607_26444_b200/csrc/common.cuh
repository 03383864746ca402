// Internal declarations shared by the kernels and the C-ABI layer (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "strata_moe.h"
#include "strata_collective.h"

namespace strata {

// ---- workspace layout -----------------------------------------------------
// word 0: device status (a strata_status, first error wins)
// word 1: ticket of the layout kernel (returns to 0 after every call)
// word 2: work-claim counter of dispatch, word 4: of combine, word 6: of the collectives (each returns
//         to 0 inside the kernel)
// bytes [256, ...): per-tile, per-expert counts, int32 [n_tiles, E]
// the last collective_table_bytes() bytes: pair table of all-to-all-v
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

// Launch-shape constants can be overridden from the environment in builds made with -DSTRATA_TUNE
// (measurement sweeps only); the shipped library compiles every call down to its default.
inline long long tune(const char* name, long long dflt)
{
#ifdef STRATA_TUNE
    const char* v = getenv(name);
    return (v && *v) ? atoll(v) : dflt;
#else
    (void)name;
    return dflt;
#endif
}

// rows of the receive buffer: all items plus the worst-case padding of aligned segments
inline long long recv_rows(const strata_moe_shape& s)
{
    if (s.slot_capacity > 0) return (long long)s.E * s.R * s.slot_capacity;
    const long long pad = s.segment_align > 1 ? s.segment_align - 1 : 0;
    return (long long)s.R * s.T * s.K + (long long)s.E * pad;
}

// The clauses of the shape check that the routing layout depends on (everything but H and the
// dispatch dtype): shared by context creation and by the allocation-free layout entry.
inline strata_status check_layout_shape(const strata_moe_shape& s)
{
    if (s.R <= 0 || s.T <= 0 || s.E <= 0 || s.K <= 0) return STRATA_ERR_SHAPE;
    if (s.E % s.R != 0 || s.E > kMaxExperts || s.K > kMaxTopK) return STRATA_ERR_SHAPE;
    if (s.segment_align < 0 || s.segment_align > 65536) return STRATA_ERR_SHAPE;
    if ((s.flags & ~STRATA_FLAG_ALLOW_UNROUTED) != 0) return STRATA_ERR_SHAPE;
    if (s.slot_capacity < 0 || (s.slot_capacity > 0 && s.segment_align > 1)) return STRATA_ERR_SHAPE;
    if (recv_rows(s) >= (1ll << 31) || (long long)s.R * s.T * s.K >= (1ll << 31)) return STRATA_ERR_SHAPE;
    return STRATA_OK;
}

// Dynamic work distribution.  CTAs (or warps) claim the next unit with one atomicAdd on a counter in
// the workspace; nothing ever waits.  Units are claimed in order, so the CTAs running at any moment
// work on neighbouring tokens, and a CTA that happens to get less memory bandwidth simply claims
// fewer units: measured on B200, CTAs given equal static shares finish between 50 % and 100 % of the
// kernel time (the split is even in bytes, the memory system is not even in service), and claiming
// lifts the dispatch pattern from 5.7 to 6.6 TB/s.  This is the SM-side answer to the core-level
// long tails that the paper's workload-balanced partitioning removes (Sec. 6.2).
// Every CTA stops claiming at its first failed claim, so a launch makes exactly gridDim.x failed
// claims; the CTA that draws the last of them puts the counter back to zero.  Nothing waits, nothing
// is reset from the host, and a launch replayed from a CUDA graph finds the counter as it needs it.
struct WorkQueue {
    unsigned int* next;    // device: next unclaimed unit; zero between launches
};
constexpr unsigned int kNoUnit = 0xffffffffu;

// Optional per-CTA stage probes (paper Sec. 6.4, in-kernel profiler with a per-core slice of a
// trace buffer): when a trace buffer is set on the context, every CTA of dispatch and combine
// records the global timer at its start and end into its own slot.
struct TraceBuf {
    unsigned long long* slots;   // device, [capacity][4] = {start_ns, end_ns, wait_in_ns, wait_out_ns}; nullptr = off
    int capacity;
    // event timeline: tl_ctas slices of (1 + tl_cap) words, word 0 = events recorded so far; nullptr = off
    unsigned long long* tl;
    int tl_ctas;
    int tl_cap;
};

// ---- launchers (defined next to their kernels) -----------------------------
cudaError_t launch_layout(const strata_moe_shape& s, const int32_t* ids, const strata_moe_layout_t& L,
                          int* ws_header, int* tile_cnt, cudaStream_t st, int* n_launches);
// x_early: the caller promised that x is complete before the kernel preceding dispatch in the stream starts,
// so the first rows may be loaded before that kernel has finished (see strata_ctx_set_x_early)
cudaError_t launch_dispatch_bf16(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv,
                                 size_t capacity_rows, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                                 bool x_early, cudaStream_t st);
cudaError_t launch_dispatch_fp8(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv_q,
                                float* recv_scale, size_t capacity_rows, int* status, WorkQueue wq, int n_sm,
                                TraceBuf trace, bool x_early, cudaStream_t st);
cudaError_t launch_combine(const strata_moe_shape& s, const int32_t* dst_row, const void* y, size_t y_rows,
                           const float* w, void* out, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                           cudaStream_t st);
cudaError_t launch_partition(const strata_moe_shape& s, const strata_moe_layout_t& L,
                             const strata_partition_policy& pol, int n_cores, const strata_partition_t& out,
                             size_t max_units, int* status, cudaStream_t st);
cudaError_t launch_dispatch_windows(const strata_moe_shape& s, const strata_moe_layout_t& L,
                                    const strata_partition_t& part, int n_cores, const void* x, void* recv,
                                    size_t capacity_rows, int* status, TraceBuf trace, cudaStream_t st);
cudaError_t launch_slice_copy(const void* in, void* out, unsigned long long n_slices, unsigned long long slice_bytes,
                              unsigned int inner, unsigned long long stride_a, unsigned long long stride_b, int fan,
                              unsigned long long fan_stride, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                              cudaStream_t st);
cudaError_t launch_slice_reduce(const void* in, void* out, unsigned long long n_vec, int R, int fan, WorkQueue wq,
                                int n_sm, TraceBuf trace, cudaStream_t st);
uint32_t collective_chunk_bytes();
int collective_max_v_ranks();
size_t collective_table_bytes();     // workspace tail used by all-to-all-v (a multiple of 256)
cudaError_t launch_slice_copyv(const void* in, unsigned long long in_stride, void* out, unsigned long long out_stride,
                               const long long* send_bytes, const long long* send_off, const long long* recv_off, int R,
                               void* table, int* status, WorkQueue wq, int n_sm, TraceBuf trace, cudaStream_t st);
cudaError_t launch_mask_ragged(const strata_moe_shape& s, const int32_t* tokens_per_rank, int32_t* ids, int n_sm,
                               cudaStream_t st);
cudaError_t launch_row_experts(const strata_moe_shape& s, const strata_moe_layout_t& L, int32_t* row_expert,
                               long long n_rows, cudaStream_t st);
cudaError_t launch_expert_affine(const strata_moe_shape& s, const strata_moe_layout_t& L, void* recv, long long n_rows,
                                 const float* scale, const float* bias, int tile_rows, int n_sm, cudaStream_t st);
int partition_max_units_supported();
int partition_max_cores_supported();
uint32_t windows_max_row_bytes();

#ifdef __CUDACC__
// ---- programmatic dependent launch ---------------------------------------------
// Every kernel of the library is launched with programmatic stream serialisation allowed, so its
// launch latency and its prologue overlap with the tail of the kernel before it in the stream.
// Protocol inside each kernel, in every CTA: griddep_wait() before the first access to global
// memory that the predecessor may write or still read (it returns once the preceding grid has
// completed and its writes are visible; it is a no-op without a programmatic dependency), then
// griddep_launch_dependents() so the next kernel may be scheduled (it launches once every CTA has
// triggered or exited).  Waiting first and triggering second keeps the chain transitive: a
// dependent never starts before our own predecessor has finished.  The long kernels trigger late,
// when a CTA finds the work queue empty: CTAs of the next kernel that sit in their wait for a whole
// millisecond slowed the running kernel by 10 % at the prefill shape, while a late trigger still
// hides the launch latency behind the last unit.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_plain(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.numAttrs = 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                              Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
#ifdef STRATA_NO_PDL
    cfg.numAttrs = 0;                 // build-time switch for A/B measurements: plain stream order
#else
    cfg.numAttrs = 1;
#endif
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Same, for a grid made of thread-block clusters of `cluster` CTAs (cluster == 1: no clusters).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                      unsigned cluster, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Dispatch and combine are launched as programmatic dependents too.  Measured on B200 with grids whose
// shared-memory request pins the number of CTAs per SM: the gap between the last CTA of one kernel and
// the first CTA of the next falls from 4 us to 1.3 us; the three-call step goes from 17.4 to 13.3 us for
// a 3 MB batch, from 96 to 90 us at the decode shape and from 2581 to 2570 us at the prefill shape.
// (Without the pinning, a dispatch launched as a dependent ran 20 % slower for its whole duration.)
// STRATA_PDL_MAX_MB, in tuning builds, restores plain stream order above a size for A/B measurements.
constexpr long long kPdlMaxBytes = 1ll << 50;
inline long long pdl_max_bytes() { return tune("STRATA_PDL_MAX_MB", kPdlMaxBytes >> 20) << 20; }
#define STRATA_LAUNCH_LONG(small, ...) ((small) ? launch_pdl(__VA_ARGS__) : launch_plain(__VA_ARGS__))

// ---- device helpers --------------------------------------------------------
__device__ __forceinline__ void report_status(int* status, int code)
{
    atomicCAS(status, 0, code);   // first error wins
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// One thread per CTA calls these; slot = blockIdx.x.
__device__ __forceinline__ void trace_begin(const TraceBuf& t)
{
    if (t.slots && (int)blockIdx.x < t.capacity) t.slots[4 * blockIdx.x] = global_timer_ns();
}
// wait_in / wait_out: nanoseconds the CTA's issuing thread spent blocked on incoming data and on the
// drain of outgoing data (0 where a kernel has no such stage)
__device__ __forceinline__ void trace_end(const TraceBuf& t, unsigned long long wait_in = 0,
                                          unsigned long long wait_out = 0)
{
    if (t.slots && (int)blockIdx.x < t.capacity) {
        t.slots[4 * blockIdx.x + 1] = global_timer_ns();
        t.slots[4 * blockIdx.x + 2] = wait_in;
        t.slots[4 * blockIdx.x + 3] = wait_out;
    }
}
// Stage stopwatch: costs two timer reads per use, and only while a trace buffer is set.
struct StageClock {
    bool on;
    unsigned long long t0, total;
    __device__ explicit StageClock(const TraceBuf& t) : on(t.slots != nullptr), t0(0), total(0) {}
    __device__ __forceinline__ void begin() { if (on) t0 = global_timer_ns(); }
    __device__ __forceinline__ void end() { if (on) total += global_timer_ns() - t0; }
};

// Event timeline (paper Sec. 6.4, manual probes).  One thread per CTA owns the writer; construct it
// after griddep_wait(), so that the event count left by the previous launch is visible.
struct Timeline {
    unsigned long long* slice;
    unsigned int n, cap, kernel;
    __device__ Timeline(const TraceBuf& t, unsigned int kernel_id, bool owner)
        : slice(nullptr), n(0), cap(0), kernel(kernel_id)
    {
        if (owner && t.tl && (int)blockIdx.x < t.tl_ctas) {
            slice = t.tl + (size_t)blockIdx.x * (size_t)(t.tl_cap + 1);
            n = (unsigned int)*reinterpret_cast<volatile unsigned long long*>(slice);
            cap = (unsigned int)t.tl_cap;
        }
    }
    __device__ __forceinline__ void mark(unsigned int stage, unsigned int is_end)
    {
        if (!slice) return;
        if (n < cap)
            slice[1 + n] = (global_timer_ns() & 0xffffffffffffull) | ((unsigned long long)(stage & 0xffu) << 48) |
                           ((unsigned long long)(is_end & 1u) << 56) | ((unsigned long long)(kernel & 0x7fu) << 57);
        ++n;
    }
    __device__ __forceinline__ void begin(unsigned int stage) { mark(stage, 0); }
    __device__ __forceinline__ void end(unsigned int stage) { mark(stage, 1); }
    __device__ __forceinline__ void finish()
    {
        if (slice) slice[0] = n;
    }
};

// One thread per CTA claims; returns kNoUnit when the queue is exhausted.  Units below `base` were
// dealt statically (every CTA starts on units it knows without asking: same-address atomics complete
// at roughly one per 3.5 ns, so a burst of one claim per CTA at launch would cost microseconds).
// `exhausted` is the caller's per-CTA flag: after the first failed claim the counter is left alone.
__device__ __forceinline__ unsigned int claim_unit(const WorkQueue& q, unsigned int n_units, unsigned int base,
                                                   bool& exhausted)
{
    if (base >= n_units || exhausted) return kNoUnit;        // all static, or already failed once
    const unsigned int old = atomicAdd(q.next, 1u);
    if (base + old < n_units) return base + old;
    exhausted = true;
    // failed claims are numbered n_units-base .. n_units-base+gridDim.x-1; the last one re-arms the queue
    if (old == n_units - base + gridDim.x - 1) *q.next = 0;
    return kNoUnit;
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
// Bounded wait: false if the phase did not complete within the iteration limit (each try suspends the
// thread for up to a hardware-defined time, so the default limit is seconds; test builds shorten it).
#ifndef STRATA_WAIT_LIMIT
#define STRATA_WAIT_LIMIT (1u << 22)
#endif
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity)
{
    for (uint32_t it = 0; it < (uint32_t)(STRATA_WAIT_LIMIT); ++it)
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
// the same load with an L2 eviction policy (see policy_evict_first)
__device__ __forceinline__ uint4 ld_stream16_hint(const void* p, uint64_t policy)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(policy));
    return v;
}
__device__ __forceinline__ void st_stream16(void* p, uint4 v)
{
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
#endif  // __CUDACC__

}  // namespace strata
