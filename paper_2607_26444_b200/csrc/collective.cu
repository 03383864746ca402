// Full-mesh collectives over emulated ranks (paper Sec. 6.1): an operator is a slice map (which
// byte ranges go where) plus a memory action (copy, or accumulate).  Two kernels execute every
// operator of the family; the frontends in the C-ABI layer only fill in the slice map.
//
// slice_copy_kernel   all-gather, all-to-all, broadcast.  A slice is cut into chunks of at most one
//     stage; a unit is one chunk: one bulk load global->shared, then `fan` bulk stores shared->global
//     (fan = R for all-gather and broadcast: the R pulls of one slice collapse into one read, since
//     every emulated rank lives in the same memory; fan = 1 for all-to-all).  Single-warp CTAs run
//     the SM's bulk-copy engine as a DMA program, exactly like the bf16 token dispatch; units are
//     claimed in order from a counter in the workspace.  Payloads too small to give every CTA two units
//     are latency bound: the fan copies of a chunk are then dealt to several units and the chunks shrink.
// slice_reduce_kernel reduce-scatter, all-reduce.  A thread owns one 16-byte vector (8 bf16) of the
//     output at a time: it issues up to 8 independent streaming loads (one per peer), adds them in
//     binary32 in rank order, repeats for the next 8 peers, rounds once to bf16 and writes `fan`
//     copies (fan = R for all-reduce).  The operands are accumulated on chip and each destination is
//     written by exactly one thread, so the paper's atomic write-back (needed when several cores
//     update the same memory) has nothing to protect here.  Payloads that do not fill the GPU run as
//     one-warp CTAs with up to 32 peers' loads in flight per thread (one round trip to memory).
#include "common.cuh"

namespace strata {

namespace {

// The collectives' grids are not pinned to a number of CTAs per SM, so only small ones are launched as
// programmatic dependents (a large one overlapped with its predecessor's tail can be placed unevenly).
constexpr long long kCollectivePdlMaxBytes = 16ll << 20;

constexpr int kCopyStages = 3;
constexpr uint32_t kCopyChunkBytes = 16384;
constexpr int kCopyCtasPerSm = 2;
constexpr int kReduceThreads = 128;
constexpr int kReduceUnitsPerCta = 24;    // vectors per unit shrink until a CTA can expect this many units

struct CopyParams {
    const unsigned char* in;
    unsigned char* out;
    unsigned long long slice_bytes;
    unsigned int chunk_bytes;             // <= kCopyChunkBytes, a multiple of 16
    unsigned int stage_bytes;             // chunk_bytes rounded up to 128: distance between two stages
    unsigned int chunks_per_slice;
    unsigned int fan_groups;              // the fan copies of a chunk are dealt to this many units
    unsigned int fan_per_group;
    unsigned int n_units;                 // n_slices * chunks_per_slice * fan_groups
    // destination of slice s, copy f:  out + f*fan_stride + (s / inner)*stride_a + (s % inner)*stride_b
    unsigned int inner;
    unsigned long long stride_a, stride_b;
    int fan;
    unsigned long long fan_stride;
    int* status;
    WorkQueue wq;
    TraceBuf trace;
};

__global__ void __launch_bounds__(32) slice_copy_kernel(CopyParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kCopyStages * p.stage_bytes);
    unsigned int* s_unit = reinterpret_cast<unsigned int*>(bars + kCopyStages);
    const int lane = threadIdx.x;
    const unsigned int n_units = p.n_units;

    if (lane == 0) {
        for (int s = 0; s < kCopyStages; ++s) {
            mbar_init(&bars[s], 1);
            s_unit[s] = kNoUnit;
        }
        mbar_fence_init();
    }
    __syncwarp();
    const uint64_t pol = policy_evict_first();
    griddep_wait();
    if (lane == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_SLICE_COPY, lane == 0);
    tl.begin(STRATA_STAGE_KERNEL);

    auto decode = [&](unsigned int u, unsigned int& slice, unsigned long long& off, uint32_t& bytes, int& f0) {
        const unsigned int c = u / p.fan_groups;               // chunk index over all slices
        f0 = (int)((u - c * p.fan_groups) * p.fan_per_group);
        slice = c / p.chunks_per_slice;
        off = (unsigned long long)(c - slice * p.chunks_per_slice) * p.chunk_bytes;
        const unsigned long long left = p.slice_bytes - off;
        bytes = left < p.chunk_bytes ? (uint32_t)left : p.chunk_bytes;
    };
    bool triggered = false, exhausted = false;
    const unsigned int n_static = (unsigned int)(kCopyStages - 1) * gridDim.x;
    auto issue_load = [&](long long j) {   // lane 0 only
        const int s = (int)(j % kCopyStages);
        unsigned int u;
        if (j < kCopyStages - 1) {
            u = blockIdx.x + (unsigned int)j * gridDim.x;
            if (u >= n_units) u = kNoUnit;
        } else {
            u = claim_unit(p.wq, n_units, n_static, exhausted);
        }
        s_unit[s] = u;
        if (u == kNoUnit) {
            if (!triggered) griddep_launch_dependents();
            triggered = true;
            return;
        }
        unsigned int slice;
        unsigned long long off;
        uint32_t bytes;
        int f0;
        decode(u, slice, off, bytes, f0);
        mbar_expect_tx(&bars[s], bytes);
        bulk_g2s(smem + (size_t)s * p.stage_bytes, p.in + (size_t)slice * p.slice_bytes + off, bytes, &bars[s], pol);
    };

    if (lane == 0)
        for (long long j = 0; j < kCopyStages - 1; ++j) issue_load(j);
    __syncwarp();

    bool ok = true;
    StageClock wait_in(p.trace), wait_out(p.trace);
    for (long long j = 0;; ++j) {
        const int s = (int)(j % kCopyStages);
        const uint32_t parity = (uint32_t)((j / kCopyStages) & 1);
        const unsigned int u = s_unit[s];
        if (u == kNoUnit) break;
        wait_in.begin();
        tl.begin(STRATA_STAGE_WAIT_IN);
        ok = mbar_wait_bounded(&bars[s], parity);
        tl.end(STRATA_STAGE_WAIT_IN);
        wait_in.end();
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) {
            unsigned int slice;
            unsigned long long off;
            uint32_t bytes;
            int f0;
            decode(u, slice, off, bytes, f0);
            tl.begin(STRATA_STAGE_WORK);
            unsigned char* dst = p.out + (size_t)(slice / p.inner) * p.stride_a + (size_t)(slice % p.inner) * p.stride_b + off;
            const int f1 = min(p.fan, f0 + (int)p.fan_per_group);
            for (int f = f0; f < f1; ++f) bulk_s2g(dst + (size_t)f * p.fan_stride, smem + (size_t)s * p.stage_bytes, bytes);
            bulk_commit();
            tl.end(STRATA_STAGE_WORK);
            wait_out.begin();
            tl.begin(STRATA_STAGE_WAIT_OUT);
            bulk_wait_read<1>();           // the stage refilled next held unit j-1: its stores have left shared memory
            tl.end(STRATA_STAGE_WAIT_OUT);
            wait_out.end();
            issue_load(j + kCopyStages - 1);
        }
        __syncwarp();
    }
    if (lane == 0) {
        if (!ok) report_status(p.status, STRATA_ERR_TIMEOUT);
        wait_out.begin();
        tl.begin(STRATA_STAGE_WAIT_OUT);
        bulk_wait_read<0>();
        tl.end(STRATA_STAGE_WAIT_OUT);
        wait_out.end();
        trace_end(p.trace, wait_in.total, wait_out.total);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

// ---- all-to-all-v: the slice map comes from device arrays -------------------------------------
// Per (sender, receiver) pair a byte count and two offsets, read on the GPU (no host round trip
// between the kernel that produced the counts, e.g. the routing layout, and this one).
// Kernel 1 (one CTA, one thread per pair) validates the pairs and writes a table into the workspace:
// chunks per pair as an inclusive prefix, bytes/16, absolute source and destination offsets.
// Kernel 2 (persistent single-warp CTAs, launched as a programmatic dependent for small payloads)
// brings the table into shared memory with one bulk copy and locates each claimed unit by a binary
// search of the prefix.  Pairs carry different volumes (the paper's first source of core-level long
// tails, Sec. 6.2); the units are equal-sized chunks claimed in order, so no CTA owns a heavy peer.
// (Letting every CTA build the table itself cost 14 us of prologue at 32 ranks: 296 CTAs reading the
// same 24 KB, one of the three arrays transposed.)
constexpr int kMaxVRanks = 32;
constexpr int kMaxVPairs = kMaxVRanks * kMaxVRanks;

struct VTable {                            // 24,592 bytes, a multiple of 16
    unsigned int prefix[kMaxVPairs + 4];   // prefix[i] = chunks of pairs < i; prefix[n_pairs] = all units
    unsigned int vec16[kMaxVPairs];        // bytes / 16 of the pair, 0 if empty or skipped
    unsigned long long src_abs[kMaxVPairs];
    unsigned long long dst_abs[kMaxVPairs];
};
static_assert(sizeof(VTable) % 16 == 0, "bulk-copy operand");

struct CopyVParams {
    const unsigned char* in;
    unsigned char* out;
    unsigned long long in_stride, out_stride;
    const long long* send_bytes;          // [R][R]
    const long long* send_off;            // [R][R]
    const long long* recv_off;            // [R][R], indexed [receiver][sender]
    VTable* table;                        // workspace
    int R;
    int* status;
    WorkQueue wq;
    TraceBuf trace;
};

__global__ void __launch_bounds__(kMaxVPairs) copyv_table_kernel(CopyVParams p)
{
    __shared__ unsigned int warp_sum[32];
    const int i = threadIdx.x, lane = i & 31, warp = i >> 5;
    const int n_pairs = p.R * p.R;
    griddep_wait();                        // the count and offset arrays may come from the kernel before
    griddep_launch_dependents();
    unsigned int chunks = 0, v = 0;
    unsigned long long sa = 0, da = 0;
    if (i < n_pairs) {
        const int snd = i / p.R, rcv = i - snd * p.R;
        const long long n = p.send_bytes[i], so = p.send_off[i], ro = p.recv_off[rcv * p.R + snd];
        if (n != 0) {
            if (n < 0 || so < 0 || ro < 0 || (unsigned long long)(so + n) > p.in_stride ||
                (unsigned long long)(ro + n) > p.out_stride) {
                report_status(p.status, STRATA_ERR_CAPACITY);        // pair skipped
            } else if (((n | so | ro) & 15) != 0) {
                report_status(p.status, STRATA_ERR_ALIGNMENT);       // pair skipped
            } else {
                v = (unsigned int)(n >> 4);
                chunks = (unsigned int)((n + kCopyChunkBytes - 1) / kCopyChunkBytes);
            }
        }
        sa = (unsigned long long)snd * p.in_stride + (unsigned long long)so;
        da = (unsigned long long)rcv * p.out_stride + (unsigned long long)ro;
    }
    unsigned int incl = chunks;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned int up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        unsigned int w = warp_sum[lane], wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned int up = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += up;
        }
        warp_sum[lane] = wi - w;           // exclusive over warps
    }
    __syncthreads();
    incl += warp_sum[warp];
    if (i == 0) p.table->prefix[0] = 0;
    if (i < n_pairs) {
        p.table->prefix[i + 1] = incl;
        p.table->vec16[i] = v;
        p.table->src_abs[i] = sa;
        p.table->dst_abs[i] = da;
    }
}

__global__ void __launch_bounds__(32) slice_copyv_kernel(CopyVParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const int n_pairs = p.R * p.R;
    unsigned char* stages = smem;
    VTable* tab = reinterpret_cast<VTable*>(smem + (size_t)kCopyStages * kCopyChunkBytes);
    unsigned long long* s_dst = reinterpret_cast<unsigned long long*>(tab + 1);   // [stages] destination of a stage's unit
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_dst + kCopyStages);            // [stages + 1], the last for the table
    unsigned int* s_unit = reinterpret_cast<unsigned int*>(bars + kCopyStages + 1);
    unsigned int* s_bytes = s_unit + kCopyStages;
    const int lane = threadIdx.x;

    if (lane == 0) {
        for (int s = 0; s <= kCopyStages; ++s) mbar_init(&bars[s], 1);
        for (int s = 0; s < kCopyStages; ++s) s_unit[s] = kNoUnit;
        mbar_fence_init();
    }
    __syncwarp();
    const uint64_t pol = policy_evict_first();
    griddep_wait();                        // the table kernel has completed and its writes are visible
    if (lane == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_SLICE_COPY, lane == 0);
    tl.begin(STRATA_STAGE_KERNEL);
    if (lane == 0) {
        mbar_expect_tx(&bars[kCopyStages], (uint32_t)sizeof(VTable));
        bulk_g2s(tab, p.table, (uint32_t)sizeof(VTable), &bars[kCopyStages], pol);
    }
    bool ok = mbar_wait_bounded(&bars[kCopyStages], 0);
    ok = __all_sync(0xffffffffu, ok);
    const unsigned int* prefix = tab->prefix;
    const unsigned int n_units = ok ? prefix[n_pairs] : 0u;

    int cur = 0;                            // lane 0: the pair the last located unit fell into
    auto locate = [&](unsigned int u) {     // the i with prefix[i] <= u < prefix[i + 1]
        if (u >= prefix[cur] && u < prefix[cur + 1]) return;
        int a = 0, b = n_pairs;             // invariant: prefix[a] <= u < prefix[b]
        while (b - a > 1) {
            const int m = (a + b) >> 1;
            if (prefix[m] <= u) a = m; else b = m;
        }
        cur = a;
    };
    bool triggered = false, exhausted = false;
    const unsigned int n_static = (unsigned int)(kCopyStages - 1) * gridDim.x;
    auto issue_load = [&](long long j) {   // lane 0 only
        const int s = (int)(j % kCopyStages);
        unsigned int u;
        if (j < kCopyStages - 1) {
            u = blockIdx.x + (unsigned int)j * gridDim.x;
            if (u >= n_units) u = kNoUnit;
        } else {
            u = claim_unit(p.wq, n_units, n_static, exhausted);
        }
        s_unit[s] = u;
        if (u == kNoUnit) {
            if (!triggered) griddep_launch_dependents();
            triggered = true;
            return;
        }
        locate(u);
        const unsigned long long off = (unsigned long long)(u - prefix[cur]) * kCopyChunkBytes;
        const unsigned long long left = (unsigned long long)tab->vec16[cur] * 16ull - off;
        const uint32_t bytes = left < kCopyChunkBytes ? (uint32_t)left : kCopyChunkBytes;
        s_bytes[s] = bytes;
        s_dst[s] = tab->dst_abs[cur] + off;
        mbar_expect_tx(&bars[s], bytes);
        bulk_g2s(stages + (size_t)s * kCopyChunkBytes, p.in + tab->src_abs[cur] + off, bytes, &bars[s], pol);
    };

    if (lane == 0)
        for (long long j = 0; j < kCopyStages - 1; ++j) issue_load(j);
    __syncwarp();

    for (long long j = 0; ok; ++j) {
        const int s = (int)(j % kCopyStages);
        const uint32_t parity = (uint32_t)((j / kCopyStages) & 1);
        if (s_unit[s] == kNoUnit) break;
        tl.begin(STRATA_STAGE_WAIT_IN);
        ok = mbar_wait_bounded(&bars[s], parity);
        tl.end(STRATA_STAGE_WAIT_IN);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        if (lane == 0) {
            tl.begin(STRATA_STAGE_WORK);
            bulk_s2g(p.out + s_dst[s], stages + (size_t)s * kCopyChunkBytes, s_bytes[s]);
            bulk_commit();
            tl.end(STRATA_STAGE_WORK);
            tl.begin(STRATA_STAGE_WAIT_OUT);
            bulk_wait_read<1>();
            tl.end(STRATA_STAGE_WAIT_OUT);
            issue_load(j + kCopyStages - 1);
        }
        __syncwarp();
    }
    if (lane == 0) {
        if (!ok) report_status(p.status, STRATA_ERR_TIMEOUT);
        bulk_wait_read<0>();
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

constexpr size_t kCopyVSmem = (size_t)kCopyStages * kCopyChunkBytes + sizeof(VTable) + kCopyStages * 8 +
                              (kCopyStages + 1) * 8 + 2 * kCopyStages * 4 + 16;

struct ReduceParams {
    const unsigned char* in;
    unsigned char* out;
    unsigned long long n_vec;             // 16-byte vectors of one reduced image
    unsigned long long rank_stride;       // bytes between two peers' operands
    int R;
    int fan;                              // copies of the result
    unsigned long long fan_stride;
    unsigned int n_units;
    unsigned int vec_per_unit;            // a multiple of the CTA size (128 threads; 32 for latency-bound sizes)
    WorkQueue wq;
    TraceBuf trace;
};

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

__device__ __forceinline__ void add8(float (&a)[8], const uint4& d)
{
    a[0] = __fadd_rn(a[0], __uint_as_float(d.x << 16));
    a[1] = __fadd_rn(a[1], __uint_as_float(d.x & 0xffff0000u));
    a[2] = __fadd_rn(a[2], __uint_as_float(d.y << 16));
    a[3] = __fadd_rn(a[3], __uint_as_float(d.y & 0xffff0000u));
    a[4] = __fadd_rn(a[4], __uint_as_float(d.z << 16));
    a[5] = __fadd_rn(a[5], __uint_as_float(d.z & 0xffff0000u));
    a[6] = __fadd_rn(a[6], __uint_as_float(d.w << 16));
    a[7] = __fadd_rn(a[7], __uint_as_float(d.w & 0xffff0000u));
}

// B = peers whose operands a thread has in flight at once.  8 keeps 9 CTAs per SM for payloads that are
// bandwidth bound; 32 serves a whole 32-rank reduction with one round trip to memory, for payloads so small
// that the grid does not fill the GPU and the time is the latency of dependent loads.
template <int B>
__global__ void __launch_bounds__(kReduceThreads) slice_reduce_kernel(ReduceParams p)
{
    const int tid = threadIdx.x;
    __shared__ unsigned int s_next[2];
    griddep_wait();
    if (tid == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_SLICE_REDUCE, tid == 0);
    tl.begin(STRATA_STAGE_KERNEL);

    unsigned int u = blockIdx.x < p.n_units ? blockIdx.x : kNoUnit;
    bool exhausted = false;
    for (int j = 0; u != kNoUnit; ++j) {
        tl.begin(STRATA_STAGE_WORK);
        if (tid == 0) {
            const unsigned int nx = claim_unit(p.wq, p.n_units, gridDim.x, exhausted);
            s_next[j & 1] = nx;
            if (nx == kNoUnit) griddep_launch_dependents();
        }
        const unsigned long long v_begin = (unsigned long long)u * p.vec_per_unit;
        const unsigned long long v_end = min(v_begin + p.vec_per_unit, p.n_vec);
        for (unsigned long long v = v_begin + tid; v < v_end; v += blockDim.x) {
            const unsigned char* src = p.in + (size_t)v * 16;
            float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int p0 = 0; p0 < p.R; p0 += B) {
                uint4 d[B];
#pragma unroll
                for (int k = 0; k < B; ++k)
                    d[k] = (p0 + k < p.R) ? ld_stream16(src + (size_t)(p0 + k) * p.rank_stride) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int k = 0; k < B; ++k)
                    if (p0 + k < p.R) add8(a, d[k]);
            }
            uint4 o;
            o.x = pack2_bf16(a[0], a[1]);
            o.y = pack2_bf16(a[2], a[3]);
            o.z = pack2_bf16(a[4], a[5]);
            o.w = pack2_bf16(a[6], a[7]);
            unsigned char* dst = p.out + (size_t)v * 16;
            for (int f = 0; f < p.fan; ++f) st_stream16(dst + (size_t)f * p.fan_stride, o);
        }
        __syncthreads();
        tl.end(STRATA_STAGE_WORK);
        u = s_next[j & 1];
    }
    if (tid == 0) {
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

constexpr size_t kCopySmem = (size_t)kCopyStages * kCopyChunkBytes + kCopyStages * sizeof(uint64_t) + kCopyStages * sizeof(unsigned int) + 16;

}  // namespace

cudaError_t configure_collective_kernels()
{
    cudaError_t err = cudaFuncSetAttribute(slice_copy_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCopySmem);
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(slice_copyv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCopyVSmem);
}

int collective_max_v_ranks() { return kMaxVRanks; }
size_t collective_table_bytes() { return (sizeof(VTable) + 255) & ~(size_t)255; }

cudaError_t launch_slice_copyv(const void* in, unsigned long long in_stride, void* out, unsigned long long out_stride,
                               const long long* send_bytes, const long long* send_off, const long long* recv_off, int R,
                               void* table, int* status, WorkQueue wq, int n_sm, TraceBuf trace, cudaStream_t st)
{
    CopyVParams p{};
    p.in = static_cast<const unsigned char*>(in);
    p.out = static_cast<unsigned char*>(out);
    p.in_stride = in_stride;
    p.out_stride = out_stride;
    p.send_bytes = send_bytes;
    p.send_off = send_off;
    p.recv_off = recv_off;
    p.table = static_cast<VTable*>(table);
    p.R = R;
    p.status = status;
    p.wq = wq;
    p.trace = trace;
    cudaError_t err = launch_pdl(copyv_table_kernel, 1u, (unsigned)kMaxVPairs, 0, st, p);
    if (err != cudaSuccess) return err;
    // the number of units is known only on the device: a full persistent grid, CTAs without work leave at once
    const bool small = (long long)R * (long long)(in_stride + out_stride) < kCollectivePdlMaxBytes;
    return STRATA_LAUNCH_LONG(small, slice_copyv_kernel, (unsigned)(n_sm * kCopyCtasPerSm), 32, kCopyVSmem, st, p);
}

uint32_t collective_chunk_bytes() { return kCopyChunkBytes; }

cudaError_t launch_slice_copy(const void* in, void* out, unsigned long long n_slices, unsigned long long slice_bytes,
                              unsigned int inner, unsigned long long stride_a, unsigned long long stride_b, int fan,
                              unsigned long long fan_stride, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                              cudaStream_t st)
{
    CopyParams p{};
    p.in = static_cast<const unsigned char*>(in);
    p.out = static_cast<unsigned char*>(out);
    p.slice_bytes = slice_bytes;
    // Large payloads: 16 KB chunks, all fan copies of a chunk from one load, two CTAs per SM.  When that
    // leaves the grid short of units the call is latency bound (a unit's copies are issued by one thread,
    // a CTA takes its units one after the other): first the fan copies of a chunk are dealt to several
    // units (each re-reads the chunk, an L2 hit), then the chunks shrink, down to 2 KB, until there are
    // four units per SM; the stages shrink with the chunks, so that up to eight CTAs fit an SM and every
    // CTA gets one unit.
    const unsigned long long want_big = 2ull * (unsigned long long)n_sm * kCopyCtasPerSm;
    const unsigned long long want_small = 4ull * (unsigned long long)n_sm;   // 4, 6, 8, 16 tried: 4 and 6 tie, more is slower
    unsigned long long chunk = kCopyChunkBytes, fpg = (unsigned long long)fan;
    auto units = [&]() {
        return n_slices * ((slice_bytes + chunk - 1) / chunk) * (((unsigned long long)fan + fpg - 1) / fpg);
    };
    const bool latency_bound = units() < want_big;
    while (latency_bound && units() < want_small) {
        if (fpg > 1) fpg = (fpg + 1) / 2;
        else if (chunk > 2048) chunk /= 2;
        else break;
    }
    p.chunk_bytes = (unsigned int)chunk;
    p.stage_bytes = (unsigned int)((min(chunk, slice_bytes) + 127) / 128 * 128);
    p.chunks_per_slice = (unsigned int)((slice_bytes + chunk - 1) / chunk);
    p.fan_per_group = (unsigned int)fpg;
    p.fan_groups = (unsigned int)(((unsigned long long)fan + fpg - 1) / fpg);
    p.n_units = (unsigned int)units();
    p.inner = inner;
    p.stride_a = stride_a;
    p.stride_b = stride_b;
    p.fan = fan;
    p.fan_stride = fan_stride;
    p.status = status;
    p.wq = wq;
    p.trace = trace;
    const size_t smem = (size_t)kCopyStages * p.stage_bytes + kCopyStages * sizeof(uint64_t) +
                        kCopyStages * sizeof(unsigned int) + 16;
    long long max_grid = (long long)n_sm * kCopyCtasPerSm;
    if (latency_bound) {
        int per_sm = 0;
        cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, slice_copy_kernel, 32, smem);
        if (err != cudaSuccess) return err;
        max_grid = (long long)n_sm * max(kCopyCtasPerSm, min(per_sm, 8));
    }
    const unsigned grid = (unsigned)max(1ll, min(max_grid, (long long)p.n_units));
    const bool small = (long long)(n_slices * slice_bytes) * (fan + 1) < kCollectivePdlMaxBytes;
    return STRATA_LAUNCH_LONG(small, slice_copy_kernel, grid, 32, smem, st, p);
}

cudaError_t launch_slice_reduce(const void* in, void* out, unsigned long long n_vec, int R, int fan,
                                WorkQueue wq, int n_sm, TraceBuf trace, cudaStream_t st)
{
    ReduceParams p{};
    p.in = static_cast<const unsigned char*>(in);
    p.out = static_cast<unsigned char*>(out);
    p.n_vec = n_vec;
    p.rank_stride = n_vec * 16ull;
    p.R = R;
    p.fan = fan;
    p.fan_stride = n_vec * 16ull;
    p.wq = wq;
    p.trace = trace;
    const bool small = (long long)(n_vec * 16ull) * (R + fan) < kCollectivePdlMaxBytes;
    if (R > 8 && n_vec <= (unsigned long long)n_sm * 2u * kReduceThreads) {
        // latency bound: one-warp CTAs so that more SMs take part, the deepest batch of loads
        p.vec_per_unit = 32;
        p.n_units = (unsigned int)((n_vec + 31) / 32);
        return STRATA_LAUNCH_LONG(small, slice_reduce_kernel<32>, p.n_units, 32, 0, st, p);
    }
    int per_sm = 0;
    cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, slice_reduce_kernel<8>, kReduceThreads, 0);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const long long max_grid = (long long)n_sm * per_sm;
    unsigned int m = 4;                   // vectors per thread per unit
    while (m > 1 && (long long)((n_vec + (unsigned long long)m * kReduceThreads - 1) / ((unsigned long long)m * kReduceThreads)) <
                        kReduceUnitsPerCta * max_grid)
        m >>= 1;
    p.vec_per_unit = m * kReduceThreads;
    p.n_units = (unsigned int)((n_vec + p.vec_per_unit - 1) / p.vec_per_unit);
    const unsigned grid = (unsigned)max(1ll, min(max_grid, (long long)p.n_units));
    return STRATA_LAUNCH_LONG(small, slice_reduce_kernel<8>, grid, kReduceThreads, 0, st, p);
}

}  // namespace strata
