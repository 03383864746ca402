// Token dispatch (paper Sec. 6.2 / 8.1): every token's hidden vector goes to the K receive rows
// the layout assigned, straight into the caller's (registered) receive buffer.
//
// Work split: a unit is one token (or one column chunk of a token when a row is larger than
// a stage): 1 row read + K row writes whatever the expert popularity is.  A persistent grid claims
// units in order from a counter in the workspace, a ring's depth ahead of the one being stored, so
// CTAs running together work on neighbouring rows and no CTA is left with a fixed share it cannot
// finish in time.  Under the caller's promise that x is complete before the preceding kernel starts
// (strata_ctx_set_x_early) the first ring of rows is loaded before the wait on that kernel.
//
// bf16: each CTA is a single warp that runs the SM's bulk-copy engine as a small DMA program
//       (the on-SM counterpart of the paper's device-issued SDMA descriptors, Sec. 6.3):
//       bulk load global->shared into a ring of stages, completion on an mbarrier, then K bulk
//       stores shared->global.  No register or ALU touches the payload.
// fp8:  128-thread CTAs; the row lands in shared memory the same way, the threads compute
//       the per-128-column amax, scale = amax/448 and the e4m3 codes into an output stage,
//       and K bulk stores ship the codes; the scales (H/128 floats per row) go out with plain
//       coalesced stores.
#include <mutex>

#include "common.cuh"

#ifdef STRATA_TEST_HOOKS
#include <atomic>
#endif

namespace strata {

namespace {

#ifdef STRATA_TEST_HOOKS
// Test builds only: the next dispatch launch makes CTA 0 expect 16 bytes more than its first copy delivers,
// so that its bounded wait runs out and the error path (status word, recovery by strata_device_status) runs
// without any fault, trap or unbounded spin.
std::atomic<int> g_inject_short_copy{0};
#endif

// Launch shape, measured on B200 (kernel time from the first CTA's start to the last CTA's end):
//  - What bounds the kernel is HBM serving a 1:8 read:write mix; a variant that moved the payload through
//    registers (16-byte loads, K 16-byte stores) was 12 % slower than the copy engine.
//  - 14 KB rows (decode and prefill shapes): one CTA per SM with an 8-stage ring beats two CTAs per SM with
//    3 stages (decode 40.9 vs 42.7 us; prefill 1281 vs 1288 us).  Rings of 10 and 12 stages copy as fast
//    alone but make the layout+dispatch+combine step at the prefill shape 0.5 % and 1.5 % slower.
//  - 8 KB rows (skew shape): one issuing lane per SM cannot keep the copy engine fed (257 vs 183 us); the
//    number of CTAs per SM follows the unit size (see launch_dispatch_bf16).
//  - Cutting the last units of the batch into halves or quarters evens out the CTAs' finish times (8 us
//    apart to 2 us apart at the decode shape) but does not shorten the kernel: the CTAs that are still
//    running get the bandwidth of those that have left.  Pieces below 4 KB copy markedly slower.
//  - The issuing lane is not the limiter.  A version that took its three memory round trips per unit off its
//    path (destination rows loaded one unit early, the claim's result first read one iteration later, more
//    store groups left in flight) issued faster but in bursts: the copy engine pushed back for 1..2 us at a
//    time, the units per CTA spread from 13..15 to 12..17, and the kernel ran 1..2 us longer.
//  - The shared-memory request is padded so that exactly the intended number of CTAs fits an SM (see
//    smem_for_residency): without it a launch overlapped with its predecessor's tail is placed unevenly.
#ifndef STRATA_BF16_STAGES
#define STRATA_BF16_STAGES 3
#endif
#ifndef STRATA_BF16_CHUNK_BYTES
#define STRATA_BF16_CHUNK_BYTES 16384
#endif
constexpr uint32_t kMaxChunkBytes = STRATA_BF16_CHUNK_BYTES;   // one stage of the bf16 ring
constexpr int kBf16Stages = STRATA_BF16_STAGES;
constexpr size_t kBf16MaxSmem = 200 * 1024;  // ring + barriers of one CTA never exceed this
constexpr long long kDeepRingMinUnitBytes = 100 * 1024;   // units (1 + K chunks) at least this long, made of chunks of at
constexpr uint32_t kDeepRingMinChunkBytes = 12 * 1024;    // least this size, take the one-CTA-per-SM shape (8 KB rows with
                                                          // top-12 make a 106 KB unit but 13 copies per unit: one lane
                                                          // per SM reached 5.2 TB/s there, two reach 6.5)
constexpr long long kUnitBytesInFlightPerSm = 144 * 1024; // what the short-ring CTAs of an SM should have in flight together
constexpr size_t kShortRingsBytesPerSm = 192 * 1024;      // shared memory their rings may take together
constexpr int kMaxCtasPerSm = 24;
constexpr size_t kDeepRingBytes = 128 * 1024;         // its ring: as many stages as fit here, at most
constexpr int kDeepRingMaxStages = 8;                 // this many
// Receive buffers far larger than L2 (126 MB) are written with an L2 evict-first policy: the kernel itself runs
// the same, but the kernel that reads the buffer next does not start on an L2 full of normal-priority dirty
// lines.  Measured: combine right after dispatch 1,270 -> 1,228 us at the prefill shape (7.5 GB); at the skew
// shape (1.1 GB) neutral; at the decode shape (235 MB) combine loses 3 us, because half of what it reads would
// still have been in L2.
constexpr long long kStoreHintMinBytes = 2ll << 30;
// 64..256 threads and 2048..4096-column chunks land within 1.5 % of each other (110..113 us at the fp8 shape);
// 1024-column chunks are 25 % slower.  Requesting the work claim one unit early (so that the CTA does not sit
// between two barriers during the atomic's round trip) helps small units a little (top-2: 4.2 -> 4.3 TB/s) and
// costs 2 % at the fp8 shape and with 7,168 columns: not taken, as in the bf16 kernel.
constexpr int kFp8Threads = 128;
constexpr int kFp8MaxChunkCols = 4096;       // 8 KB in, 4 KB out per stage

struct DispatchParams {
    const int32_t* dst_row;
    const unsigned char* x;
    unsigned char* recv;
    float* recv_scale;
    long long n_units;          // n_tok * chunks_per_row
    long long capacity_rows;
    int K;
    int H;
    int chunks_per_row;
    uint32_t chunk_cols;        // columns per chunk (last chunk of a row may be shorter)
    int stages;                 // bf16 only: depth of the ring in shared memory
    int test_flags;             // always 0 in the shipped library
    int x_early;                // the first loads of x may go out before the preceding kernel has finished
    int store_hint;             // bf16 only: the bulk stores carry an L2 evict-first policy
    int* status;
    WorkQueue wq;
    TraceBuf trace;
};

__global__ void __launch_bounds__(32) dispatch_bf16_kernel(DispatchParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t stage_bytes = p.chunk_cols * 2u;
    const int n_stages = p.stages;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)n_stages * stage_bytes);
    unsigned int* s_unit = reinterpret_cast<unsigned int*>(bars + n_stages);   // unit held by each stage
    const int lane = threadIdx.x;
    const size_t row_bytes = (size_t)p.H * 2u;
    const unsigned int n_units = (unsigned int)p.n_units;

    if (lane == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&bars[s], 1);
            s_unit[s] = kNoUnit;
        }
        mbar_fence_init();
    }
    __syncwarp();
    const uint64_t pol = policy_evict_first();

    auto decode = [&](unsigned int u, long long& tok, uint32_t& col0, uint32_t& bytes) {
        tok = u / (unsigned int)p.chunks_per_row;
        const uint32_t ch = u - (unsigned int)tok * (unsigned int)p.chunks_per_row;
        col0 = ch * p.chunk_cols;
        bytes = min(p.chunk_cols, (uint32_t)p.H - col0) * 2u;
    };
    bool triggered = false, exhausted = false, waited = false;
    // The first stages-1 units of a CTA are fixed (blockIdx + j*grid); the rest are claimed.
    const unsigned int n_static = (unsigned int)(n_stages - 1) * gridDim.x;
    auto issue_load = [&](long long j) {   // lane 0 only: next unit into stage j % stages
        const int s = (int)(j % n_stages);
        unsigned int u;
        if (j < n_stages - 1) {
            u = blockIdx.x + (unsigned int)j * gridDim.x;
            if (u >= n_units) u = kNoUnit;
        } else {
            u = claim_unit(p.wq, n_units, n_static, exhausted);
        }
        s_unit[s] = u;
        if (u == kNoUnit) {
            // queue empty: the next kernel may be scheduled (never before this kernel's own wait: a dependent
            // must not start before our predecessor has finished)
            if (waited && !triggered) {
                griddep_launch_dependents();
                triggered = true;
            }
            return;
        }
        long long tok;
        uint32_t col0, bytes;
        decode(u, tok, col0, bytes);
        uint32_t expect = bytes;
#ifdef STRATA_TEST_HOOKS
        if ((p.test_flags & 1) && blockIdx.x == 0 && j == 0) expect += 16;
#endif
        mbar_expect_tx(&bars[s], expect);
        bulk_g2s(smem + (size_t)s * stage_bytes, p.x + (size_t)tok * row_bytes + (size_t)col0 * 2u, bytes, &bars[s],
                 pol);
    };

    // The first stages-1 units are fixed, so their loads need nothing from the layout: when the caller has
    // promised that x was complete before the preceding kernel started, they go out before the wait and are
    // in shared memory by the time the layout is done.  dst_row and the claim counter are touched after it.
    if (p.x_early && lane == 0)
        for (long long j = 0; j < n_stages - 1; ++j) issue_load(j);
    griddep_wait();                       // dst_row (and, without the promise, x) belong to earlier kernels in the stream
    if (lane == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_DISPATCH_BF16, lane == 0);
    tl.begin(STRATA_STAGE_KERNEL);
    waited = true;
    if (lane == 0) {
        if (!p.x_early)
            for (long long j = 0; j < n_stages - 1; ++j) issue_load(j);
        else if (s_unit[(n_stages - 2) % n_stages] == kNoUnit) {   // fewer fixed units than stages: nothing left to claim
            griddep_launch_dependents();
            triggered = true;
        }
    }
    __syncwarp();

    bool ok = true;
    StageClock wait_in(p.trace), wait_out(p.trace);
    long long j = 0;
    for (;; ++j) {
        const int s = (int)(j % n_stages);
        const uint32_t parity = (uint32_t)((j / n_stages) & 1);
        const unsigned int u = s_unit[s];
        if (u == kNoUnit) break;          // claims fail in order: nothing is in flight behind this stage
        long long tok;
        uint32_t col0, bytes;
        decode(u, tok, col0, bytes);

        const int my_row = (lane < p.K) ? p.dst_row[tok * p.K + lane] : -1;
        const bool row_ok = (lane >= p.K) || (my_row >= 0 && my_row < p.capacity_rows);
        if (!row_ok && my_row != -1) report_status(p.status, STRATA_ERR_BAD_ROW);

        wait_in.begin();
        tl.begin(STRATA_STAGE_WAIT_IN);
        ok = mbar_wait_bounded(&bars[s], parity);
        tl.end(STRATA_STAGE_WAIT_IN);
        wait_in.end();
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;

        tl.begin(STRATA_STAGE_WORK);
        for (int k = 0; k < p.K; ++k) {
            const int row = __shfl_sync(0xffffffffu, my_row, k);
            if (lane == 0 && row >= 0 && row < p.capacity_rows) {
                if (p.store_hint)
                    bulk_s2g_hint(p.recv + (size_t)row * row_bytes + (size_t)col0 * 2u, smem + (size_t)s * stage_bytes,
                                  bytes, pol);
                else
                    bulk_s2g(p.recv + (size_t)row * row_bytes + (size_t)col0 * 2u, smem + (size_t)s * stage_bytes, bytes);
            }
        }
        if (lane == 0) {
            bulk_commit();
            tl.end(STRATA_STAGE_WORK);
            // The stage that unit j-1 used is refilled next; its stores must have left shared memory.
            wait_out.begin();
            tl.begin(STRATA_STAGE_WAIT_OUT);
            bulk_wait_read<1>();
            tl.end(STRATA_STAGE_WAIT_OUT);
            wait_out.end();
            issue_load(j + n_stages - 1);
        }
        __syncwarp();
    }
    if (!ok) {
        // A wait ran out.  The loads issued behind the unit that gave up may still be on their way: wait for
        // them, again with a limit, so that nothing is written into this CTA's shared memory after it has left.
        for (long long jj = j + 1; jj < j + n_stages - 1; ++jj) {
            const int s2 = (int)(jj % n_stages);
            if (s_unit[s2] != kNoUnit) mbar_wait_bounded(&bars[s2], (uint32_t)((jj / n_stages) & 1));
        }
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

// ---- fp8 -------------------------------------------------------------------------

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// e4m3 (OCP "fn"), round to nearest even, saturating to +-448; `hi` lands in the upper byte.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi, float lo)
{
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

__global__ void __launch_bounds__(kFp8Threads) dispatch_fp8_kernel(DispatchParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t in_bytes = p.chunk_cols * 2u, out_bytes = p.chunk_cols;
    auto in_stage = [&](int s) { return smem + (size_t)s * in_bytes; };
    auto out_stage = [&](int s) { return smem + 2 * (size_t)in_bytes + (size_t)s * out_bytes; };
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * in_bytes + 2 * out_bytes);
    const int tid = threadIdx.x, lane = tid & 31;
    const size_t in_row_bytes = (size_t)p.H * 2u, out_row_bytes = (size_t)p.H;
    const int nb_row = p.H / 128;
    const unsigned int n_units = (unsigned int)p.n_units;

    __shared__ unsigned int s_unit[2];     // unit held by each input stage
    __shared__ int s_rows[kMaxTopK];
    __shared__ float s_scale[kFp8MaxChunkCols / 128];

    if (tid == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        mbar_fence_init();
    }
    __syncthreads();
    const uint64_t pol = policy_evict_first();

    auto decode = [&](unsigned int u, long long& tok, uint32_t& col0, uint32_t& cols) {
        tok = u / (unsigned int)p.chunks_per_row;
        const uint32_t ch = u - (unsigned int)tok * (unsigned int)p.chunks_per_row;
        col0 = ch * p.chunk_cols;
        cols = min(p.chunk_cols, (uint32_t)p.H - col0);
    };
    bool triggered = false, exhausted = false, waited = false;
    const unsigned int n_static = 2u * gridDim.x;   // the first two units of a CTA are fixed
    auto issue_load = [&](long long j) {   // thread 0 only
        const int s = (int)(j & 1);
        unsigned int u;
        if (j < 2) {
            u = blockIdx.x + (unsigned int)j * gridDim.x;
            if (u >= n_units) u = kNoUnit;
        } else {
            u = claim_unit(p.wq, n_units, n_static, exhausted);
        }
        s_unit[s] = u;
        if (u == kNoUnit) {
            if (waited && !triggered) {                    // queue empty: the next kernel may be scheduled
                griddep_launch_dependents();
                triggered = true;
            }
            return;
        }
        long long tok;
        uint32_t col0, cols;
        decode(u, tok, col0, cols);
        uint32_t expect = cols * 2u;
#ifdef STRATA_TEST_HOOKS
        if ((p.test_flags & 1) && blockIdx.x == 0 && j == 0) expect += 16;
#endif
        mbar_expect_tx(&bars[s], expect);
        bulk_g2s(in_stage(s), p.x + (size_t)tok * in_row_bytes + (size_t)col0 * 2u, cols * 2u, &bars[s], pol);
    };
    if (p.x_early && tid == 0) {          // the two fixed units need nothing from the layout (see the bf16 kernel)
        issue_load(0);
        issue_load(1);
    }
    griddep_wait();
    if (tid == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_DISPATCH_FP8, tid == 0);
    tl.begin(STRATA_STAGE_KERNEL);
    waited = true;
    if (tid == 0) {
        if (!p.x_early) {
            issue_load(0);
            issue_load(1);
        } else if (s_unit[1] == kNoUnit) {
            griddep_launch_dependents();
            triggered = true;
        }
    }
    __syncthreads();

    bool ok = true;
    long long j = 0;
    for (;; ++j) {
        const int s = (int)(j & 1);
        const uint32_t parity = (uint32_t)((j >> 1) & 1);
        const unsigned int u = s_unit[s];
        if (u == kNoUnit) break;
        long long tok;
        uint32_t col0, cols;
        decode(u, tok, col0, cols);

        if (tid < p.K) {
            const int row = p.dst_row[tok * p.K + tid];
            const bool row_ok = row >= 0 && row < p.capacity_rows;
            if (!row_ok && row != -1) report_status(p.status, STRATA_ERR_BAD_ROW);
            s_rows[tid] = row_ok ? row : -1;
        }
        if (tid == 0) {
            tl.begin(STRATA_STAGE_WAIT_OUT);
            bulk_wait_read<1>();               // stores of unit j-2 have left out_stage(s)
            tl.end(STRATA_STAGE_WAIT_OUT);
        }
        tl.begin(STRATA_STAGE_WAIT_IN);
        ok = mbar_wait_bounded(&bars[s], parity);
        ok = __syncthreads_and(ok);
        tl.end(STRATA_STAGE_WAIT_IN);
        if (!ok) break;
        tl.begin(STRATA_STAGE_WORK);

        const uint4* in = reinterpret_cast<const uint4*>(in_stage(s));
        uint2* outq = reinterpret_cast<uint2*>(out_stage(s));
        const uint32_t nvec = cols / 8;        // multiple of 16
        for (uint32_t v0 = (uint32_t)(tid - lane); v0 < nvec; v0 += kFp8Threads) {
            const uint32_t v = v0 + lane;
            const bool act = v < nvec;
            uint4 d = act ? in[v] : make_uint4(0, 0, 0, 0);
            float f[8] = {bf16lo(d.x), bf16hi(d.x), bf16lo(d.y), bf16hi(d.y),
                          bf16lo(d.z), bf16hi(d.z), bf16lo(d.w), bf16hi(d.w)};
            float amax = 0.0f;
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(f[i]));
#pragma unroll
            for (int m = 8; m >= 1; m >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
            const float scale = __fdiv_rn(amax, 448.0f);
            const float dv = (amax == 0.0f) ? 1.0f : scale;
            float q[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) q[i] = __fdiv_rn(f[i], dv);
            uint2 o;
            o.x = cvt_e4m3x2(q[1], q[0]) | (cvt_e4m3x2(q[3], q[2]) << 16);
            o.y = cvt_e4m3x2(q[5], q[4]) | (cvt_e4m3x2(q[7], q[6]) << 16);
            if (act) {
                outq[v] = o;
                if ((lane & 15) == 0) s_scale[v >> 4] = scale;
            }
        }
        fence_async_smem();
        __syncthreads();
        {   // scales: K rows x (cols/128) floats, coalesced along the row
            const int nb = (int)(cols >> 7);
            for (int idx = tid; idx < p.K * nb; idx += kFp8Threads) {
                const int k = idx / nb, b = idx - k * nb;
                const int row = s_rows[k];
                if (row >= 0) p.recv_scale[(size_t)row * nb_row + (col0 >> 7) + b] = s_scale[b];
            }
        }
        if (tid == 0) {
            for (int k = 0; k < p.K; ++k) {
                const int row = s_rows[k];
                if (row >= 0) bulk_s2g(p.recv + (size_t)row * out_row_bytes + col0, out_stage(s), cols);
            }
            bulk_commit();
            issue_load(j + 2);                      // in_stage(s) was fully consumed before the barrier above
        }
        __syncthreads();                            // s_rows, s_scale and s_unit[s] are rewritten next
        tl.end(STRATA_STAGE_WORK);
    }
    if (!ok && s_unit[(j + 1) & 1] != kNoUnit)      // the other stage's load may still be on its way
        mbar_wait_bounded(&bars[(j + 1) & 1], (uint32_t)(((j + 1) >> 1) & 1));
    if (tid == 0) {
        if (!ok) report_status(p.status, STRATA_ERR_TIMEOUT);
        bulk_wait_read<0>();
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

// Shared memory to request so that exactly `want` CTAs of `kernel` fit on an SM (fewer if `need` is too
// large for that).  The persistent grids have want * n_sm CTAs and assume `want` on every SM.  When such a
// grid is launched as a programmatic dependent, its CTAs are placed while the preceding kernel still
// holds part of some SMs; if more than `want` fitted on an SM, the free SMs would take several CTAs and
// others none, and the kernel would run with a lopsided placement for its whole life (measured: 20 %
// slower at the prefill shape).  Asking for more shared memory than needed makes the surplus CTA not fit.
// The answer depends only on (device, kernel, threads, need, want), and a context asks the same question on
// every call: the last few answers are kept, so a call costs a lock instead of four runtime queries.
struct ResidencyAnswer {
    const void* kernel;
    int dev, threads, want;
    size_t need, max_smem, smem;
    int per_sm;
};
std::mutex g_residency_mu;
ResidencyAnswer g_residency[8];
int g_residency_n = 0, g_residency_next = 0;

template <typename Kernel>
cudaError_t smem_for_residency(Kernel kernel, int threads, size_t need, int want, size_t max_smem, size_t* smem_out,
                               int* per_sm_out)
{
    int dev = 0, sm_total = 0, reserved = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const void* kptr = reinterpret_cast<const void*>(kernel);
    {
        std::lock_guard<std::mutex> lk(g_residency_mu);
        for (int i = 0; i < g_residency_n; ++i) {
            const ResidencyAnswer& a = g_residency[i];
            if (a.kernel == kptr && a.dev == dev && a.threads == threads && a.want == want && a.need == need &&
                a.max_smem == max_smem) {
                *smem_out = a.smem;
                *per_sm_out = a.per_sm;
                return cudaSuccess;
            }
        }
    }
    err = cudaDeviceGetAttribute(&sm_total, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev);
    if (err != cudaSuccess) return err;
    err = cudaDeviceGetAttribute(&reserved, cudaDevAttrReservedSharedMemoryPerBlock, dev);
    if (err != cudaSuccess) return err;
    if (want < 1) want = 1;
    // want + 1 CTAs must not fit: (want + 1) * (smem + reserved) > sm_total
    size_t excl = (size_t)sm_total / (size_t)(want + 1) + 1;
    excl = excl > (size_t)reserved ? excl - (size_t)reserved : 0;
    size_t smem = max(need, (excl + 127) & ~(size_t)127);
    if (smem > max_smem) smem = max(need, max_smem);
    int per_sm = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem);
    if (err != cudaSuccess) return err;
    *smem_out = smem;
    *per_sm_out = max(1, min(per_sm, want));
    {
        std::lock_guard<std::mutex> lk(g_residency_mu);
        g_residency[g_residency_next] = ResidencyAnswer{kptr, dev, threads, want, need, max_smem, *smem_out, *per_sm_out};
        g_residency_next = (g_residency_next + 1) % 8;
        if (g_residency_n < 8) ++g_residency_n;
    }
    return cudaSuccess;
}

uint32_t pick_chunk_cols_bf16(int H, uint32_t max_chunk_bytes)
{
    const uint32_t row_bytes = (uint32_t)H * 2u;
    if (row_bytes <= max_chunk_bytes) return (uint32_t)H;
    const uint32_t n = (row_bytes + max_chunk_bytes - 1) / max_chunk_bytes;
    uint32_t cols = ((uint32_t)H + n - 1) / n;
    cols = (cols + 7u) & ~7u;        // chunks start on 16-byte boundaries
    return cols;
}

}  // namespace

cudaError_t configure_dispatch_kernels()
{
    cudaError_t err = cudaFuncSetAttribute(dispatch_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)kBf16MaxSmem);
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(dispatch_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBf16MaxSmem);
}

cudaError_t launch_dispatch_bf16(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv,
                                 size_t capacity_rows, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                                 bool x_early, cudaStream_t st)
{
    DispatchParams p{};
    p.x_early = x_early ? 1 : 0;
    p.trace = trace;
    p.wq = wq;
    p.dst_row = dst_row;
    p.x = static_cast<const unsigned char*>(x);
    p.recv = static_cast<unsigned char*>(recv);
    p.recv_scale = nullptr;
    p.K = s.K;
    p.H = s.H;
    p.chunk_cols = pick_chunk_cols_bf16(s.H, (uint32_t)tune("STRATA_DISP_CHUNK", kMaxChunkBytes));
    p.chunks_per_row = (int)(((uint32_t)s.H + p.chunk_cols - 1) / p.chunk_cols);
    p.capacity_rows = (long long)capacity_rows;
    p.status = status;
    // A unit (one chunk read, K chunk writes) occupies its issuing lane for about 2.5 us whatever its size
    // (destination rows, claim and stage hand-over are round trips to memory), so an SM needs enough lanes
    // working side by side to move its share of the bandwidth: about 144 KB of units in flight per SM.  Units of
    // 100 KB and more (14 KB rows with top-8) get one CTA per SM with a deep ring; smaller units get
    // ceil(144 KB / unit) CTAs per SM with a short ring each (measured at 16,384 tokens, top-8: 2 KB rows 2.3 ->
    // 6.1 TB/s with 8 CTAs per SM, 4 KB rows 4.3 -> 6.4 TB/s with 4; top-2, 4 KB rows 2.1 -> 6.1 TB/s with 12).
    const uint32_t stage_bytes = p.chunk_cols * 2u;
    const long long unit_bytes = (long long)(s.K + 1) * stage_bytes;
    const bool deep = unit_bytes >= kDeepRingMinUnitBytes && stage_bytes >= kDeepRingMinChunkBytes;
    int lanes = (int)((kUnitBytesInFlightPerSm + unit_bytes - 1) / unit_bytes);
    lanes = max(2, min(kMaxCtasPerSm, min(lanes, (int)(kShortRingsBytesPerSm / ((size_t)kBf16Stages * stage_bytes)))));
    int want_per_sm = (int)tune("STRATA_DISP_CTAS", deep ? 1 : lanes);
    p.stages = (int)tune("STRATA_DISP_STAGES", deep ? min(kDeepRingMaxStages, (int)(kDeepRingBytes / stage_bytes)) : kBf16Stages);
    while (p.stages > 2 && (size_t)p.stages * (stage_bytes + 12) + 16 > kBf16MaxSmem) --p.stages;
    const size_t need = (size_t)p.stages * stage_bytes + 12 * (size_t)p.stages + 16;   // stages | mbarriers | unit ids
    size_t smem = 0;
    int per_sm = 0;
    cudaError_t err = smem_for_residency(dispatch_bf16_kernel, 32, need, want_per_sm, kBf16MaxSmem, &smem, &per_sm);
    if (err != cudaSuccess) return err;
    p.n_units = (long long)s.R * s.T * p.chunks_per_row;
    p.store_hint = (long long)s.R * s.T * s.K * s.H * 2 >= (tune("STRATA_DISP_STORE_HINT_MB", kStoreHintMinBytes >> 20) << 20);
#ifdef STRATA_TEST_HOOKS
    p.test_flags = g_inject_short_copy.exchange(0);
#endif
    const long long max_grid = (long long)n_sm * per_sm;
    const long long grid = max(1ll, min(max_grid, p.n_units));
    const bool small = (long long)s.R * s.T * s.H * 2 * (s.K + 1) < pdl_max_bytes();
    return STRATA_LAUNCH_LONG(small, dispatch_bf16_kernel, (unsigned)grid, 32, smem, st, p);
}

cudaError_t launch_dispatch_fp8(const strata_moe_shape& s, const int32_t* dst_row, const void* x, void* recv_q,
                                float* recv_scale, size_t capacity_rows, int* status, WorkQueue wq, int n_sm,
                                TraceBuf trace, bool x_early, cudaStream_t st)
{
    DispatchParams p{};
    p.x_early = x_early ? 1 : 0;
    p.trace = trace;
    p.wq = wq;
    p.dst_row = dst_row;
    p.x = static_cast<const unsigned char*>(x);
    p.recv = static_cast<unsigned char*>(recv_q);
    p.recv_scale = recv_scale;
    p.K = s.K;
    p.H = s.H;
    p.chunk_cols = (uint32_t)min(s.H, kFp8MaxChunkCols);
    p.chunks_per_row = (int)(((uint32_t)s.H + p.chunk_cols - 1) / p.chunk_cols);
    p.n_units = (long long)s.R * s.T * p.chunks_per_row;
#ifdef STRATA_TEST_HOOKS
    p.test_flags = g_inject_short_copy.exchange(0);
#endif
    p.capacity_rows = (long long)capacity_rows;
    p.status = status;
    const size_t need = (size_t)p.chunk_cols * 6u + 64;
    // as many CTAs per SM as fit, and the request padded so that not one more does
    int natural = 0;
    cudaError_t err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&natural, dispatch_fp8_kernel, kFp8Threads, need);
    if (err != cudaSuccess) return err;
    size_t smem = 0;
    int per_sm = 0;
    err = smem_for_residency(dispatch_fp8_kernel, kFp8Threads, need, max(1, natural), kBf16MaxSmem, &smem, &per_sm);
    if (err != cudaSuccess) return err;
    const long long grid = max(1ll, min((long long)n_sm * per_sm, p.n_units));
    const bool small = (long long)s.R * s.T * s.H * (s.K + 2) < pdl_max_bytes();
    return STRATA_LAUNCH_LONG(small, dispatch_fp8_kernel, (unsigned)grid, kFp8Threads, smem, st, p);
}

}  // namespace strata

#ifdef STRATA_TEST_HOOKS
// Test builds only (not declared in the public header): arms the one-shot short-copy injection above.
extern "C" void strata_test_inject_short_copy(int on) { strata::g_inject_short_copy.store(on ? 1 : 0); }
#endif
