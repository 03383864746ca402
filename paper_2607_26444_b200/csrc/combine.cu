// Gate-weighted combine (paper Sec. 6.1, reduction-bearing operators: remote operands are
// accumulated into the local destination).  Per token n and column c:
//   out[n,c] = bf16_rne( fma(w[n,K-1], y[row(n,K-1),c], ... fma(w[n,0], y[row(n,0),c], +0) ) )
// with binary32 fused multiply-adds in slot order 0..K-1.
//
// Work split: a unit is one token, or one column part of a token when there are too few tokens to
// give every CTA several units: K (part-)row reads and one write whatever the expert popularity is.
// The CTAs of a persistent grid start on unit blockIdx.x and then claim units in order from a
// counter in the workspace, one unit ahead of the one being worked on (the claim travels while the
// rows stream in), so no CTA is left with a fixed share it cannot finish in time.  A thread owns one
// 16-byte column vector at a time: it issues the K independent 16-byte streaming loads first
// (K requests in flight per thread), then runs the FMA chain in registers and writes 16 bytes.
// The accumulation lives in registers; no atomics and no shared-memory staging are needed
// because one thread sees all K operands of its columns.
#include "common.cuh"

namespace strata {

namespace {

#ifndef STRATA_COMBINE_THREADS
#define STRATA_COMBINE_THREADS 128
#endif
#ifndef STRATA_COMBINE_MAX_CTAS_PER_SM
#define STRATA_COMBINE_MAX_CTAS_PER_SM 0     // 0: as many as fit
#endif
#ifndef STRATA_COMBINE_UNITS_PER_CTA
#define STRATA_COMBINE_UNITS_PER_CTA 24      // rows are split into column parts until a CTA can expect this many units
#endif
#ifndef STRATA_COMBINE_LOAD_HINT
#define STRATA_COMBINE_LOAD_HINT 0           // 1: the row loads carry an L2 evict-first policy (measured: no effect at any shape)
#endif
constexpr int kCombineThreads = STRATA_COMBINE_THREADS;

struct CombineParams {
    const int32_t* dst_row;
    const unsigned char* y;
    const float* w;
    unsigned char* out;
    long long n_tok;
    long long y_rows;
    int H;
    int K;
    int parts;             // units per token
    int vec_per_part;      // 16-byte vectors per unit, a multiple of the CTA size (last part may be shorter)
    int* status;
    WorkQueue wq;
    TraceBuf trace;
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

__device__ __forceinline__ void fma8(float (&a)[8], float wv, const uint4& d)
{
    a[0] = __fmaf_rn(wv, __uint_as_float(d.x << 16), a[0]);
    a[1] = __fmaf_rn(wv, __uint_as_float(d.x & 0xffff0000u), a[1]);
    a[2] = __fmaf_rn(wv, __uint_as_float(d.y << 16), a[2]);
    a[3] = __fmaf_rn(wv, __uint_as_float(d.y & 0xffff0000u), a[3]);
    a[4] = __fmaf_rn(wv, __uint_as_float(d.z << 16), a[4]);
    a[5] = __fmaf_rn(wv, __uint_as_float(d.z & 0xffff0000u), a[5]);
    a[6] = __fmaf_rn(wv, __uint_as_float(d.w << 16), a[6]);
    a[7] = __fmaf_rn(wv, __uint_as_float(d.w & 0xffff0000u), a[7]);
}

// K known at compile time: row pointers and weights of the token live in registers.
template <int K>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(CombineParams p)
{
    const int tid = threadIdx.x;
    const int vpr = p.H / 8;                       // 16-byte vectors per row
    const size_t row_bytes = (size_t)p.H * 2u;
    const unsigned int n_units = (unsigned int)(p.n_tok * p.parts);
    __shared__ unsigned int s_next[2];             // the claim made during unit j is read for unit j+1
#if STRATA_COMBINE_LOAD_HINT
    const uint64_t pol = policy_evict_first();
#endif
    griddep_wait();
    if (tid == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_COMBINE, tid == 0);
    tl.begin(STRATA_STAGE_KERNEL);

    unsigned int u = blockIdx.x < n_units ? blockIdx.x : kNoUnit;
    bool exhausted = false;                        // thread 0's view of the queue
    for (int j = 0; u != kNoUnit; ++j) {
        tl.begin(STRATA_STAGE_WORK);
        if (tid == 0) {
            const unsigned int nx = claim_unit(p.wq, n_units, gridDim.x, exhausted);
            s_next[j & 1] = nx;
            if (nx == kNoUnit) griddep_launch_dependents();   // last unit of this CTA: let the next kernel in
        }
        const unsigned int n = u / (unsigned int)p.parts;
        const int part = (int)(u - n * (unsigned int)p.parts);
        const int v_begin = part * p.vec_per_part, v_end = min(v_begin + p.vec_per_part, vpr);
        const unsigned char* src[K];
        float wk[K];
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const int row = p.dst_row[(long long)n * K + k];
            const bool row_ok = row >= 0 && row < p.y_rows;
            if (!row_ok && row != -1 && tid == 0 && part == 0) report_status(p.status, STRATA_ERR_BAD_ROW);
            src[k] = row_ok ? p.y + (size_t)row * row_bytes : nullptr;
            wk[k] = p.w[(long long)n * K + k];
        }
        unsigned char* dst = p.out + (size_t)n * row_bytes;
        for (int v = v_begin + tid; v < v_end; v += kCombineThreads) {
            uint4 d[K];
#pragma unroll
            for (int k = 0; k < K; ++k)
#if STRATA_COMBINE_LOAD_HINT
                d[k] = src[k] ? ld_stream16_hint(src[k] + (size_t)v * 16, pol) : make_uint4(0, 0, 0, 0);
#else
                d[k] = src[k] ? ld_stream16(src[k] + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
#endif
            float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int k = 0; k < K; ++k)
                if (src[k]) fma8(a, wk[k], d[k]);
            uint4 o;
            o.x = pack_bf16x2(a[0], a[1]);
            o.y = pack_bf16x2(a[2], a[3]);
            o.z = pack_bf16x2(a[4], a[5]);
            o.w = pack_bf16x2(a[6], a[7]);
            st_stream16(dst + (size_t)v * 16, o);
        }
        __syncthreads();                           // one barrier per unit: publishes the next claim
        tl.end(STRATA_STAGE_WORK);
        u = s_next[j & 1];
    }
    if (tid == 0) {
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

// Any K <= kMaxTopK: a CTA claims whole tokens; slots are taken in groups of up to 8, in slot order.
template <>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel<0>(CombineParams p)
{
    const int tid = threadIdx.x, K = p.K;
    const int vpr = p.H / 8;
    const size_t row_bytes = (size_t)p.H * 2u;
    const unsigned int n_units = (unsigned int)p.n_tok;
    __shared__ long long s_off[kMaxTopK];          // byte offset of the row, -1 if skipped
    __shared__ float s_w[kMaxTopK];
    __shared__ unsigned int s_tok;
    griddep_wait();
    if (tid == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_COMBINE, tid == 0);
    tl.begin(STRATA_STAGE_KERNEL);

    bool exhausted = false;
    for (int j = 0;; ++j) {
        __syncthreads();                           // everyone is done with the previous token's tables
        if (tid == 0) s_tok = j == 0 ? (blockIdx.x < n_units ? blockIdx.x : kNoUnit)
                                     : claim_unit(p.wq, n_units, gridDim.x, exhausted);
        __syncthreads();
        const unsigned int n = s_tok;
        if (n == kNoUnit) break;
        tl.begin(STRATA_STAGE_WORK);
        if (tid < K) {
            const int row = p.dst_row[(long long)n * K + tid];
            const bool row_ok = row >= 0 && row < p.y_rows;
            if (!row_ok && row != -1) report_status(p.status, STRATA_ERR_BAD_ROW);
            s_off[tid] = row_ok ? (long long)row * (long long)row_bytes : -1;
            s_w[tid] = p.w[(long long)n * K + tid];
        }
        __syncthreads();
        unsigned char* dst = p.out + (size_t)n * row_bytes;
        for (int v = tid; v < vpr; v += kCombineThreads) {
            float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int k0 = 0; k0 < K; k0 += 8) {
                uint4 d[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const long long off = (k0 + k < K) ? s_off[k0 + k] : -1;
                    d[k] = off >= 0 ? ld_stream16(p.y + off + (size_t)v * 16) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    if (k0 + k < K && s_off[k0 + k] >= 0) fma8(a, s_w[k0 + k], d[k]);
            }
            uint4 o;
            o.x = pack_bf16x2(a[0], a[1]);
            o.y = pack_bf16x2(a[2], a[3]);
            o.z = pack_bf16x2(a[4], a[5]);
            o.w = pack_bf16x2(a[6], a[7]);
            st_stream16(dst + (size_t)v * 16, o);
        }
        tl.end(STRATA_STAGE_WORK);
    }
    if (tid == 0) {
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

template <int KT>
cudaError_t launch_k(const CombineParams& p, int n_sm, cudaStream_t st)
{
    int per_sm = 0;
    cudaError_t err =
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, combine_kernel<KT>, kCombineThreads, 0);
    if (err != cudaSuccess) return err;
    if (per_sm < 1) per_sm = 1;
    const int cap_per_sm = (int)tune("STRATA_COMB_CTAS", STRATA_COMBINE_MAX_CTAS_PER_SM);
    if (cap_per_sm > 0) per_sm = min(per_sm, cap_per_sm);
    CombineParams q = p;
    const long long max_grid = (long long)n_sm * per_sm;
    q.parts = 1;
    q.vec_per_part = (p.H / 8 + kCombineThreads - 1) / kCombineThreads * kCombineThreads;
    if (KT > 0) {
        // split rows into column parts until every CTA can expect about 6 units (never below one
        // vector per thread per unit)
        const int m_full = q.vec_per_part / kCombineThreads;
        int parts = 1;
        const long long want_units = tune("STRATA_COMB_UNITS", STRATA_COMBINE_UNITS_PER_CTA) * max_grid;
        while (parts < m_full && p.n_tok * parts < want_units) ++parts;
        q.vec_per_part = (m_full + parts - 1) / parts * kCombineThreads;
        q.parts = (p.H / 8 + q.vec_per_part - 1) / q.vec_per_part;
    }
    const long long grid = max(1ll, min(max_grid, p.n_tok * q.parts));
    const bool small = p.n_tok * p.H * 2 * (p.K + 1) < pdl_max_bytes();
    return STRATA_LAUNCH_LONG(small, combine_kernel<KT>, (unsigned)grid, kCombineThreads, 0, st, q);
}

}  // namespace

cudaError_t launch_combine(const strata_moe_shape& s, const int32_t* dst_row, const void* y, size_t y_rows,
                           const float* w, void* out, int* status, WorkQueue wq, int n_sm, TraceBuf trace,
                           cudaStream_t st)
{
    CombineParams p{};
    p.trace = trace;
    p.wq = wq;
    p.dst_row = dst_row;
    p.y = static_cast<const unsigned char*>(y);
    p.w = w;
    p.out = static_cast<unsigned char*>(out);
    p.n_tok = (long long)s.R * s.T;
    p.y_rows = (long long)y_rows;
    p.H = s.H;
    p.K = s.K;
    p.status = status;
    switch (s.K) {
        case 1: return launch_k<1>(p, n_sm, st);
        case 2: return launch_k<2>(p, n_sm, st);
        case 3: return launch_k<3>(p, n_sm, st);
        case 4: return launch_k<4>(p, n_sm, st);
        case 5: return launch_k<5>(p, n_sm, st);
        case 6: return launch_k<6>(p, n_sm, st);
        case 7: return launch_k<7>(p, n_sm, st);
        case 8: return launch_k<8>(p, n_sm, st);
        default: return launch_k<0>(p, n_sm, st);
    }
}

}  // namespace strata
