// Small helpers around the layout.
// Row -> expert map of the receive buffer: the per-row group index a grouped expert GEMM needs to
// read the buffer in place (one expert per tile once the segments are aligned to the tile height).
// row_expert[row] = the expert whose segment holds the row if a token was placed there, else -1.
// One thread per row; the E+1 offsets (or the R*E slot counts) are staged in shared memory and a
// row finds its expert by a binary search of the offsets.
#include "common.cuh"

namespace strata {

namespace {

constexpr int kRowMapThreads = 256;

struct RowMapParams {
    const int32_t* expert_count;
    const int32_t* expert_offset;
    const int32_t* src_expert_count;      // fixed-capacity layout only
    int32_t* row_expert;
    long long n_rows;
    int R, E, capacity;
};

__global__ void __launch_bounds__(kRowMapThreads) row_experts_kernel(RowMapParams p)
{
    extern __shared__ int sm[];           // packed: offs[E+1] | cnt[E]
    griddep_wait();                       // the layout arrays come from the kernel before
    griddep_launch_dependents();
    const long long row0 = (long long)blockIdx.x * kRowMapThreads * 4;
    if (p.capacity > 0) {
        // row = (e*R + r)*C + j holds a token iff j < src_expert_count[r][e]
        for (int q = 0; q < 4; ++q) {
            const long long row = row0 + q * kRowMapThreads + threadIdx.x;
            if (row >= p.n_rows) break;
            const long long slot = row / p.capacity;
            const int j = (int)(row - slot * p.capacity);
            const int e = (int)(slot / p.R), r = (int)(slot - (long long)e * p.R);
            p.row_expert[row] = j < p.src_expert_count[r * p.E + e] ? e : -1;
        }
        return;
    }
    int* offs = sm;
    int* cnt = sm + p.E + 1;
    for (int x = threadIdx.x; x <= p.E; x += kRowMapThreads) offs[x] = p.expert_offset[x];
    for (int x = threadIdx.x; x < p.E; x += kRowMapThreads) cnt[x] = p.expert_count[x];
    __syncthreads();
    for (int q = 0; q < 4; ++q) {
        const long long row = row0 + q * kRowMapThreads + threadIdx.x;
        if (row >= p.n_rows) break;
        int e = -1;
        if (row < offs[p.E]) {
            int a = 0, b = p.E;           // invariant: offs[a] <= row < offs[b]; empty experts have equal offsets
            while (b - a > 1) {
                const int m = (a + b) >> 1;
                if (offs[m] <= row) a = m; else b = m;
            }
            e = row - offs[a] < cnt[a] ? a : -1;      // beyond the count: padding of an aligned segment
        }
        p.row_expert[row] = e;
    }
}

// Ranks with different token counts: the slots of the tokens t >= tokens_per_rank[r] become -1 ("not routed").
__global__ void __launch_bounds__(kRowMapThreads) mask_ragged_kernel(const int32_t* tokens_per_rank, int32_t* ids, int R,
                                                                      int T, int K)
{
    griddep_wait();
    griddep_launch_dependents();
    const long long n = (long long)R * T * K;
    const long long per_rank = (long long)T * K;
    for (long long i = (long long)blockIdx.x * kRowMapThreads + threadIdx.x; i < n; i += (long long)gridDim.x * kRowMapThreads) {
        const int r = (int)(i / per_rank);
        const int t = (int)((i - (long long)r * per_rank) / K);
        if (t >= tokens_per_rank[r]) ids[i] = -1;
    }
}

}  // namespace

cudaError_t launch_mask_ragged(const strata_moe_shape& s, const int32_t* tokens_per_rank, int32_t* ids, int n_sm,
                               cudaStream_t st)
{
    const long long n = (long long)s.R * s.T * s.K;
    const unsigned grid = (unsigned)max(1ll, min((long long)n_sm * 8, (n + kRowMapThreads - 1) / kRowMapThreads));
    return launch_pdl(mask_ragged_kernel, grid, kRowMapThreads, 0, st, tokens_per_rank, ids, (int)s.R, (int)s.T, (int)s.K);
}

cudaError_t launch_row_experts(const strata_moe_shape& s, const strata_moe_layout_t& L, int32_t* row_expert,
                               long long n_rows, cudaStream_t st)
{
    RowMapParams p{};
    p.expert_count = L.expert_count;
    p.expert_offset = L.expert_offset;
    p.src_expert_count = L.src_expert_count;
    p.row_expert = row_expert;
    p.n_rows = n_rows;
    p.R = s.R;
    p.E = s.E;
    p.capacity = s.slot_capacity > 0 ? s.slot_capacity : 0;
    const long long per_cta = (long long)kRowMapThreads * 4;
    const unsigned grid = (unsigned)((n_rows + per_cta - 1) / per_cta);
    const size_t smem = (size_t)(2 * s.E + 1) * sizeof(int);
    return launch_pdl(row_experts_kernel, grid, kRowMapThreads, smem, st, p);
}

}  // namespace strata
