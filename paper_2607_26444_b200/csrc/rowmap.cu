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

}  // namespace

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
