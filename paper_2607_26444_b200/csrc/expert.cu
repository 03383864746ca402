// In-place consumer of the receive buffer (paper Sec. 2.2 / 8.1: the buffer dispatch fills is the input of
// the expert computation, with no staging copy in between).  The paper's expert is a grouped GEMM, which is
// not part of this path; what is built here is the part of such a consumer that touches the hand-over: the
// walk over row tiles, each tile finding the expert that owns it from the layout's offsets (segments are
// aligned to the tile height, so a tile never holds two experts) and the number of occupied rows in it,
// with a per-expert affine map standing in for the GEMM:
//   recv[row][c] = bf16_rne( fma( f32(recv[row][c]), scale[e], bias[e] ) )
// Bound by HBM: every occupied row is read once and written once, 16 bytes per thread per access, eight
// independent loads in flight per thread.  One CTA per (tile, column part): the hardware's CTA scheduler
// deals the units out as SMs free up, so nothing is statically partitioned.
#include "common.cuh"

namespace strata {

namespace {

constexpr int kExpertThreads = 256;
constexpr int kExpertVecPerThread = 8;

struct ExpertParams {
    const int32_t* expert_count;
    const int32_t* expert_offset;
    const float* scale;
    const float* bias;
    unsigned char* recv;
    int E, H, tile_rows;
    int parts;              // column parts per tile
    int vec_per_part;       // 16-byte vectors of one row in a part (the last part may be shorter)
};

__device__ __forceinline__ uint32_t affine_pack(uint32_t u, float s, float b)
{
    const float lo = __fmaf_rn(__uint_as_float(u << 16), s, b);
    const float hi = __fmaf_rn(__uint_as_float(u & 0xffff0000u), s, b);
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

__global__ void __launch_bounds__(kExpertThreads) expert_affine_kernel(ExpertParams p)
{
    extern __shared__ int offs[];         // [E + 1]
    __shared__ int s_expert, s_rows;
    griddep_wait();                       // the layout arrays and the rows come from earlier kernels
    const unsigned int tile = blockIdx.x / (unsigned int)p.parts;
    const int part = (int)(blockIdx.x - tile * (unsigned int)p.parts);
    const long long row0 = (long long)tile * p.tile_rows;
    for (int x = threadIdx.x; x <= p.E; x += kExpertThreads) offs[x] = p.expert_offset[x];
    __syncthreads();
    if (threadIdx.x == 0) {
        int e = -1, rows = 0;
        if (row0 < offs[p.E]) {
            int a = 0, b = p.E;           // invariant: offs[a] <= row0 < offs[b]; empty experts have equal offsets
            while (b - a > 1) {
                const int m = (a + b) >> 1;
                if (offs[m] <= row0) a = m; else b = m;
            }
            e = a;
            const long long left = (long long)offs[a] + p.expert_count[a] - row0;    // occupied rows from row0 on
            rows = (int)max(0ll, min((long long)p.tile_rows, left));
        }
        s_expert = e;
        s_rows = rows;
    }
    __syncthreads();
    griddep_launch_dependents();
    const int rows = s_rows;
    if (rows == 0) return;                // a tile of padding only, or beyond the last segment
    const float sc = p.scale[s_expert], bi = p.bias[s_expert];
    const int vpr = p.H / 8;              // 16-byte vectors per row
    const int v0 = part * p.vec_per_part, nv = min(p.vec_per_part, vpr - v0);
    const size_t row_bytes = (size_t)p.H * 2u;
    unsigned char* base = p.recv + (size_t)row0 * row_bytes + (size_t)v0 * 16u;
    // Threads form 256 / tpr groups of tpr threads (tpr a power of two, at most the vectors of a row part): a
    // group takes every (256 / tpr)-th row, a thread of it every tpr-th vector of the row.  Lanes of a warp read
    // consecutive vectors, and no index needs a division.
    int tpr_log2 = 0;
    while ((2 << tpr_log2) <= min(nv, kExpertThreads)) ++tpr_log2;
    const int tpr = 1 << tpr_log2, groups = kExpertThreads >> tpr_log2;
    const int my_v = (int)threadIdx.x & (tpr - 1), my_g = (int)threadIdx.x >> tpr_log2;
    for (int v = my_v; v < nv; v += tpr) {
        unsigned char* col = base + (size_t)v * 16u;
        for (int r0 = my_g; r0 < rows; r0 += groups * kExpertVecPerThread) {
            uint4 d[kExpertVecPerThread];
#pragma unroll
            for (int q = 0; q < kExpertVecPerThread; ++q) {
                const int r = r0 + q * groups;
                if (r < rows) d[q] = *reinterpret_cast<const uint4*>(col + (size_t)r * row_bytes);
            }
#pragma unroll
            for (int q = 0; q < kExpertVecPerThread; ++q) {
                const int r = r0 + q * groups;
                if (r >= rows) continue;
                uint4 o;
                o.x = affine_pack(d[q].x, sc, bi);
                o.y = affine_pack(d[q].y, sc, bi);
                o.z = affine_pack(d[q].z, sc, bi);
                o.w = affine_pack(d[q].w, sc, bi);
                *reinterpret_cast<uint4*>(col + (size_t)r * row_bytes) = o;
            }
        }
    }
}

}  // namespace

cudaError_t launch_expert_affine(const strata_moe_shape& s, const strata_moe_layout_t& L, void* recv, long long n_rows,
                                 const float* scale, const float* bias, int tile_rows, int n_sm, cudaStream_t st)
{
    ExpertParams p{};
    p.expert_count = L.expert_count;
    p.expert_offset = L.expert_offset;
    p.scale = scale;
    p.bias = bias;
    p.recv = static_cast<unsigned char*>(recv);
    p.E = s.E;
    p.H = s.H;
    p.tile_rows = tile_rows;
    const long long tiles = (n_rows + tile_rows - 1) / tile_rows;
    // column parts: units of about 128 KB, but enough of them to fill the GPU several times over
    const int vpr = s.H / 8;
    long long per_part = max(1ll, (128ll * 1024 / 16) / tile_rows);          // vectors of a row in one part
    while (per_part > 1 && tiles * ((vpr + per_part - 1) / per_part) < (long long)n_sm * 32) per_part = (per_part + 1) / 2;
    p.vec_per_part = (int)min(per_part, (long long)vpr);
    p.parts = (vpr + p.vec_per_part - 1) / p.vec_per_part;
    const long long grid = tiles * p.parts;
    if (grid >= (1ll << 31)) return cudaErrorInvalidConfiguration;
    return launch_pdl(expert_affine_kernel, (unsigned)grid, kExpertThreads, (size_t)(s.E + 1) * sizeof(int), st, p);
}

}  // namespace strata
