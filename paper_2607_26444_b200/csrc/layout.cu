// Routing layout (paper App. C, level 1 "token placement"): per-expert counts, prefix-sum
// offsets and token-local offsets, as a stable counting sort of the items by expert id.
//
// Two launches, no device-side waiting anywhere:
//   1. layout_count_scan_kernel: one CTA per tile of 1024 items (a tile never spans two
//      source ranks).  Each warp aggregates equal ids with match.any so a popular expert
//      costs one shared-memory update per warp instead of 32; the tile's histogram goes
//      to the workspace.  The CTA that draws the last ticket turns the per-tile counts
//      into per-tile exclusive prefixes (per expert, in tile order = (rank, token, slot)
//      order), and produces expert_count/offset, rank_count/offset and src_expert_count.
//   2. layout_rank_kernel: one CTA per tile again; rank of an item inside its tile =
//      (items with the same id in earlier warps) + (same id in earlier lanes), both
//      from match.any masks, so the order is exact and no atomics decide a row.
#include <mutex>

#include "common.cuh"

namespace strata {

namespace {

struct LayoutParams {
    const int32_t* ids;
    int32_t* expert_count;
    int32_t* expert_offset;
    int32_t* rank_count;
    int32_t* rank_offset;
    int32_t* src_expert_count;
    int32_t* dst_row;
    int32_t* src_of_row;
    int* status;
    int* ticket;
    int* tile_cnt;
    int R, E, e_loc;
    int items_per_rank, tiles_per_rank, n_tiles;
};

// Exclusive scan of one value per thread over a 1024-thread block.
__device__ __forceinline__ int block_exclusive_scan_1024(int v, int* warp_sums /*[32]*/, int* total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) warp_sums[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        int s = warp_sums[lane];
        int si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, si, d);
            if (lane >= d) si += t;
        }
        warp_sums[lane] = si - s;   // exclusive
        if (lane == 31) *total = si;
    }
    __syncthreads();
    return warp_sums[wid] + inc - v;
}

__global__ void __launch_bounds__(kLayoutTile) layout_count_scan_kernel(LayoutParams p)
{
    extern __shared__ int sm[];          // part[groups*E] | offs[E+1] | warp_sums[32] | total
    const int tid = threadIdx.x, lane = tid & 31;
    const int E = p.E;
    int* hist = sm;

    const int tile = blockIdx.x;
    const int r = tile / p.tiles_per_rank, tt = tile - r * p.tiles_per_rank;
    const int in_rank = tt * kLayoutTile + tid;
    const long long item = (long long)r * p.items_per_rank + in_rank;

    for (int e = tid; e < E; e += kLayoutTile) hist[e] = 0;
    __syncthreads();

    bool valid = in_rank < p.items_per_rank;
    int e = valid ? p.ids[item] : -1;
    if (valid && (unsigned)e >= (unsigned)E) {
        report_status(p.status, STRATA_ERR_BAD_EXPERT_ID);
        valid = false;
        e = -1;
    }
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (valid && lane == __ffs(peers) - 1) atomicAdd(&hist[e], __popc(peers));
    __syncthreads();
    for (int x = tid; x < E; x += kLayoutTile) p.tile_cnt[(size_t)tile * E + x] = hist[x];

    // ---- last CTA to finish does the scans (a ticket, never a wait) ----
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(p.ticket, 1) == p.n_tiles - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // Threads form `groups` groups of E; group g scans the tiles of a block of ranks.
    const int groups = max(1, kLayoutTile / E);              // E <= 1024
    const int g = tid / E, ee = tid - g * E;
    const int ranks_per_group = (p.R + groups - 1) / groups;
    const int r0 = min(p.R, g * ranks_per_group), r1 = min(p.R, r0 + ranks_per_group);
    const bool active = g < groups;
    int* part = sm;                       // [groups, E]
    int* offs = sm + groups * E;          // [E + 1]
    int* warp_sums = offs + E + 1;        // [32]
    int* total = warp_sums + 32;

    int mine = 0;
    if (active) {
        for (int t = r0 * p.tiles_per_rank; t < r1 * p.tiles_per_rank; ++t)
            mine += __ldcg(&p.tile_cnt[(size_t)t * E + ee]);
        part[g * E + ee] = mine;
    }
    __syncthreads();
    int before = 0, count_e = 0;
    if (active) {
        for (int gg = 0; gg < groups; ++gg) {
            const int v = part[gg * E + ee];
            if (gg < g) before += v;
            count_e += v;
        }
    }

    // exclusive scan over experts (one expert per thread of group 0)
    const int v = (tid < E) ? count_e : 0;
    const int off = block_exclusive_scan_1024(v, warp_sums, total);
    if (tid < E) {
        p.expert_count[tid] = count_e;
        p.expert_offset[tid] = off;
        offs[tid] = off;
    }
    if (tid == 0) {
        p.expert_offset[E] = *total;
        p.rank_offset[p.R] = *total;
        offs[E] = *total;
    }
    __syncthreads();
    for (int d = tid; d < p.R; d += kLayoutTile) {
        const int lo = offs[d * p.e_loc], hi = offs[(d + 1) * p.e_loc];
        p.rank_offset[d] = lo;
        p.rank_count[d] = hi - lo;
    }

    // per-tile exclusive prefix (within the expert, across tiles in order) and per-source-rank counts
    if (active) {
        int running = before;
        for (int rr = r0; rr < r1; ++rr) {
            const int start = running;
            for (int t = rr * p.tiles_per_rank; t < (rr + 1) * p.tiles_per_rank; ++t) {
                int* c = &p.tile_cnt[(size_t)t * E + ee];
                const int n = __ldcg(c);
                *c = running;
                running += n;
            }
            if (p.src_expert_count) p.src_expert_count[(size_t)rr * E + ee] = running - start;
        }
    }
    if (tid == 0) *p.ticket = 0;          // ready for the next call on this stream
}

__global__ void __launch_bounds__(kLayoutTile) layout_rank_kernel(LayoutParams p)
{
    extern __shared__ int warp_cnt[];    // [32 warps, E]
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int E = p.E;
    const int tile = blockIdx.x;
    const int r = tile / p.tiles_per_rank, tt = tile - r * p.tiles_per_rank;
    const int in_rank = tt * kLayoutTile + tid;
    const long long item = (long long)r * p.items_per_rank + in_rank;

    for (int x = tid; x < 32 * E; x += kLayoutTile) warp_cnt[x] = 0;
    __syncthreads();

    const bool in_range = in_rank < p.items_per_rank;
    int e = in_range ? p.ids[item] : -1;
    const bool valid = in_range && (unsigned)e < (unsigned)E;
    if (!valid) e = -1;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (valid && lane == __ffs(peers) - 1) warp_cnt[wid * E + e] = __popc(peers);
    __syncthreads();
    // exclusive prefix over the 32 warps, per expert
    for (int x = tid; x < E; x += kLayoutTile) {
        int running = 0;
#pragma unroll 8
        for (int w = 0; w < 32; ++w) {
            const int c = warp_cnt[w * E + x];
            warp_cnt[w * E + x] = running;
            running += c;
        }
    }
    __syncthreads();
    if (valid) {
        const unsigned lt = (1u << lane) - 1u;
        const int row = p.expert_offset[e] + p.tile_cnt[(size_t)tile * E + e] + warp_cnt[wid * E + e] +
                        __popc(peers & lt);
        p.dst_row[item] = row;
        if (p.src_of_row) p.src_of_row[row] = (int32_t)item;
    } else if (in_range) {
        p.dst_row[item] = -1;
    }
}

size_t count_scan_smem(int E)
{
    const int groups = max(1, kLayoutTile / E);
    return (size_t)(groups * E + E + 1 + 32 + 2) * sizeof(int);
}

}  // namespace

cudaError_t configure_layout_kernels()
{
    cudaError_t err = cudaFuncSetAttribute(layout_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           32 * kMaxExperts * (int)sizeof(int));
    return err;
}

cudaError_t launch_layout(const strata_moe_shape& s, const int32_t* ids, const strata_moe_layout_t& L,
                          int* ws_header, int* tile_cnt, cudaStream_t st, int* n_launches)
{
    const LayoutGeom g = layout_geom(s);
    LayoutParams p;
    p.ids = ids;
    p.expert_count = L.expert_count;
    p.expert_offset = L.expert_offset;
    p.rank_count = L.rank_count;
    p.rank_offset = L.rank_offset;
    p.src_expert_count = L.src_expert_count;
    p.dst_row = L.dst_row;
    p.src_of_row = L.src_of_row;
    p.status = ws_header;
    p.ticket = ws_header + 1;
    p.tile_cnt = tile_cnt;
    p.R = s.R;
    p.E = s.E;
    p.e_loc = s.E / s.R;
    p.items_per_rank = g.items_per_rank;
    p.tiles_per_rank = g.tiles_per_rank;
    p.n_tiles = g.n_tiles;

    layout_count_scan_kernel<<<g.n_tiles, kLayoutTile, count_scan_smem(s.E), st>>>(p);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    layout_rank_kernel<<<g.n_tiles, kLayoutTile, (size_t)32 * s.E * sizeof(int), st>>>(p);
    *n_launches = 2;
    return cudaGetLastError();
}

}  // namespace strata

// ---------------------------------------------------------------------------------------------
// Allocation-free routing layout.
//
// Some callers have no way to give this library a workspace: a serving process whose framework pool
// has already claimed all device memory (a fresh cudaMalloc would fail or fragment it), a plug-in
// hook that must not cause the device-wide synchronisation that cudaMalloc/cudaFree imply, or a thin
// language binding that owns no device allocator at all.  For them the scratch of the layout kernels
// (status word, ticket, per-tile histograms) lives in the fixed array below instead of a workspace.
// Every GPU that loads this library holds the array (2 MiB) until the process exits.
// ---------------------------------------------------------------------------------------------
namespace strata {
namespace {

constexpr size_t kStaticScratchBytes = 2u << 20;       // header + int32[n_tiles, E]
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress, never an address to pass on.
static __device__ __align__(256) unsigned char g_layout_scratch[kStaticScratchBytes];

std::mutex g_scratch_mu;
int* g_scratch_ptr[kMaxDevices];                       // device address of the array, per device
bool g_scratch_ready[kMaxDevices];

// One-time set-up for the current device: resolve the array's device address and allow the rank
// kernel its shared-memory table.  Neither call allocates.
strata_status static_scratch_for_current_device(int** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return STRATA_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(g_scratch_mu);
    if (!g_scratch_ready[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_layout_scratch) != cudaSuccess || ptr == nullptr) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
        if (cudaFuncSetAttribute(layout_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 32 * kMaxExperts * (int)sizeof(int)) != cudaSuccess) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<int*>(ptr);
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_ptr[dev];
    return STRATA_OK;
}

}  // namespace
}  // namespace strata

extern "C" strata_status strata_moe_layout_noalloc(const strata_moe_shape* shape, const int32_t* topk_ids,
                                                   const strata_moe_layout_t* layout, int32_t* device_status,
                                                   void* stream)
{
    using namespace strata;
    if (!shape || !topk_ids || !layout) return STRATA_ERR_INVALID_ARG;
    if (!layout->expert_count || !layout->expert_offset || !layout->rank_count || !layout->rank_offset ||
        !layout->dst_row)
        return STRATA_ERR_INVALID_ARG;
    const strata_moe_shape& s = *shape;
    if (s.R <= 0 || s.T <= 0 || s.E <= 0 || s.K <= 0) return STRATA_ERR_SHAPE;
    if (s.E % s.R != 0 || s.E > kMaxExperts || s.K > kMaxTopK) return STRATA_ERR_SHAPE;
    if ((long long)s.R * s.T * s.K >= (1ll << 31)) return STRATA_ERR_SHAPE;
    const LayoutGeom g = layout_geom(s);
    const size_t need = (size_t)kWsHeaderBytes + (size_t)g.n_tiles * s.E * sizeof(int);
    if (need > kStaticScratchBytes) return STRATA_ERR_CAPACITY;     // beyond the fixed array: use a workspace

    int* scratch = nullptr;
    strata_status rc = static_scratch_for_current_device(&scratch);
    if (rc != STRATA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The array keeps whatever the previous call left: status word and ticket must start at zero.
    if (cudaMemsetAsync(scratch, 0, kWsHeaderBytes, st) != cudaSuccess) {
        cudaGetLastError();
        return STRATA_ERR_CUDA;
    }
    LayoutParams p;
    p.ids = topk_ids;
    p.expert_count = layout->expert_count;
    p.expert_offset = layout->expert_offset;
    p.rank_count = layout->rank_count;
    p.rank_offset = layout->rank_offset;
    p.src_expert_count = layout->src_expert_count;
    p.dst_row = layout->dst_row;
    p.src_of_row = layout->src_of_row;
    p.status = device_status ? device_status : scratch;
    p.ticket = scratch + 1;
    p.tile_cnt = scratch + kWsHeaderBytes / sizeof(int);
    p.R = s.R;
    p.E = s.E;
    p.e_loc = s.E / s.R;
    p.items_per_rank = g.items_per_rank;
    p.tiles_per_rank = g.tiles_per_rank;
    p.n_tiles = g.n_tiles;
    layout_count_scan_kernel<<<g.n_tiles, kLayoutTile, count_scan_smem(s.E), st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return STRATA_ERR_CUDA;
    layout_rank_kernel<<<g.n_tiles, kLayoutTile, (size_t)32 * s.E * sizeof(int), st>>>(p);
    return cudaGetLastError() == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}
