// Routing layout (paper App. D, level 1 "token placement"): per-expert counts, prefix-sum
// offsets and token-local offsets, as a stable counting sort of the items by expert id.
//
// Batches of up to 32,768 items take one launch of one thread-block cluster (layout_cluster_kernel).
// Larger batches take two launches, no device-side waiting anywhere:
//   1. layout_count_scan_kernel: one CTA per tile of 4096 items (a tile never spans two
//      source ranks).  Each warp aggregates equal ids with ballot-built same-id masks so a popular expert
//      costs one shared-memory update per warp instead of 32; the tile's histogram goes
//      to the workspace.  The CTA that draws the last ticket turns the per-tile counts
//      into per-tile exclusive prefixes (per expert, in tile order = (rank, token, slot)
//      order), and produces expert_count/offset, rank_count/offset and src_expert_count.
//   2. layout_rank_kernel: one CTA per tile again; rank of an item inside its tile =
//      (items with the same id in earlier warps) + (same id in earlier lanes), both
//      from same-id lane masks, so the order is exact and no atomics decide a row.
#include <cooperative_groups.h>

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
    int align;            // >= 1: rows every expert segment is padded to
    int allow_unrouted;   // id -1 is legal and means "not routed"
    int capacity;         // > 0: fixed-capacity layout [E][R][capacity]
};

__device__ __forceinline__ int round_up_rows(int n, int a) { return (n + a - 1) / a * a; }

// Lanes of the warp holding the same key (0 <= key < 2^nbits), from nbits ballots.  Invalid lanes
// (key < 0) get a mask of the other invalid lanes, which callers ignore.  Measured several times
// faster than match.any when all 32 warps of a CTA use it back to back.
__device__ __forceinline__ unsigned same_key_lanes(int key, int nbits)
{
    unsigned peers = 0xffffffffu;
    const unsigned ukey = (unsigned)key;
    for (int b = 0; b < nbits; ++b) {
        const unsigned vote = __ballot_sync(0xffffffffu, (ukey >> b) & 1u);
        peers &= ((ukey >> b) & 1u) ? vote : ~vote;
    }
    const unsigned neg = __ballot_sync(0xffffffffu, key < 0);
    return peers & (key < 0 ? neg : ~neg);
}

__device__ __forceinline__ int key_bits(int n_keys)      // bits needed for keys in [0, n_keys)
{
    return n_keys <= 1 ? 0 : 32 - __clz(n_keys - 1);
}

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

// Items a warp owns inside a tile: kItemsPerThread rounds of 32 consecutive items, so the order
// inside a tile is (warp, round, lane) = increasing item index.
constexpr int kWarpItems = 32 * kItemsPerThread;

__global__ void __launch_bounds__(kLayoutThreads) layout_count_scan_kernel(LayoutParams p)
{
    extern __shared__ int sm[];          // part[groups*E] | offs[E+1] | warp_sums[32] | total
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int E = p.E;
    int* hist = sm;

    const int tile = blockIdx.x;
    const int r = tile / p.tiles_per_rank, tt = tile - r * p.tiles_per_rank;
    const int warp_first = tt * kLayoutTile + wid * kWarpItems;      // index inside the rank
    const long long rank_base = (long long)r * p.items_per_rank;

    for (int e = tid; e < E; e += kLayoutThreads) hist[e] = 0;
    __syncthreads();
    const int ebits = key_bits(E);
    griddep_wait();
    griddep_launch_dependents();          // the rank kernel may start its local pass now

    int ids[kItemsPerThread];
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        ids[q] = in_rank < p.items_per_rank ? p.ids[rank_base + in_rank] : -1;
    }
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        bool valid = in_rank < p.items_per_rank;
        int e = ids[q];
        if (valid && (unsigned)e >= (unsigned)E) {
            if (!(p.allow_unrouted && e == -1)) report_status(p.status, STRATA_ERR_BAD_EXPERT_ID);
            valid = false;
            e = -1;
        }
        const unsigned peers = same_key_lanes(e, ebits);
        if (valid && lane == __ffs(peers) - 1) atomicAdd(&hist[e], __popc(peers));
    }
    __syncthreads();
    for (int x = tid; x < E; x += kLayoutThreads) p.tile_cnt[(size_t)tile * E + x] = hist[x];

    // ---- last CTA to finish does the scans (a ticket, never a wait) ----
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(p.ticket, 1) == p.n_tiles - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // Threads form `groups` groups of E; group g scans a contiguous chunk of tiles for expert ee.
    // Loads go out in independent batches of 8 so the chain is latency/8, and the first
    // kScanCache counts stay in registers for the second walk.
    const int groups = max(1, kLayoutThreads / E);           // E <= 1024
    const int g = tid / E, ee = tid - g * E;
    const int chunk = (p.n_tiles + groups - 1) / groups;
    const int t0 = min(p.n_tiles, g * chunk), t1 = min(p.n_tiles, t0 + chunk);
    const bool active = g < groups;
    int* part = sm;                       // [groups, E]
    int* offs = sm + groups * E;          // [E + 1]
    int* warp_sums = offs + E + 1;        // [32]
    int* total = warp_sums + 32;

    constexpr int kScanCache = 32;
    int cache[kScanCache];
    int mine = 0;
    if (active) {
        const int* col = p.tile_cnt + ee;
#pragma unroll
        for (int b = 0; b < kScanCache; b += 8) {
            int v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (t0 + b + i < t1) ? __ldcg(col + (size_t)(t0 + b + i) * E) : 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                cache[b + i] = v[i];
                mine += v[i];
            }
        }
        for (int t = t0 + kScanCache; t < t1; t += 8) {
            int v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (t + i < t1) ? __ldcg(col + (size_t)(t + i) * E) : 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) mine += v[i];
        }
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

    // exclusive scan over experts of the padded segment lengths (one expert per thread of group 0)
    const int v = (tid < E) ? round_up_rows(count_e, p.align) : 0;
    const int off = block_exclusive_scan_1024(v, warp_sums, total);
    if (tid < E) {
        p.expert_count[tid] = count_e;
        p.expert_offset[tid] = off;
        offs[tid] = off;
        if (p.src_of_row)                 // padding rows of this segment have no source item
            for (int row = off + count_e; row < off + v; ++row) p.src_of_row[row] = -1;
    }
    if (tid == 0) {
        p.expert_offset[E] = *total;
        p.rank_offset[p.R] = *total;
        offs[E] = *total;
    }
    __syncthreads();
    for (int d = tid; d < p.R; d += kLayoutThreads) {
        p.rank_offset[d] = offs[d * p.e_loc];
        int real = 0;
        for (int e2 = d * p.e_loc; e2 < (d + 1) * p.e_loc; ++e2) real += p.expert_count[e2];
        p.rank_count[d] = real;
    }

    // per-tile exclusive prefix (within the expert, across tiles in order).  The prefix at the first
    // tile of each source rank also gives src_expert_count by differences.
    if (active) {
        int* col = p.tile_cnt + ee;
        int running = before;
#pragma unroll
        for (int i = 0; i < kScanCache; ++i) {
            const int t = t0 + i;
            if (t < t1) {
                col[(size_t)t * E] = running;
                running += cache[i];
            }
        }
        for (int t = t0 + kScanCache; t < t1; t += 8) {
            int v8[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v8[i] = (t + i < t1) ? __ldcg(col + (size_t)(t + i) * E) : 0;
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (t + i < t1) {
                    col[(size_t)(t + i) * E] = running;
                    running += v8[i];
                }
        }
    }
    if (p.capacity > 0) {
        // Fixed-capacity layout: rows are [E][R][capacity]; counts are clamped to the capacity, the
        // offsets are constants, and every row starts empty.
        __syncthreads();                  // the prefixes written above, by this CTA, are read below
        const int C = p.capacity;
        if (tid < E) {
            int kept_sum = 0;
            bool over = false;
            for (int rr = 0; rr < p.R; ++rr) {
                const int lo = p.tile_cnt[(size_t)(rr * p.tiles_per_rank) * E + tid];
                const int hi = (rr + 1 < p.R) ? p.tile_cnt[(size_t)((rr + 1) * p.tiles_per_rank) * E + tid] : count_e;
                const int kept = min(hi - lo, C);
                over |= hi - lo > C;
                if (p.src_expert_count) p.src_expert_count[(size_t)rr * E + tid] = kept;
                kept_sum += kept;
            }
            if (over) report_status(p.status, STRATA_ERR_CAPACITY);
            p.expert_count[tid] = kept_sum;
            p.expert_offset[tid] = tid * p.R * C;
            offs[tid] = kept_sum;         // reused below for the per-rank sums
        }
        if (tid == 0) {
            p.expert_offset[E] = E * p.R * C;
            p.rank_offset[p.R] = E * p.R * C;
        }
        __syncthreads();
        for (int d = tid; d < p.R; d += kLayoutThreads) {
            int real = 0;
            for (int e2 = d * p.e_loc; e2 < (d + 1) * p.e_loc; ++e2) real += offs[e2];
            p.rank_count[d] = real;
            p.rank_offset[d] = d * p.e_loc * p.R * C;
        }
        if (p.src_of_row)
            for (long long x = tid; x < (long long)E * p.R * C; x += kLayoutThreads) p.src_of_row[x] = -1;
    } else if (p.src_expert_count) {
        __syncthreads();                  // the prefixes written above, by this CTA, are read below
        for (int x = tid; x < p.R * E; x += kLayoutThreads) {
            const int rr = x / E, e2 = x - rr * E;
            const int lo = p.tile_cnt[(size_t)(rr * p.tiles_per_rank) * E + e2];
            const int hi = (rr + 1 < p.R) ? p.tile_cnt[(size_t)((rr + 1) * p.tiles_per_rank) * E + e2]
                                          : p.expert_count[e2];
            p.src_expert_count[x] = hi - lo;
        }
    }
    if (tid == 0) *p.ticket = 0;          // ready for the next call on this stream
}

__global__ void __launch_bounds__(kLayoutThreads) layout_rank_kernel(LayoutParams p)
{
    extern __shared__ int warp_cnt[];    // [32 warps, E]
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int E = p.E;
    const int tile = blockIdx.x;
    const int r = tile / p.tiles_per_rank, tt = tile - r * p.tiles_per_rank;
    const int warp_first = tt * kLayoutTile + wid * kWarpItems;
    const long long rank_base = (long long)r * p.items_per_rank;

    int ids[kItemsPerThread];
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        ids[q] = in_rank < p.items_per_rank ? p.ids[rank_base + in_rank] : -1;
    }
    for (int x = tid; x < 32 * E; x += kLayoutThreads) warp_cnt[x] = 0;
    __syncthreads();

    // rank inside the warp's 128 items: same id in earlier rounds (running count in shared memory,
    // touched by this warp only) + same id in earlier lanes of this round
    int in_warp[kItemsPerThread];
    const int ebits = key_bits(E);
    int* mine = warp_cnt + wid * E;
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        int e = ids[q];
        const bool valid = (unsigned)e < (unsigned)E;
        if (!valid) e = -1;
        const unsigned peers = same_key_lanes(e, ebits);
        const int leader = __ffs(peers) - 1;
        int old = 0;
        if (valid && lane == leader) {
            old = mine[e];
            mine[e] = old + __popc(peers);
        }
        old = __shfl_sync(0xffffffffu, old, leader);
        in_warp[q] = old + __popc(peers & lt);
        __syncwarp();
    }
    __syncthreads();
    // exclusive prefix over the 32 warps, per expert
    for (int x = tid; x < E; x += kLayoutThreads) {
        int running = 0;
#pragma unroll 8
        for (int w = 0; w < 32; ++w) {
            const int c = warp_cnt[w * E + x];
            warp_cnt[w * E + x] = running;
            running += c;
        }
    }
    __syncthreads();
    // Everything above only read the ids (complete before the counting kernel was allowed to start
    // us).  The tile prefixes and expert offsets below come from the counting kernel itself.
    griddep_wait();
    griddep_launch_dependents();
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        if (in_rank >= p.items_per_rank) continue;
        const long long item = rank_base + in_rank;
        const int e = ids[q];
        if ((unsigned)e < (unsigned)E) {
            int row;
            if (p.capacity > 0) {         // index inside the (expert, source rank) slot; dropped beyond the capacity
                const int idx = p.tile_cnt[(size_t)tile * E + e] - p.tile_cnt[(size_t)(r * p.tiles_per_rank) * E + e] +
                                mine[e] + in_warp[q];
                row = idx < p.capacity ? (e * p.R + r) * p.capacity + idx : -1;
            } else {
                row = p.expert_offset[e] + p.tile_cnt[(size_t)tile * E + e] + mine[e] + in_warp[q];
            }
            p.dst_row[item] = row;
            if (p.src_of_row && row >= 0) p.src_of_row[row] = (int32_t)item;
        } else {
            p.dst_row[item] = -1;
        }
    }
}

// ---- small and medium batches: the whole layout in one launch ---------------------------------
// One thread-block cluster (1 CTA up to 4,096 items, 8 CTAs up to 32,768: the decode shape has
// 16,384).  Warp w of CTA c owns a contiguous run of up to kSmallRounds*32 items, kept in registers
// between the counting pass and the ranking pass; all tables live in shared memory, and the CTAs
// of the cluster read each other's per-expert totals through distributed shared memory after one
// hardware cluster barrier.  Nothing goes through global memory between the passes and nothing spins.
constexpr int kSmallRounds = 4;
constexpr int kSmallItems = 32 * 32 * kSmallRounds;      // per CTA
constexpr int kLayoutCluster = 8;


#ifdef STRATA_LAYOUT_PROBE
#define LPROBE(k) do { if (threadIdx.x == 0) p.tile_cnt[1024 + blockIdx.x * 16 + (k)] = (int)(global_timer_ns() & 0x7fffffff); } while (0)
#else
#define LPROBE(k) do { } while (0)
#endif

// The two halves of a cluster barrier.  A CTA arrives as soon as it has finished reading the other
// CTAs' shared memory and waits only before it exits, so the barrier costs no idle time.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Threads that share the per-expert scan over the CTA's 32 warps: groups of E threads, each group
// taking a contiguous run of warps (at most 8 groups, so the second step reads at most 7 partial sums).
__host__ __device__ __forceinline__ int small_scan_groups(int E) { return max(1, min(8, kLayoutThreads / E)); }

__global__ void __launch_bounds__(kLayoutThreads) layout_cluster_kernel(LayoutParams p, int n_items)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int n_cta = (int)cluster.num_blocks(), cta = (int)cluster.block_rank();

    // warp_cnt[32*E] | offs[E+1] | cta_cnt[E] | all_cnt[E] | warp_sums[32] | total[2] | grp_sum[G*E] | grp_pre[G*E] | src_cnt[R*E]
    extern __shared__ int sm[];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int E = p.E;
    const int G = small_scan_groups(E), wpg = (32 + G - 1) / G;     // warps per scan group
    int* warp_cnt = sm;
    int* offs = sm + 32 * E;
    int* cta_cnt = offs + E + 1;          // this CTA's per-expert totals, read by the other CTAs of the cluster
    int* all_cnt = cta_cnt + E;           // cluster-wide per-expert counts (local copy)
    int* warp_sums = all_cnt + E;
    int* total = warp_sums + 32;
    int* grp_sum = total + 2;             // [G, E] items per (scan group, expert)
    int* grp_pre = grp_sum + G * E;       // [G, E] the same, as an exclusive prefix over the groups
    int* src_cnt = grp_pre + G * E;       // [R*E], only when src_expert_count is wanted
    int* mine = warp_cnt + wid * E;
    const int ebits = key_bits(E);

    // the tables do not depend on anything an earlier kernel wrote: clear them before the wait
    for (int x = tid; x < 32 * E; x += kLayoutThreads) warp_cnt[x] = 0;
    if (p.src_expert_count)
        for (int x = tid; x < p.R * E; x += kLayoutThreads) src_cnt[x] = 0;
    LPROBE(0);
    griddep_wait();
    LPROBE(1);
    griddep_launch_dependents();
    // contiguous run per warp over all warps of the cluster, a multiple of 32 items
    const int n_warps = 32 * n_cta;
    const int run = ((n_items + n_warps - 1) / n_warps + 31) / 32 * 32;
    const int first = (cta * 32 + wid) * run;

    int ids[kSmallRounds];
#pragma unroll
    for (int q = 0; q < kSmallRounds; ++q) {
        const int i = first + q * 32 + lane;
        ids[q] = (q * 32 < run && i < n_items) ? p.ids[i] : -1;
    }
    __syncthreads();
    LPROBE(2);

    // pass 1: per-warp counts, and for every item the number of same-id items in front of it inside its
    // warp's run (earlier rounds from the running count, earlier lanes from the lane mask); also the
    // per-source-rank counts, which are order independent
    int in_warp[kSmallRounds];
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int q = 0; q < kSmallRounds; ++q) {
        if (q * 32 >= run) break;
        const int i = first + q * 32 + lane;
        int e = ids[q];
        bool valid = i < n_items;
        if (valid && (unsigned)e >= (unsigned)E) {
            if (!(p.allow_unrouted && e == -1)) report_status(p.status, STRATA_ERR_BAD_EXPERT_ID);
            valid = false;
        }
        if (!valid) e = -1;
        ids[q] = e;
        const unsigned peers = same_key_lanes(e, ebits);
        const int lead_lane = __ffs(peers) - 1;
        const bool leader = valid && lane == lead_lane;
        int old = 0;
        if (leader) {
            old = mine[e];
            mine[e] = old + __popc(peers);
        }
        old = __shfl_sync(0xffffffffu, old, lead_lane);
        in_warp[q] = old + __popc(peers & lt);
        if (p.src_expert_count) {
            // Source rank relative to the rank of the round's first item: defined for every lane whether or
            // not its id is valid, and in [0, 31] because a round holds 32 consecutive items.
            const int r0 = (first + q * 32) / p.items_per_rank;
            const int rel = i / p.items_per_rank - r0;
            const unsigned all_same = __all_sync(0xffffffffu, rel == 0 || !valid);
            if (all_same) {
                if (leader) atomicAdd(&src_cnt[r0 * E + e], __popc(peers));
            } else {
                const unsigned peers2 = peers & same_key_lanes(rel, 5);
                if (valid && lane == __ffs(peers2) - 1) atomicAdd(&src_cnt[(r0 + rel) * E + e], __popc(peers2));
            }
        }
        __syncwarp();
    }
    __syncthreads();
    LPROBE(3);

    // exclusive prefix over this CTA's 32 warps per expert, in two steps: every scan group walks its own
    // run of warps, then the groups' sums are combined.  The totals go to cta_cnt for the cluster.
    const int sg = tid / E, se = tid - sg * E;
    if (sg < G) {
        int running = 0;
        const int w_end = min(32, (sg + 1) * wpg);
        for (int w = sg * wpg; w < w_end; ++w) {
            const int c = warp_cnt[w * E + se];
            warp_cnt[w * E + se] = running;
            running += c;
        }
        grp_sum[sg * E + se] = running;
    }
    __syncthreads();
    if (sg < G) {
        int before_g = 0, all_g = 0;
        for (int g2 = 0; g2 < G; ++g2) {
            const int v = grp_sum[g2 * E + se];
            if (g2 < sg) before_g += v;
            all_g += v;
        }
        grp_pre[sg * E + se] = before_g;
        if (sg == 0) cta_cnt[se] = all_g;
    }
    LPROBE(4);
    cluster.sync();                       // every CTA's cta_cnt and src_cnt are complete and visible
    LPROBE(5);

    // items with the same id in earlier CTAs of the cluster, and the cluster-wide count
    int before = 0, count_e = 0;
    if (tid < E) {
        int v[kLayoutCluster];
#pragma unroll
        for (int c = 0; c < kLayoutCluster; ++c) v[c] = c < n_cta ? *cluster.map_shared_rank(&cta_cnt[tid], c) : 0;
#pragma unroll
        for (int c = 0; c < kLayoutCluster; ++c) {
            if (c < cta) before += v[c];
            count_e += v[c];
        }
    }
    // the other remote reads (the per-source-rank table: CTA c sums its contiguous slice) go out before
    // the block scan, so that this CTA can tell the cluster early that it needs nobody's memory any more
    if (p.src_expert_count) {
        const int slice = (p.R * E + n_cta - 1) / n_cta;
        const int x_end = min(p.R * E, (cta + 1) * slice);
        for (int x = cta * slice + tid; x < x_end; x += kLayoutThreads) {
            int v[kLayoutCluster];
#pragma unroll
            for (int c = 0; c < kLayoutCluster; ++c)        // all remote reads in flight together
                v[c] = c < n_cta ? *cluster.map_shared_rank(&src_cnt[x], c) : 0;
            int sum = 0;
#pragma unroll
            for (int c = 0; c < kLayoutCluster; ++c) sum += v[c];
            p.src_expert_count[x] = sum;
        }
    }
    cluster_arrive();                     // matched by cluster_wait() before the exit
    const int padded = round_up_rows(count_e, p.align);
    const int off = block_exclusive_scan_1024(tid < E ? padded : 0, warp_sums, total);
    if (tid < E) {
        offs[tid] = off + before;         // first row of this CTA's items in each expert's segment
        all_cnt[tid] = count_e;
    }
    LPROBE(6);
    if (cta == 0) {
        if (tid < E) {
            p.expert_count[tid] = count_e;
            p.expert_offset[tid] = off;
            if (p.src_of_row)             // padding rows of this segment have no source item
                for (int row = off + count_e; row < off + padded; ++row) p.src_of_row[row] = -1;
            if (tid % p.e_loc == 0) p.rank_offset[tid / p.e_loc] = off;
        }
        if (tid == 0) {
            p.expert_offset[E] = *total;
            p.rank_offset[p.R] = *total;
        }
    }
    __syncthreads();
    if (cta == 0)
        for (int d = tid; d < p.R; d += kLayoutThreads) {
            int real = 0;
            for (int e2 = d * p.e_loc; e2 < (d + 1) * p.e_loc; ++e2) real += all_cnt[e2];
            p.rank_count[d] = real;
        }
    LPROBE(7);

    // pass 2: rows.  Everything an item needs is a table look-up away.
    const int* my_grp = grp_pre + (wid / wpg) * E;
#pragma unroll
    for (int q = 0; q < kSmallRounds; ++q) {
        if (q * 32 >= run) break;
        const int i = first + q * 32 + lane;
        const int e = ids[q];
        if (e >= 0) {
            const int row = offs[e] + my_grp[e] + mine[e] + in_warp[q];
            p.dst_row[i] = row;
            if (p.src_of_row) p.src_of_row[row] = i;
        } else if (i < n_items) {
            p.dst_row[i] = -1;
        }
    }
    LPROBE(8);
    cluster_wait();                       // no CTA leaves while another may still read its shared memory
    LPROBE(9);
}

// ---- fixed-capacity layout of small batches: one launch, one CTA per source rank ---------------
// In the [E][R][C] layout a row depends only on the items of the same source rank (the index of an
// item inside its (expert, rank) slot), and the offsets are constants, so the ranks are independent:
// CTA r counts and ranks the T*K <= 4096 items of rank r entirely in shared memory, fills its own
// slots of src_of_row (placed items and -1 for the empty rows), and leaves its clamped counts in the
// workspace; the CTA that draws the last ticket adds them up over the ranks.  Nothing waits.
__global__ void __launch_bounds__(kLayoutThreads) layout_capacity_kernel(LayoutParams p)
{
    extern __shared__ int sm[];          // warp_cnt[32*E] | kept[E]
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int E = p.E, C = p.capacity, r = blockIdx.x;
    int* warp_cnt = sm;
    int* kept = sm + 32 * E;
    int* mine = warp_cnt + wid * E;
    const int ebits = key_bits(E);
    const long long rank_base = (long long)r * p.items_per_rank;
    const int warp_first = wid * kWarpItems;

    for (int x = tid; x < 32 * E; x += kLayoutThreads) warp_cnt[x] = 0;
    griddep_wait();
    griddep_launch_dependents();
    int ids[kItemsPerThread];
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        ids[q] = in_rank < p.items_per_rank ? p.ids[rank_base + in_rank] : -1;
    }
    __syncthreads();

    // pass 1: per-warp counts
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        bool valid = in_rank < p.items_per_rank;
        int e = ids[q];
        if (valid && (unsigned)e >= (unsigned)E) {
            if (!(p.allow_unrouted && e == -1)) report_status(p.status, STRATA_ERR_BAD_EXPERT_ID);
            valid = false;
        }
        if (!valid) e = -1;
        ids[q] = e;
        const unsigned peers = same_key_lanes(e, ebits);
        if (valid && lane == __ffs(peers) - 1) mine[e] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    // exclusive prefix over the 32 warps per expert; the total is this rank's count for the expert
    for (int x = tid; x < E; x += kLayoutThreads) {
        int running = 0;
#pragma unroll 8
        for (int w = 0; w < 32; ++w) {
            const int c = warp_cnt[w * E + x];
            warp_cnt[w * E + x] = running;
            running += c;
        }
        const int k = min(running, C);
        if (running > C) report_status(p.status, STRATA_ERR_CAPACITY);       // items beyond the capacity are dropped
        kept[x] = k;
        p.tile_cnt[(size_t)r * E + x] = k;
        if (p.src_expert_count) p.src_expert_count[(size_t)r * E + x] = k;
    }
    __syncthreads();

    // pass 2: rows.  mine[e] counts the same-id items of earlier warps and earlier rounds of this rank.
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int q = 0; q < kItemsPerThread; ++q) {
        const int in_rank = warp_first + q * 32 + lane;
        const int e = ids[q];
        const bool valid = e >= 0;
        const unsigned peers = same_key_lanes(e, ebits);
        const int leader = __ffs(peers) - 1;
        int old = 0;
        if (valid && lane == leader) {
            old = mine[e];
            mine[e] = old + __popc(peers);
        }
        old = __shfl_sync(0xffffffffu, old, leader);
        if (valid) {
            const int idx = old + __popc(peers & lt);
            const int row = idx < C ? (e * p.R + r) * C + idx : -1;
            p.dst_row[rank_base + in_rank] = row;
            if (p.src_of_row && row >= 0) p.src_of_row[row] = (int32_t)(rank_base + in_rank);
        } else if (in_rank < p.items_per_rank) {
            p.dst_row[rank_base + in_rank] = -1;
        }
        __syncwarp();
    }
    // the empty rows of this rank's slots
    if (p.src_of_row)
        for (int x = tid; x < E * C; x += kLayoutThreads) {
            const int e = x / C, j = x - e * C;
            if (j >= kept[e]) p.src_of_row[(size_t)(e * p.R + r) * C + j] = -1;
        }

    // ---- last CTA to finish adds the ranks up (a ticket, never a wait) ----
    __shared__ int s_last;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(p.ticket, 1) == p.R - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    int* sum_e = warp_cnt;                // reused: [E]
    for (int x = tid; x < E; x += kLayoutThreads) {
        int sum = 0;
        for (int r0 = 0; r0 < p.R; r0 += 8) {
            int v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (r0 + i < p.R) ? __ldcg(p.tile_cnt + (size_t)(r0 + i) * E + x) : 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) sum += v[i];
        }
        sum_e[x] = sum;
        p.expert_count[x] = sum;
        p.expert_offset[x] = x * p.R * C;
    }
    if (tid == 0) {
        p.expert_offset[E] = E * p.R * C;
        p.rank_offset[p.R] = E * p.R * C;
    }
    __syncthreads();
    for (int d = tid; d < p.R; d += kLayoutThreads) {
        int real = 0;
        for (int e2 = d * p.e_loc; e2 < (d + 1) * p.e_loc; ++e2) real += sum_e[e2];
        p.rank_count[d] = real;
        p.rank_offset[d] = d * p.e_loc * p.R * C;
    }
    if (tid == 0) *p.ticket = 0;          // ready for the next call on this stream
}

// shared memory of the cluster kernel; the per-source-rank table is only there when asked for
size_t small_smem(int E, int R, bool with_src)
{
    return (size_t)(32 * E + E + 1 + E + E + 32 + 2 + 2 * small_scan_groups(E) * E + (with_src ? R * E : 0)) * sizeof(int);
}
constexpr size_t kSmallSmemLimit = 200 * 1024;

size_t count_scan_smem(int E)
{
    const int groups = max(1, kLayoutThreads / E);
    return (size_t)(groups * E + E + 1 + 32 + 2) * sizeof(int);
}

}  // namespace

cudaError_t configure_layout_kernels()
{
    cudaError_t err = cudaFuncSetAttribute(layout_rank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           32 * kMaxExperts * (int)sizeof(int));
    if (err != cudaSuccess) return err;
    err = cudaFuncSetAttribute(layout_capacity_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               33 * kMaxExperts * (int)sizeof(int));
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(layout_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)kSmallSmemLimit);
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
    p.align = s.segment_align > 1 ? s.segment_align : 1;
    p.allow_unrouted = (s.flags & STRATA_FLAG_ALLOW_UNROUTED) ? 1 : 0;
    p.capacity = s.slot_capacity > 0 ? s.slot_capacity : 0;

    const long long n_items = (long long)s.R * s.T * s.K;
    const size_t small_bytes = small_smem(s.E, s.R, L.src_expert_count != nullptr);
    // the fixed-capacity layout ranks items per source rank: its own one-launch kernel below when a rank
    // fits one tile, else the tiled path
    if (p.capacity == 0 && n_items <= (long long)kSmallItems * kLayoutCluster && small_bytes <= kSmallSmemLimit) {
        const unsigned n_cta = n_items <= kSmallItems ? 1u : (unsigned)kLayoutCluster;
        *n_launches = 1;
        return launch_pdl_cluster(layout_cluster_kernel, n_cta, kLayoutThreads, small_bytes, n_cta, st, p,
                                  (int)n_items);
    }
    if (p.capacity > 0 && g.tiles_per_rank == 1) {
        *n_launches = 1;
        return launch_pdl(layout_capacity_kernel, (unsigned)s.R, kLayoutThreads, (size_t)33 * s.E * sizeof(int), st, p);
    }
    *n_launches = 2;
    cudaError_t err = launch_pdl(layout_count_scan_kernel, (unsigned)g.n_tiles, kLayoutThreads, count_scan_smem(s.E), st, p);
    if (err != cudaSuccess) return err;
    return launch_pdl(layout_rank_kernel, (unsigned)g.n_tiles, kLayoutThreads, (size_t)32 * s.E * sizeof(int), st, p);
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
    const strata_status shape_rc = check_layout_shape(s);
    if (shape_rc != STRATA_OK) return shape_rc;
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
    p.align = s.segment_align > 1 ? s.segment_align : 1;
    p.allow_unrouted = (s.flags & STRATA_FLAG_ALLOW_UNROUTED) ? 1 : 0;
    p.capacity = s.slot_capacity > 0 ? s.slot_capacity : 0;
    layout_count_scan_kernel<<<g.n_tiles, kLayoutThreads, count_scan_smem(s.E), st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return STRATA_ERR_CUDA;
    layout_rank_kernel<<<g.n_tiles, kLayoutThreads, (size_t)32 * s.E * sizeof(int), st>>>(p);
    return cudaGetLastError() == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

