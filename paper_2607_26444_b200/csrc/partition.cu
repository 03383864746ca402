// Hierarchical workload partitioning for dispatch, the paper's own scheme (Sec. 6.2, App. B to D), as
// an optional work-assignment variant next to the default ordered work claiming:
//   level 2  expert-window aggregation: rows that source rank r sends to expert e are one contiguous
//            window of the receive buffer (win_base[r][e], src_expert_count[r][e] rows);
//   level 3  peer-window partitioning: the expert windows of (source r -> destination rank d),
//            concatenated in expert order, are cut into transfer units of at most S_t rows, t the tier
//            of (r,d); cost tau = alpha_t + ceil(bytes / beta_t);
//   policy   LPT-style list scheduling: units by decreasing cost onto the least-loaded core, and on that core
//            into the earliest issue stripe after its previous unit that still has room for the unit's
//            destination rank (fan-out cap H_t; a core issues at most one unit per stripe and may leave a
//            stripe empty, so the cap moves a unit to a later stripe, never to a busier core); the output is
//            one task list per core with the stripe of every entry.  The window-major dispatch kernel simply
//            follows the lists (CTAs do not synchronise per stripe on one GPU).
// The policy is generated ON the GPU by one CTA (no host round trip): a bitonic sort of the units and a
// greedy loop run by one warp, whose "least-loaded core" step is a warp-wide arg-min, with runs of
// equal-cost units handed out in closed-form rounds; then, only when a cap can bind (H_t below the number
// of cores), one sequential pass that gives every unit its stripe.
#include "common.cuh"

namespace strata {

namespace {

constexpr int kPartThreads = 1024;
constexpr int kPartMaxUnits = 8192;       // sort keys live in shared memory
constexpr int kPartMaxCores = 1024;       // core ids take 10 bits of the arg-min keys
constexpr int kFanSmemInts = 12288;       // fan-out counts F[stripe][dest] kept in shared memory
constexpr int kMaxTiers = 3;

struct PartitionParams {
    const int32_t* src_expert_count;   // [R,E]
    const int32_t* expert_offset;      // [E+1]
    int32_t* win_base;                 // [R,E]
    int32_t* unit_desc;                // [max_units,4]
    long long* unit_cost;              // [max_units]
    int32_t* n_units;                  // [1]
    int32_t* task_offset;              // [n_cores+1]
    int32_t* task_unit;                // [max_units]
    int32_t* task_stripe;              // [max_units]
    long long* core_load;              // [n_cores]
    int32_t* scratch;                  // [2*max_units + max_units*R]: core_of | pos_of | fan-out counts beyond shared memory
    int* status;
    int R, E, e_loc, n_cores, max_units, n_tiers, g0, g1;
    long long row_bytes;
    long long alpha[kMaxTiers], beta[kMaxTiers], unit_rows[kMaxTiers];
    int cap[kMaxTiers];
};

__device__ __forceinline__ int tier_of(const PartitionParams& p, int r, int d)
{
    const int t = (r / p.g0 == d / p.g0) ? 0 : (r / p.g1 == d / p.g1) ? 1 : 2;
    return min(t, p.n_tiers - 1);
}

// One CTA in the whole grid: tell the compiler so.  Left to its own heuristics it keeps the greedy loop's
// state in 54 registers and the lone warp's loop runs 30..70 % slower than with the 62 it takes here.
__global__ void __launch_bounds__(kPartThreads, 1) partition_kernel(PartitionParams p)
{
    extern __shared__ unsigned long long sm64[];
    unsigned long long* keys = sm64;                                   // [kPartMaxUnits] sort keys
    long long* load = reinterpret_cast<long long*>(keys + kPartMaxUnits);   // [kPartMaxCores]
    int* len = reinterpret_cast<int*>(load + kPartMaxCores);               // [kPartMaxCores]
    int* fan = len + kPartMaxCores;                                         // [kFanSmemInts]
    int* scan = fan + kFanSmemInts;                                         // [kPartThreads + 34]
    __shared__ int s_total;

    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int R = p.R, E = p.E;
    griddep_wait();
    griddep_launch_dependents();

    // ---- level 2: base row of every expert window ----
    for (int e = tid; e < E; e += kPartThreads) {
        int row = p.expert_offset[e];
        for (int r = 0; r < R; ++r) {
            p.win_base[r * E + e] = row;
            row += p.src_expert_count[r * E + e];
        }
    }

    // ---- level 3: units per peer window, exclusive scan over (r,d) in id order ----
    // R*R <= 4096 peer windows, up to 4 per thread, each thread's windows consecutive
    const int n_win = R * R;
    const int per_thread = (n_win + kPartThreads - 1) / kPartThreads;
    int my_units = 0;
    for (int i = 0; i < per_thread; ++i) {
        const int w = tid * per_thread + i;
        if (w < n_win) {
            const int r = w / R, d = w - r * R;
            long long B = 0;
            for (int e = d * p.e_loc; e < (d + 1) * p.e_loc; ++e) B += p.src_expert_count[r * E + e];
            const long long S = p.unit_rows[tier_of(p, r, d)];
            my_units += (int)((B + S - 1) / S);
        }
    }
    {   // block exclusive scan of my_units
        int inc = my_units;
#pragma unroll
        for (int dlt = 1; dlt < 32; dlt <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, dlt);
            if (lane >= dlt) inc += t;
        }
        if (lane == 31) scan[wid] = inc;
        __syncthreads();
        if (wid == 0) {
            const int s = scan[lane];
            int si = s;
#pragma unroll
            for (int dlt = 1; dlt < 32; dlt <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, si, dlt);
                if (lane >= dlt) si += t;
            }
            scan[lane] = si - s;
            if (lane == 31) s_total = si;
        }
        __syncthreads();
        my_units = scan[wid] + inc - my_units;     // now: first unit id of this thread's windows
    }
    const int U = s_total;
    if (U > p.max_units || U > kPartMaxUnits) {
        if (tid == 0) {
            report_status(p.status, STRATA_ERR_CAPACITY);
            *p.n_units = -1;
        }
        return;
    }
    // unit descriptors and costs
    {
        int j = my_units;
        for (int i = 0; i < per_thread; ++i) {
            const int w = tid * per_thread + i;
            if (w < n_win) {
                const int r = w / R, d = w - r * R;
                long long B = 0;
                for (int e = d * p.e_loc; e < (d + 1) * p.e_loc; ++e) B += p.src_expert_count[r * E + e];
                const int t = tier_of(p, r, d);
                const long long S = p.unit_rows[t];
                for (long long a = 0; a < B; a += S, ++j) {
                    const long long rows = min(S, B - a);
                    const long long cost = p.alpha[t] + (rows * p.row_bytes + p.beta[t] - 1) / p.beta[t];
                    p.unit_desc[j * 4 + 0] = r;
                    p.unit_desc[j * 4 + 1] = d;
                    p.unit_desc[j * 4 + 2] = (int)a;
                    p.unit_desc[j * 4 + 3] = (int)rows;
                    p.unit_cost[j] = cost;
                    // largest cost first, ties by lower unit id: ascending order of this key
                    keys[j] = ((unsigned long long)((1ll << 43) - 1 - cost) << 20) | (unsigned)j;
                }
            }
        }
    }
    int P = 1;
    while (P < U) P <<= 1;
    for (int j = U + tid; j < P; j += kPartThreads) keys[j] = ~0ull;
    for (int c = tid; c < p.n_cores; c += kPartThreads) {
        load[c] = 0;
        len[c] = 0;
    }
    for (int x = tid; x < kFanSmemInts; x += kPartThreads) fan[x] = 0;
    int* core_of = p.scratch;
    int* pos_of = p.scratch + p.max_units;             // position of a unit in its core's list
    int* fan_global = p.scratch + 2 * p.max_units;     // stripes beyond shared memory
    const int smem_stripes = kFanSmemInts / R;
    for (int x = tid; x < U * R; x += kPartThreads) fan_global[x] = 0;
    __syncthreads();

    // ---- bitonic sort of the keys ----
    for (int k = 2; k <= P; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < P; i += kPartThreads) {
                const int ixj = i ^ j;
                if (ixj > i) {
                    const unsigned long long a = keys[i], b = keys[ixj];
                    const bool up = (i & k) == 0;
                    if ((a > b) == up) {
                        keys[i] = b;
                        keys[ixj] = a;
                    }
                }
            }
            __syncthreads();
        }

    // After the sort every key is replaced by what the greedy loop needs, so that the loop touches
    // shared memory only: cost (37 bits) | destination rank (12) | unit id (13) | tier (2).
    {
        unsigned long long meta[kPartMaxUnits / kPartThreads];
#pragma unroll
        for (int i = 0; i < kPartMaxUnits / kPartThreads; ++i) {
            const int o = tid + i * kPartThreads;
            if (o < U) {
                const int j = (int)(keys[o] & 0xfffffu);
                const int r = p.unit_desc[j * 4 + 0], d = p.unit_desc[j * 4 + 1];
                meta[i] = ((unsigned long long)p.unit_cost[j] << 27) | ((unsigned long long)d << 15) |
                          ((unsigned long long)j << 2) | (unsigned)tier_of(p, r, d);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kPartMaxUnits / kPartThreads; ++i) {
            const int o = tid + i * kPartThreads;
            if (o < U) keys[o] = meta[i];
        }
        __syncthreads();
    }

    // ---- list scheduling: one warp, one unit per iteration; lane l speaks for cores l, l+32, ... ----
    // The loop is sequential in the units and a lone warp pays full ALU latency on every dependent
    // instruction, so the arithmetic is kept narrow: while every core's load fits 21 bits the key
    // (load | core) is one 32-bit word and the arg-min is one redux instruction; the first load that
    // would not fit switches the rest of the run to 64-bit keys.
    if (wid == 0) {
        // slots past the last core (the table is padded to a multiple of 128) hold all ones and can never win
        unsigned int* st32 = reinterpret_cast<unsigned int*>(scan);        // [kPartMaxCores] (scan[] is free here)
        const int padded = (p.n_cores + 127) / 128 * 128;
        for (int c = lane; c < padded; c += 32) st32[c] = c < p.n_cores ? 0u : 0xffffffffu;
        __syncwarp();
        int o = 0;
        // The core of a unit does not depend on the fan-out cap, so no fan-out table is consulted here: a
        // core's key changes only when the core wins, and every lane keeps its own cores' keys in registers
        // (up to 384 cores; beyond, the lane minimum): a unit costs one min tree, one redux and the winner's
        // update, about 0.2 us per unit measured on B200.
        {
            // here st32[c] is the key itself, load << 10 | core, and the list lengths live in len[]
            for (int c = lane; c < padded; c += 32) {
                st32[c] = c < p.n_cores ? (unsigned)c : 0xffffffffu;
                if (c < p.n_cores) len[c] = 0;
            }
            __syncwarp();
            auto lane_min = [&]() {
                unsigned int m0 = 0xffffffffu, m1 = 0xffffffffu, m2 = 0xffffffffu, m3 = 0xffffffffu;
                for (int c = lane; c < padded; c += 128) {       // padded is a multiple of 128
                    m0 = min(m0, st32[c]);
                    m1 = min(m1, st32[c + 32]);
                    m2 = min(m2, st32[c + 64]);
                    m3 = min(m3, st32[c + 96]);
                }
                return min(min(m0, m1), min(m2, m3));
            };
            unsigned long long m = U > 0 ? keys[0] : 0ull;
            if (padded <= 384) {
                // up to 12 cores per lane: their keys stay in registers, the winner's rescan is a min tree
                unsigned int k[12];
#pragma unroll
                for (int i = 0; i < 12; ++i) k[i] = lane + 32 * i < padded ? st32[lane + 32 * i] : 0xffffffffu;
                // Units of equal cost come in long runs (all full-size units of a tier).  For such a run the
                // greedy choice has a closed form per round: after the least-loaded core (key K0) takes a unit
                // its key becomes T = K0 + cost, and every updated key is >= T, so the next picks are exactly
                // the cores whose keys are below T, once each, in key order.  A round hands out that many units
                // at once (each lane ranks its selected cores against all keys); short runs, rounds that would
                // select few cores and everything else go one unit at a time.
                int run_end = 0;                 // first index past the run of equal costs that contains o
                while (o < U) {
                    m = keys[o];
                    const unsigned long long cost64 = m >> 27;
                    const unsigned int cost = (unsigned int)min(cost64, (unsigned long long)0x7fffffffu);
                    if (o >= run_end) {
                        for (int t = o;; t += 32) {
                            const int idx = t + lane;
                            const bool eq = idx < U && (keys[idx] >> 27) == cost64;
                            const unsigned int b = __ballot_sync(0xffffffffu, eq);
                            if (b != 0xffffffffu) {
                                run_end = t + __ffs(~b) - 1;
                                break;
                            }
                        }
                    }
                    const unsigned int mine = min(min(min(k[0], k[1]), min(k[2], k[3])), min(min(min(k[4], k[5]), min(k[6], k[7])),
                                                                                             min(min(k[8], k[9]), min(k[10], k[11]))));
                    const unsigned int best = __reduce_min_sync(0xffffffffu, mine);
                    const unsigned int new_load = (best >> 10) + cost;
                    if (new_load >= (1u << 21)) break;
                    const int left = run_end - o;
                    if (left >= 32 && cost > 0 && new_load + cost < (1u << 21)) {
                        const unsigned int T = best + (cost << 10);
                        int n_sel = 0;
#pragma unroll
                        for (int i = 0; i < 12; ++i) n_sel += k[i] < T ? 1 : 0;
                        const int k_total = (int)__reduce_add_sync(0xffffffffu, (unsigned)n_sel);
                        if (k_total >= 32) {
#pragma unroll
                            for (int i = 0; i < 12; ++i)
                                if (lane + 32 * i < padded) st32[lane + 32 * i] = k[i];
                            __syncwarp();
                            const int take = min(k_total, left);
                            // rank of each of this lane's keys among all keys: one pass over the table, the
                            // twelve counters packed three to a register (a rank is below 2^10)
                            unsigned int rk[4] = {0u, 0u, 0u, 0u};
#pragma unroll 4
                            for (int c = 0; c < padded; ++c) {
                                const unsigned int v = st32[c];
#pragma unroll
                                for (int i = 0; i < 12; ++i) rk[i / 3] += (v < k[i] ? 1u : 0u) << (10 * (i % 3));
                            }
#pragma unroll
                            for (int i = 0; i < 12; ++i) {
                                const int rank = (int)((rk[i / 3] >> (10 * (i % 3))) & 1023u);
                                if (k[i] < T && rank < take) {
                                    const int core = lane + 32 * i;
                                    const int j = (int)((keys[o + rank] >> 2) & 0x1fffu);
                                    const int kk = len[core];
                                    core_of[j] = core;
                                    pos_of[j] = kk;
                                    len[core] = kk + 1;
                                    k[i] += cost << 10;
                                }
                            }
                            __syncwarp();
                            o += take;
                            continue;
                        }
                    }
                    const int win = (int)(best & 1023u);
                    const int j = (int)((m >> 2) & 0x1fffu);
                    if (lane == (win & 31)) {
                        const unsigned int nk = (new_load << 10) | (unsigned)win;
                        const int slot = win >> 5;
#pragma unroll
                        for (int i = 0; i < 12; ++i)
                            if (i == slot) k[i] = nk;
                        const int kk = len[win];
                        core_of[j] = win;
                        pos_of[j] = kk;
                        len[win] = kk + 1;
                    }
                    ++o;
                }
                if (o < U) m = keys[o];
#pragma unroll
                for (int i = 0; i < 12; ++i)
                    if (lane + 32 * i < padded) st32[lane + 32 * i] = k[i];
            }
            unsigned int my_min = lane_min();
            for (; o < U; ++o) {
                const unsigned long long m_next = o + 1 < U ? keys[o + 1] : 0ull;
                const unsigned int cost = (unsigned int)min(m >> 27, (unsigned long long)0x7fffffffu);
                const int j = (int)((m >> 2) & 0x1fffu);
                const unsigned int best = __reduce_min_sync(0xffffffffu, my_min);
                const int win = (int)(best & 1023u);
                const unsigned int new_load = (best >> 10) + cost;
                if (new_load >= (1u << 21)) break;                  // the wide loop below takes over
                if (lane == (win & 31)) {
                    const int kk = len[win];
                    core_of[j] = win;
                    pos_of[j] = kk;
                    len[win] = kk + 1;
                    st32[win] = (new_load << 10) | (unsigned)win;
                    my_min = lane_min();
                }
                m = m_next;
            }
            __syncwarp();
            for (int c = lane; c < p.n_cores; c += 32) load[c] = (long long)(st32[c] >> 10);
        }
        __syncwarp();
        const int cores_per_lane_w = (p.n_cores + 31) / 32;
        for (; o < U; ++o) {                        // wide keys: load << 10 | core in 64 bits (load < 2^53)
            const unsigned long long m = keys[o];
            const long long cost = (long long)(m >> 27);
            const int j = (int)((m >> 2) & 0x1fffu);
            unsigned long long best = ~0ull;
            for (int i = 0; i < cores_per_lane_w; ++i) {
                const int c = lane + 32 * i;
                if (c < p.n_cores) best = min(best, ((unsigned long long)load[c] << 10) | (unsigned)c);
            }
#pragma unroll
            for (int dlt = 16; dlt > 0; dlt >>= 1) {
                const unsigned lo = __shfl_xor_sync(0xffffffffu, (unsigned)best, dlt);
                const unsigned hi = __shfl_xor_sync(0xffffffffu, (unsigned)(best >> 32), dlt);
                best = min(best, ((unsigned long long)hi << 32) | lo);
            }
            const int win = (int)(best & 1023u);
            if (lane == (win & 31)) {
                const int kk = len[win];
                core_of[j] = win;
                pos_of[j] = kk;
                len[win] = kk + 1;
                load[win] += cost;
            }
            __syncwarp();
        }
    }
    __syncthreads();

    // ---- per-core task lists in issue order ----
    {
        const int v = tid < p.n_cores ? len[tid] : 0;
        int inc = v;
#pragma unroll
        for (int dlt = 1; dlt < 32; dlt <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, dlt);
            if (lane >= dlt) inc += t;
        }
        if (lane == 31) scan[wid] = inc;
        __syncthreads();
        if (wid == 0) {
            const int s = scan[lane];
            int si = s;
#pragma unroll
            for (int dlt = 1; dlt < 32; dlt <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, si, dlt);
                if (lane >= dlt) si += t;
            }
            scan[lane] = si - s;
        }
        __syncthreads();
        const int off = scan[wid] + inc - v;
        if (tid < p.n_cores) {
            p.task_offset[tid] = off;
            p.core_load[tid] = load[tid];
            scan[34 + tid] = off;              // scan[] has room for kPartThreads + 34 ints
        }
        if (tid == 0) {
            p.task_offset[p.n_cores] = U;
            *p.n_units = U;
        }
        __syncthreads();
        for (int j = tid; j < U; j += kPartThreads) p.task_unit[scan[34 + core_of[j]] + pos_of[j]] = j;
    }

    // ---- issue stripes ----
    // A stripe holds at most one unit per core, so a cap of n_cores or more can never bind: the stripe of a
    // unit is then its position in the list.
    bool cap_binds = false;
    for (int t = 0; t < p.n_tiers; ++t) cap_binds = cap_binds || p.cap[t] < p.n_cores;
    if (!cap_binds) {
        for (int j = tid; j < U; j += kPartThreads) p.task_stripe[scan[34 + core_of[j]] + pos_of[j]] = pos_of[j];
        return;
    }
    // Otherwise the stripes follow from one pass over the units in list-scheduling order (keys[] still holds
    // it): a unit takes the earliest stripe at or after its core's next free one in which fewer than H_t units
    // target its destination.  The walk is sequential (F[stripe][d] and the cores' next stripes evolve with
    // every unit), so one lane does it; the other lanes fetch the next 32 units' cores and list slots.  A
    // stripe below the highest one in use is never empty, so no stripe index reaches U.
    __syncthreads();
    if (wid != 0) return;
    for (int c = lane; c < p.n_cores; c += 32) len[c] = 0;     // from here on: the first stripe the core may use
    __syncwarp();
    for (int o0 = 0; o0 < U; o0 += 32) {
        const int o = o0 + lane;
        const unsigned long long m = o < U ? keys[o] : 0ull;
        const int j = (int)((m >> 2) & 0x1fffu);
        const int my_d = (int)((m >> 15) & 0xfffu);
        const int my_cap = (m & 3u) == 0 ? p.cap[0] : (m & 3u) == 1 ? p.cap[1] : p.cap[2];
        const int my_core = o < U ? core_of[j] : 0;
        const int my_slot = o < U ? scan[34 + my_core] + pos_of[j] : 0;
        const int n = min(32, U - o0);
        for (int i = 0; i < n; ++i) {
            const int core = __shfl_sync(0xffffffffu, my_core, i), d = __shfl_sync(0xffffffffu, my_d, i);
            const int cap = __shfl_sync(0xffffffffu, my_cap, i), slot = __shfl_sync(0xffffffffu, my_slot, i);
            if (lane == 0) {
                int k = len[core];
                for (;; ++k) {
                    const int f = k < smem_stripes ? fan[k * R + d] : fan_global[(size_t)k * R + d];
                    if (f < cap) break;
                }
                if (k < smem_stripes) fan[k * R + d] += 1;
                else fan_global[(size_t)k * R + d] += 1;
                len[core] = k + 1;
                p.task_stripe[slot] = k;
            }
        }
    }
}

constexpr size_t kPartSmem = (size_t)kPartMaxUnits * 8 + (size_t)kPartMaxCores * 8 + (size_t)kPartMaxCores * 4 +
                             (size_t)kFanSmemInts * 4 + (size_t)(kPartThreads + 34) * 4;

// ---- window-major dispatch: every CTA follows its task list ---------------------------------
constexpr int kWinStages = 4;
constexpr uint32_t kWinMaxRowBytes = 16384;

struct WindowsParams {
    const int32_t* src_expert_count;
    const int32_t* win_base;
    const int32_t* unit_desc;
    const int32_t* task_offset;
    const int32_t* task_unit;
    const int32_t* src_of_row;
    const unsigned char* x;
    unsigned char* recv;
    const int32_t* n_units;
    long long capacity_rows, n_tok;
    int R, E, e_loc, K, H;
    int* status;
    TraceBuf trace;
};

// One warp per core.  Rows are produced in batches of 32 (receive-row ids by lane 0 walking the task
// list, their source tokens by all lanes from src_of_row), then lane 0 runs them through a ring of
// stages: bulk load of the source row, then a bulk store to the receive row.  Ring protocol, with
// `issued` loads and `stored` stores so far: never more than stages-1 loaded rows wait for their
// store; before a stage is reloaded, wait_group.read<1> retires every store but the newest, which
// includes the one that last read this stage.
__global__ void __launch_bounds__(32) dispatch_windows_kernel(WindowsParams p)
{
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t row_bytes = (uint32_t)p.H * 2u;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kWinStages * row_bytes);
    __shared__ int s_row[32];
    __shared__ int s_dst[kWinStages];          // receive row of the load held by each stage
    const int lane = threadIdx.x;
    const int core = blockIdx.x;

    if (lane == 0) {
        for (int s = 0; s < kWinStages; ++s) mbar_init(&bars[s], 1);
        mbar_fence_init();
    }
    __syncwarp();
    const uint64_t pol = policy_evict_first();
    griddep_wait();
    griddep_launch_dependents();
    if (lane == 0) trace_begin(p.trace);
    Timeline tl(p.trace, STRATA_KERNEL_DISPATCH_WINDOWS, lane == 0);
    tl.begin(STRATA_STAGE_KERNEL);

    // lane 0 only: store the oldest loaded row
    long long issued = 0, stored = 0;
    auto store_oldest = [&]() -> bool {
        const int s = (int)(stored % kWinStages);
        if (!mbar_wait_bounded(&bars[s], (uint32_t)((stored / kWinStages) & 1))) return false;
        bulk_s2g(p.recv + (size_t)s_dst[s] * row_bytes, smem + (size_t)s * row_bytes, row_bytes);
        bulk_commit();
        ++stored;
        return true;
    };

    // cursor over this core's rows (lane 0)
    int q = p.task_offset[core];
    const int q_end = p.task_offset[core + 1];
    int r = 0, e = 0, e_end = 0, first = 0, rows_left = 0;
    const int n_units_total = *p.n_units;
    bool ok = true;

    while (ok) {
        // ---- next batch of up to 32 receive rows ----
        int n = 0;
        if (lane == 0) {
            while (n < 32) {
                if (rows_left == 0) {
                    if (q >= q_end) break;
                    const int j = p.task_unit[q++];
                    if (j < 0 || j >= n_units_total) {          // a task list that names no unit of this partition
                        report_status(p.status, STRATA_ERR_INVALID_ARG);
                        q = q_end;
                        break;
                    }
                    r = p.unit_desc[j * 4 + 0];
                    const int d = p.unit_desc[j * 4 + 1];
                    first = p.unit_desc[j * 4 + 2];
                    rows_left = p.unit_desc[j * 4 + 3];
                    if (r < 0 || r >= p.R || d < 0 || d >= p.R || first < 0 || rows_left < 0) {
                        report_status(p.status, STRATA_ERR_INVALID_ARG);
                        rows_left = 0;
                        q = q_end;
                        break;
                    }
                    e = d * p.e_loc;
                    e_end = e + p.e_loc;
                }
                int cnt = p.src_expert_count[r * p.E + e];
                while (first >= cnt && e + 1 < e_end) {     // expert windows in front of the first logical row
                    first -= cnt;
                    ++e;
                    cnt = p.src_expert_count[r * p.E + e];
                }
                const int take = min(min(cnt - first, rows_left), 32 - n);
                if (take <= 0) {                            // inconsistent lists: report, never loop forever
                    report_status(p.status, STRATA_ERR_INVALID_ARG);
                    rows_left = 0;
                    q = q_end;
                    break;
                }
                const int base = p.win_base[r * p.E + e] + first;
                for (int i = 0; i < take; ++i) s_row[n + i] = base + i;
                n += take;
                first += take;
                rows_left -= take;
            }
        }
        n = __shfl_sync(0xffffffffu, n, 0);
        if (n == 0) break;
        __syncwarp();
        const int my_row = lane < n ? s_row[lane] : -1;
        const bool row_ok = my_row >= 0 && my_row < p.capacity_rows;
        const int my_src = row_ok ? p.src_of_row[my_row] : -1;      // -1: a padding or empty row has no source item
        long long my_tok = my_src >= 0 ? (long long)my_src / p.K : -1;
        if (lane < n && (my_tok < 0 || my_tok >= p.n_tok)) {
            report_status(p.status, STRATA_ERR_BAD_ROW);
            my_tok = -1;
        }
        // ---- run the batch through the ring ----
        for (int i = 0; i < n; ++i) {
            const int row = __shfl_sync(0xffffffffu, my_row, i);
            const long long tok = __shfl_sync(0xffffffffu, my_tok, i);
            if (lane == 0 && tok >= 0 && ok) {
                if (issued - stored == kWinStages - 1) ok = store_oldest();
                if (ok) {
                    if (issued >= kWinStages) bulk_wait_read<1>();
                    const int s = (int)(issued % kWinStages);
                    s_dst[s] = row;
                    mbar_expect_tx(&bars[s], row_bytes);
                    bulk_g2s(smem + (size_t)s * row_bytes, p.x + (size_t)tok * row_bytes, row_bytes, &bars[s], pol);
                    ++issued;
                }
            }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
        __syncwarp();
    }
    if (lane == 0) {
        while (ok && stored < issued) ok = store_oldest();
        if (!ok) report_status(p.status, STRATA_ERR_TIMEOUT);
        bulk_wait_read<0>();
        trace_end(p.trace);
        tl.end(STRATA_STAGE_KERNEL);
        tl.finish();
    }
}

}  // namespace

cudaError_t configure_partition_kernels()
{
    cudaError_t err =
        cudaFuncSetAttribute(partition_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPartSmem);
    if (err != cudaSuccess) return err;
    return cudaFuncSetAttribute(dispatch_windows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kWinStages * (int)kWinMaxRowBytes + 64);
}

cudaError_t launch_partition(const strata_moe_shape& s, const strata_moe_layout_t& L,
                             const strata_partition_policy& pol, int n_cores, const strata_partition_t& out,
                             size_t max_units, int* status, cudaStream_t st)
{
    PartitionParams p{};
    p.src_expert_count = L.src_expert_count;
    p.expert_offset = L.expert_offset;
    p.win_base = out.win_base;
    p.unit_desc = out.unit_desc;
    p.unit_cost = reinterpret_cast<long long*>(out.unit_cost);
    p.n_units = out.n_units;
    p.task_offset = out.task_offset;
    p.task_unit = out.task_unit;
    p.task_stripe = out.task_stripe;
    p.core_load = reinterpret_cast<long long*>(out.core_load);
    p.scratch = out.scratch;
    p.status = status;
    p.R = s.R;
    p.E = s.E;
    p.e_loc = s.E / s.R;
    p.n_cores = n_cores;
    p.max_units = (int)max_units;
    p.n_tiers = pol.n_tiers;
    p.g0 = pol.g0;
    p.g1 = pol.g1;
    p.row_bytes = (long long)s.H * 2;
    for (int t = 0; t < pol.n_tiers; ++t) {
        p.alpha[t] = pol.tiers[t].alpha;
        p.beta[t] = pol.tiers[t].beta;
        p.unit_rows[t] = pol.tiers[t].unit_rows;
        p.cap[t] = pol.tiers[t].fanout_cap;
    }
    return launch_pdl(partition_kernel, 1, kPartThreads, kPartSmem, st, p);
}

cudaError_t launch_dispatch_windows(const strata_moe_shape& s, const strata_moe_layout_t& L,
                                    const strata_partition_t& part, int n_cores, const void* x, void* recv,
                                    size_t capacity_rows, int* status, TraceBuf trace, cudaStream_t st)
{
    WindowsParams p{};
    p.src_expert_count = L.src_expert_count;
    p.win_base = part.win_base;
    p.unit_desc = part.unit_desc;
    p.task_offset = part.task_offset;
    p.task_unit = part.task_unit;
    p.src_of_row = L.src_of_row;
    p.n_units = part.n_units;
    p.x = static_cast<const unsigned char*>(x);
    p.recv = static_cast<unsigned char*>(recv);
    p.capacity_rows = (long long)capacity_rows;
    p.n_tok = (long long)s.R * s.T;
    p.R = s.R;
    p.E = s.E;
    p.e_loc = s.E / s.R;
    p.K = s.K;
    p.H = s.H;
    p.status = status;
    p.trace = trace;
    const size_t smem = (size_t)kWinStages * s.H * 2 + 64;
    return launch_plain(dispatch_windows_kernel, (unsigned)n_cores, 32, smem, st, p);
}

int partition_max_units_supported() { return kPartMaxUnits; }
int partition_max_cores_supported() { return kPartMaxCores; }
uint32_t windows_max_row_bytes() { return kWinMaxRowBytes; }

}  // namespace strata
