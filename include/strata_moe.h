/*
 * strata_moe.h -- C ABI of the B200 (sm_100a) MoE routing-layout / token-dispatch /
 * gate-weighted-combine library.
 *
 * Conventions for every function
 *  - Returns a strata_status.  Nothing throws, traps, asserts or aborts.
 *  - "device pointer" = address in the memory of the context's GPU; "host
 *    pointer" = ordinary process memory.  All data buffers belong to the
 *    caller; the library owns only the opaque host-side strata_ctx and never
 *    allocates or frees device memory.
 *  - The three moe calls enqueue kernels on the given CUDA stream
 *    (a cudaStream_t passed as void*; NULL = the legacy default stream) and
 *    return without synchronising.  Errors that can be seen on the host
 *    (NULL pointer, shape, alignment, unregistered receive buffer, capacity)
 *    are returned before anything is launched.  Errors that only the device
 *    can see (an expert id outside [0,E), a destination row outside the
 *    receive buffer, a bounded wait that ran out) set a device status word
 *    (first error wins), the offending item is skipped, nothing is accessed
 *    out of bounds, and the error is reported by strata_device_status().
 *  - One context serves one stream of work: its calls must reach the GPU in the order they were
 *    made (issue them to one stream, or order the streams yourself).  The workspace holds state
 *    that consecutive launches hand to each other (work-claim counters, the layout ticket, the
 *    status word); two calls on the same context whose kernels could overlap would corrupt it.
 *    Use one context per concurrent stream.
 *  - Index convention: rank r in [0,R), token t in [0,T), slot k in [0,K);
 *    flat item i = (r*T + t)*K + k; token n = r*T + t; N = R*T*K.
 *    Expert e belongs to rank e / (E/R).  All R ranks are partitions of one
 *    GPU's memory.
 *  - bf16 tensors are row-major arrays of 16-bit patterns.
 */
#ifndef STRATA_MOE_H
#define STRATA_MOE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STRATA_OK = 0,
    STRATA_ERR_INVALID_ARG = 1,    /* NULL or otherwise unusable argument            */
    STRATA_ERR_SHAPE = 2,          /* shape outside what the kernels support          */
    STRATA_ERR_ALIGNMENT = 3,      /* a data pointer is not 16-byte aligned           */
    STRATA_ERR_NOT_REGISTERED = 4, /* receive buffer not inside a registered region   */
    STRATA_ERR_CAPACITY = 5,       /* receive buffer / region / workspace too small   */
    STRATA_ERR_BAD_EXPERT_ID = 6,  /* device: an id outside [0,E) was skipped         */
    STRATA_ERR_WORKSPACE = 7,      /* no workspace set on the context                 */
    STRATA_ERR_CUDA = 8,           /* a CUDA runtime call failed                      */
    STRATA_ERR_TIMEOUT = 9,        /* device: a bounded wait ran out                  */
    STRATA_ERR_BAD_ROW = 10        /* device: a destination row outside the buffer    */
} strata_status;

typedef enum {
    STRATA_BF16 = 0,               /* dispatch copies bf16 rows bit for bit           */
    STRATA_FP8_E4M3_B128 = 1       /* dispatch quantises to e4m3, one fp32 scale per
                                      token per block of 128 columns                  */
} strata_dtype;

/* Problem shape.  Requirements: R,T,H,E,K > 0; E % R == 0; E <= 1024; K <= 32;
 * H % 8 == 0 (rows are whole 16-byte vectors); H % 128 == 0 for FP8;
 * R*T*K + E*(segment_align-1) < 2^31.
 * Two production variants of the layout (zero = off, the packed strict layout):
 *  segment_align A > 1: every expert segment starts at a multiple of A rows (what a grouped GEMM
 *    with A-row tiles wants): expert_offset[e+1] = round_up(expert_offset[e] + expert_count[e], A).
 *    Rows between a segment's end and the next start are padding: dispatch never writes them and
 *    src_of_row is -1 there.  rank_offset follows the padded offsets, rank_count and expert_count
 *    stay the numbers of real rows.  The receive buffer needs strata_moe_recv_rows() rows.
 *  STRATA_FLAG_ALLOW_UNROUTED: an id of -1 means "not routed" (dropped token slot): dst_row = -1,
 *    counted nowhere, skipped by dispatch, contributes nothing in combine, and is not an error.
 *  slot_capacity C > 0: fixed-capacity layout, a receive buffer of static shape [E][R][C] rows for the
 *    low-latency mode (pairs with CUDA-graph replay; excludes segment_align).  The j-th item, in
 *    (token, slot) order, that source rank r sends to expert e lands in row (e*R + r)*C + j if j < C;
 *    otherwise it is dropped (dst_row = -1) and STRATA_ERR_CAPACITY is raised on the device status.
 *    Counts are the rows present: src_expert_count[r][e] = min(count, C), expert_count[e] their sum,
 *    expert_offset[e] = e*R*C, rank_offset[d] = d*(E/R)*R*C; src_of_row is -1 on empty rows.  The
 *    window-partitioning calls do not support this layout. */
#define STRATA_FLAG_ALLOW_UNROUTED 1
typedef struct {
    int32_t R, T, H, E, K;
    int32_t dispatch_dtype;        /* a strata_dtype */
    int32_t segment_align;         /* rows; 0 or 1 = packed segments; at most 65536 */
    int32_t flags;                 /* STRATA_FLAG_* */
    int32_t slot_capacity;         /* rows per (expert, source rank) slot; 0 = packed/aligned segments */
} strata_moe_shape;

typedef struct strata_ctx strata_ctx;   /* opaque, host side */

/* Routing metadata (paper App. D, "token placement": destination expert,
 * per-expert counts, prefix-sum offsets, token-local offsets), produced by
 * strata_moe_layout and consumed by dispatch and combine.  All members are
 * device pointers to int32 arrays owned by the caller. */
typedef struct {
    int32_t *expert_count;      /* [E]    items routed to expert e                       */
    int32_t *expert_offset;     /* [E+1]  exclusive scan; segment e = rows [off[e],off[e+1]) */
    int32_t *rank_count;        /* [R]    rows received by rank d                        */
    int32_t *rank_offset;       /* [R+1]  rank d's partition = rows [off[d],off[d+1])    */
    int32_t *src_expert_count;  /* [R,E]  items of source rank r routed to e; may be NULL */
    int32_t *dst_row;           /* [R,T,K] receive row of item i (-1 for a skipped or unrouted item) */
    int32_t *src_of_row;        /* [strata_moe_recv_rows] inverse of dst_row, -1 on padding rows; may be NULL */
} strata_moe_layout_t;

const char *strata_status_string(strata_status s);

/* ---- context ------------------------------------------------------------ */

/* Creates a context for one shape on CUDA device `device` (made current for the
 * duration of each call).  Host errors: INVALID_ARG, SHAPE, CUDA.
 * device = -1 creates a host-only context: the pool and all argument validation
 * work as usual (pointers are recorded, never dereferenced), and every call that
 * would launch or touch device memory returns STRATA_ERR_CUDA instead.  It
 * computes nothing; it exists so that host logic can be exercised without a GPU. */
strata_status strata_ctx_create(strata_ctx **out, const strata_moe_shape *shape, int device);
strata_status strata_ctx_destroy(strata_ctx *ctx);

/* Scratch memory the kernels need for this shape (the device status word, a ticket
 * and work-claim counters, the layout's per-tile histograms, and 24.8 KB for the pair
 * table of strata_alltoallv).  The caller allocates at least `bytes`
 * bytes of device memory, 256-byte aligned, and hands it over with
 * strata_ctx_set_workspace, which zeroes it (synchronously).  It must stay
 * valid and unshared while calls on this context are in flight. */
strata_status strata_moe_workspace_bytes(const strata_moe_shape *shape, size_t *bytes);
/* Rows the receive buffer (and src_of_row) must hold: R*T*K + E*(segment_align-1), the worst case of
 * the padded layout (R*T*K for packed segments), or E*R*slot_capacity for the fixed-capacity layout.
 * Host arithmetic only. */
strata_status strata_moe_recv_rows(const strata_moe_shape *shape, size_t *rows);
strata_status strata_ctx_set_workspace(strata_ctx *ctx, void *dptr, size_t bytes);

/* Number of kernels this context has launched so far (for accounting). */
strata_status strata_ctx_launch_count(strata_ctx *ctx, uint64_t *count);

/* SM budget.  Dispatch, combine and the collectives run as persistent grids sized for the whole GPU
 * (a fixed number of CTAs per SM).  n_sm > 0 sizes them for n_sm SMs instead, so that a compute kernel
 * running beside them on another stream keeps the rest (the paper's Sec. 3.2 observation that a fraction
 * of the cores saturates the fabric, and its Sec. 6.3 aim of freeing cores for computation); 0 restores
 * the default, values above the device's SM count are clamped.  The budget bounds the number of CTAs,
 * it does not pin them to particular SMs.  Results do not depend on it.  The layout kernels are not
 * affected. */
strata_status strata_ctx_set_sm_budget(strata_ctx *ctx, int32_t n_sm);

/* A promise about the caller's stream order that lets dispatch start earlier (paper Sec. 5.2 / 6.2 want the
 * transfer issued as soon as its operands exist; the paper defines no such call).  In an MoE layer the hidden
 * states x exist before routing starts, while dispatch is enqueued right behind the layout call.  on != 0
 * promises, for every later strata_moe_dispatch on this context: the x passed to it is complete before the
 * operation that directly precedes that dispatch call in its stream STARTS, and nothing writes x until the
 * dispatch has finished.  Dispatch, which is launched so that its prologue overlaps the preceding kernel, then
 * loads its first rows of x while that kernel (normally the layout) is still running; only its stores wait for
 * the layout.  Measured at the decode shape: 1.5 us off a 90 us step.  Off (0) by default: without the promise
 * dispatch reads x only after everything before it in the stream has finished.  A broken promise yields stale
 * rows, never an out-of-bounds access.  strata_moe_roundtrip_host never uses it. */
strata_status strata_ctx_set_x_early(strata_ctx *ctx, int32_t on);

/* Per-CTA stage probes (after the paper's in-kernel profiler, Sec. 6.4: probes at stage boundaries
 * writing a cycle counter into a per-core slice of a trace buffer).  dptr: device array of
 * 4*capacity_ctas uint64, owned by the caller; while set, CTA b (b < capacity_ctas) of every
 * dispatch and combine launch stores in dptr[4b .. 4b+3]: the GPU's global nanosecond timer at its
 * start, the timer at its end, the nanoseconds its issuing thread was blocked waiting for incoming
 * rows, and the nanoseconds it was blocked waiting for outgoing rows to leave shared memory (the
 * last two are filled by the bf16 dispatch kernel, zero elsewhere).  Each launch overwrites the
 * previous one's records.  dptr = NULL turns tracing off (the default).  The spread of the end
 * times is the load-balance evidence the paper reports per core (Sec. 9.6). */
strata_status strata_ctx_set_trace(strata_ctx *ctx, uint64_t *dptr, size_t capacity_ctas);

/* Per-CTA event timeline (the paper's in-kernel profiler, Sec. 6.4, manual mode: named begin/end probes
 * at stage boundaries; every core appends time-stamped events to its own slice of a trace buffer, which
 * is decoded into per-core timelines afterwards).
 * buf: n_ctas slices of (1 + events_per_cta) uint64, owned by the caller, zeroed by the caller before
 * use, and readable/writable by the GPU: device memory, or page-locked host memory (under unified
 * addressing the kernels write it in place across PCIe, as the paper's cores write a host-pinned
 * buffer).  Word 0 of slice b counts the events CTA b has recorded so far (events beyond
 * events_per_cta are counted but not stored); the following words are events, appended by every launch
 * on this context while the timeline is set, in stream order:
 *   bits  0..47  GPU global timer, nanoseconds (low 48 bits)
 *   bits 48..55  stage   (strata_stage)
 *   bit  56      0 = begin, 1 = end
 *   bits 57..63  kernel  (strata_kernel_id)
 * One thread per CTA records; a probe costs one timer read and one 8-byte store, and nothing when the
 * timeline is off (buf = NULL, the default).  CTAs with blockIdx >= n_ctas record nothing.
 * Every probed kernel records its CTA lifetime (STRATA_STAGE_KERNEL).  Inside it, per unit of work: the
 * bf16 dispatch and the collectives' copy kernel record WAIT_IN, WORK and WAIT_OUT; combine and the
 * collectives' reduce kernel record WORK; the fp8 dispatch records WAIT_OUT, WAIT_IN (including the block
 * barrier) and WORK (quantise, scales, store issue); the window-major dispatch records the lifetime only.
 * The layout kernels are not probed. */
typedef enum {
    STRATA_STAGE_KERNEL = 0,     /* the CTA's lifetime inside one launch                        */
    STRATA_STAGE_WAIT_IN = 1,    /* blocked until a unit's input has arrived in shared memory   */
    STRATA_STAGE_WORK = 2,       /* issuing a unit's stores / computing a unit                  */
    STRATA_STAGE_WAIT_OUT = 3    /* blocked until earlier stores have left shared memory        */
} strata_stage;
typedef enum {
    STRATA_KERNEL_DISPATCH_BF16 = 1, STRATA_KERNEL_DISPATCH_FP8 = 2, STRATA_KERNEL_COMBINE = 3,
    STRATA_KERNEL_DISPATCH_WINDOWS = 4, STRATA_KERNEL_SLICE_COPY = 5, STRATA_KERNEL_SLICE_REDUCE = 6
} strata_kernel_id;
strata_status strata_ctx_set_timeline(strata_ctx *ctx, uint64_t *buf, size_t n_ctas, size_t events_per_cta);

/* One decoded interval of a timeline: CTA `cta` of kernel `kernel` spent [begin_ns, end_ns) in `stage`. */
typedef struct {
    uint32_t cta;
    uint8_t kernel;              /* strata_kernel_id */
    uint8_t stage;               /* strata_stage     */
    uint16_t flags;              /* 1: a begin that was never closed; 2: an end without a begin (end_ns = begin_ns) */
    uint64_t begin_ns, end_ns;   /* 48-bit timer values, made monotonic within the slice */
} strata_span;
/* Host-only: pairs the begin/end events of a timeline buffer (a HOST copy, same layout as above) into
 * spans, slice by slice in event order; nested stages are allowed (a stack per slice).  Writes at most
 * max_spans spans; *n_spans is the number found (> max_spans: call again with more room); *dropped is
 * the number of events the kernels counted but could not store.  INVALID_ARG on NULL pointers. */
strata_status strata_timeline_decode(const uint64_t *host_buf, size_t n_ctas, size_t events_per_cta,
                                     strata_span *spans, size_t max_spans, size_t *n_spans, size_t *dropped);

/* ---- pool: registration at allocation time ------------------------------
 * Analogue of the paper's registration-on-allocation (Sec. 5.1): a buffer is
 * registered once, when it is allocated (phase 1); every later operator call
 * only performs a cheap local readiness check (phase 2).  Here the caller
 * allocates (e.g. a torch tensor), the library records [base, base+bytes) and
 * can sub-allocate from it, so the receive buffer handed to dispatch is the
 * very tensor the expert GEMM reads: no staging copy exists (Sec. 2.2 / 8.1
 * describe the staging copies this removes).  Rank partitions are disjoint
 * sub-ranges of one address space (Sec. 5.2). */
strata_status strata_pool_register(strata_ctx *ctx, void *dbase, size_t bytes, uint64_t *region_id);
/* OK iff [dptr, dptr+bytes) lies inside one registered region; pure host lookup. */
strata_status strata_pool_is_ready(strata_ctx *ctx, const void *dptr, size_t bytes);
strata_status strata_pool_unregister(strata_ctx *ctx, uint64_t region_id);
/* Bump sub-allocation inside a region (align: power of two, >= 1).  CAPACITY if it does not fit. */
strata_status strata_pool_carve(strata_ctx *ctx, uint64_t region_id, size_t bytes, size_t align, void **dptr);
strata_status strata_pool_reset(strata_ctx *ctx, uint64_t region_id);

/* ---- the hot path --------------------------------------------------------- */

/* Routing layout (paper App. D, level 1).  topk_ids: device int32 [R,T,K].
 * Computes a stable counting sort of the items by expert id: dst_row[i] =
 * expert_offset[e_i] + #{j < i : e_j = e_i}, i.e. segments ordered by expert,
 * then source rank, then token, then slot, packed without padding.
 * Duplicate ids inside a token are legal.  An id outside [0,E) is skipped
 * (dst_row = -1, not counted) and raises BAD_EXPERT_ID on the device status
 * (except -1 under STRATA_FLAG_ALLOW_UNROUTED, which is legal).
 * Needs a workspace.  One kernel launch for up to 32,768 items, two beyond
 * (fixed-capacity layout: one launch while T*K <= 4096, else two). */
strata_status strata_moe_layout(strata_ctx *ctx, const int32_t *topk_ids,
                                const strata_moe_layout_t *layout, void *stream);

/* Routing layout without any allocation or workspace (the paper has no counterpart: this entry
 * exists for this library's callers only).  It is for callers that cannot hand over a workspace
 * because they cannot allocate device memory where they run: a serving process whose framework
 * pool already owns all of the GPU's memory, a plug-in hook that must avoid the device-wide
 * synchronisation cudaMalloc and cudaFree bring, or a binding with no device allocator of its own.
 * Same inputs, outputs, ordering and error rules as strata_moe_layout, computed by the same kernels;
 * the kernels' scratch lives in a fixed 2 MiB array inside the library (each GPU that loads the
 * library holds it until the process exits) instead of a caller workspace.
 *  - Runs on the CURRENT CUDA device; no context is needed.  `shape->H` and `dispatch_dtype` are ignored;
 *    segment_align, flags and slot_capacity are honoured and checked as strata_ctx_create checks them
 *    (an unknown flag bit, or aligned segments together with fixed slots: STRATA_ERR_SHAPE).
 *  - Limit: 256 + ceil(T*K/4096) * R * E * 4 bytes must fit in 2 MiB (all five benchmark shapes do;
 *    the prefill shape needs 0.13 MiB).  Larger shapes return STRATA_ERR_CAPACITY and launch nothing:
 *    use strata_moe_layout with a workspace for those.
 *  - device_status: device pointer to one int32 owned by the caller, zeroed by the caller; receives
 *    STRATA_ERR_BAD_EXPERT_ID if an id outside [0,E) was skipped and, under slot_capacity > 0,
 *    STRATA_ERR_CAPACITY if a slot overflowed (the first error wins).  May be NULL: skipped and
 *    dropped items are then only visible as dst_row = -1, and a caller that must tell an overflow
 *    from an unrouted slot has to pass the word.
 *  - The first call on each device resolves the array's device address and sets one kernel
 *    attribute (no allocation).  Make that first call before any stream capture begins.
 *  - All calls on a device share the one array, which keeps the previous call's contents; the
 *    entry clears the words that must start at zero, in stream order.  Two calls whose kernels can
 *    overlap on the GPU (different streams, no dependency between them) race on the array and give
 *    wrong results: serialise them.
 *  - Calls no cudaMalloc, cudaFree or any other allocating routine. */
strata_status strata_moe_layout_noalloc(const strata_moe_shape *shape, const int32_t *topk_ids,
                                        const strata_moe_layout_t *layout, int32_t *device_status,
                                        void *stream);

/* Dispatch (paper Sec. 6.2 / 8.1).  x: device bf16 [R,T,H].
 * BF16:  recv is device bf16 [capacity_rows, H]; recv[dst_row[i], :] = x[n(i), :] bit for bit;
 *        recv_scale must be NULL.
 * FP8:   recv is device uint8 [capacity_rows, H], recv_scale device float [capacity_rows, H/128];
 *        per token and block of 128 columns: amax = max|x|, scale = amax/448 (IEEE binary32
 *        division), q = e4m3_rne_satfinite(x / (amax == 0 ? 1 : scale)); codes and the stored
 *        scale (amax/448) go to each of the token's K rows.
 * recv (and recv_scale) must lie inside a registered region (NOT_REGISTERED otherwise); x and recv
 * must be 16-byte aligned, recv_scale 4-byte aligned; capacity_rows >= strata_moe_recv_rows (CAPACITY
 * otherwise).  Items with dst_row = -1 are skipped silently; any other dst_row outside
 * [0, capacity_rows) is skipped and raises BAD_ROW.  One kernel launch. */
strata_status strata_moe_dispatch(strata_ctx *ctx, const strata_moe_layout_t *layout, const void *x,
                                  void *recv, float *recv_scale, size_t capacity_rows, void *stream);

/* Combine (paper Sec. 6.1, reduction-bearing operators).  y: device bf16 [y_rows, H] (expert
 * outputs, row j answers receive row j; may be the receive buffer itself), topk_w: device
 * float [R,T,K], out: device bf16 [R,T,H].
 * out[n,c] = bf16_rne( fma(w[n,K-1], y[dst_row[n,K-1],c], ... fma(w[n,0], y[dst_row[n,0],c], +0)) ):
 * binary32 fused multiply-add chain in slot order, one rounding to bf16.  Slots with dst_row = -1
 * contribute nothing; any other dst_row outside [0, y_rows) contributes nothing and raises BAD_ROW.
 * One kernel launch. */
strata_status strata_moe_combine(strata_ctx *ctx, const strata_moe_layout_t *layout, const void *y,
                                 size_t y_rows, const float *topk_w, void *out, void *stream);

/* Ranks with different token counts (production variant; the paper's Sec. 5.3 motivates batch sizes that
 * change from step to step, it defines no interface).  The batch is stored as R x T with T the largest count;
 * this call writes -1 ("not routed") into the K slots of every token t >= tokens_per_rank[r], in place, so
 * that the layout call that follows on the same stream skips them: the real items then get exactly the rows
 * of the compacted ragged batch, dispatch writes nothing for the padding tokens and combine returns zero rows
 * for them.  tokens_per_rank: device int32 [R] (values above T keep the whole rank, negative values mask it);
 * topk_ids: device int32 [R,T,K].  The context must have been created with STRATA_FLAG_ALLOW_UNROUTED
 * (STRATA_ERR_SHAPE otherwise).  One launch. */
strata_status strata_moe_mask_ragged(strata_ctx *ctx, const int32_t *tokens_per_rank, int32_t *topk_ids, void *stream);

/* In-place consumer of the receive buffer (paper Sec. 2.2 / 8.1: the receive buffer is the input of the expert
 * computation, no staging copy).  The paper's expert is a grouped GEMM, which this library does not contain;
 * this call is the hand-over part of such a consumer with a per-expert affine map standing in for the GEMM.
 * It walks recv in tiles of tile_rows rows; every tile finds the expert e that owns it and its number of
 * occupied rows from expert_offset / expert_count as the layout call on the same stream left them, and
 * rewrites those rows in place:  recv[row][c] = bf16_rne(fma(f32(recv[row][c]), scale[e], bias[e]))
 * (one binary32 fused multiply-add, one rounding).  Padding rows are not touched.  With it, layout ->
 * dispatch -> expert -> combine runs on the device with no host step and no copy between the calls.
 * recv: device bf16 [capacity_rows >= strata_moe_recv_rows, H] inside a registered region; scale, bias:
 * device float [E].  tile_rows >= 1 must divide the context's segment_align (1 for packed segments), so
 * that no tile holds rows of two experts (STRATA_ERR_SHAPE otherwise, and for e4m3 or fixed-capacity
 * contexts).  One launch. */
strata_status strata_moe_expert_affine_inplace(strata_ctx *ctx, const strata_moe_layout_t *layout, void *recv,
                                               size_t capacity_rows, const float *scale, const float *bias,
                                               int32_t tile_rows, void *stream);

/* Row -> expert map of the receive buffer (production variant; the paper names no such array): the per-row
 * group index a grouped expert GEMM needs to read the receive buffer in place, completing the zero-copy
 * hand-over (with segment_align set to the GEMM's tile height, every tile of rows belongs to one expert or
 * is empty).  row_expert: device int32 [capacity_rows >= strata_moe_recv_rows]; row_expert[row] = the
 * expert whose segment holds the row if the layout placed a token there, -1 for the padding of aligned
 * segments and the empty rows of the fixed-capacity layout (rows beyond strata_moe_recv_rows are not
 * written).  Reads expert_count and expert_offset (and src_expert_count for the fixed-capacity layout,
 * where it must be present) as the layout call on the same stream left them.  One launch. */
strata_status strata_moe_row_experts(strata_ctx *ctx, const strata_moe_layout_t *layout, int32_t *row_expert,
                                     size_t capacity_rows, void *stream);

/* ---- optional: the paper's hierarchical workload partitioning (Sec. 6.2, App. B to D) -----------
 * The default dispatch balances at run time by ordered work claiming.  These two calls build and run
 * the paper's own static scheme instead, so that it can be compared on this hardware:
 *   expert windows  (source rank r, expert e): src_expert_count[r][e] contiguous receive rows starting
 *                   at win_base[r][e];
 *   peer windows    (r -> destination rank d): the expert windows of d's experts in expert order, cut
 *                   into transfer units of at most unit_rows rows of the tier of (r,d);
 *                   tier(r,d) = 0 if r/g0 == d/g0, else 1 if r/g1 == d/g1, else 2 (clamped to n_tiers-1);
 *   unit cost       tau = alpha + ceil(bytes / beta), integers;
 *   policy          LPT-style list scheduling: units by decreasing cost (ties: lower unit id) onto the
 *                   least-loaded core (ties: lower core id), and on that core into the earliest issue
 *                   stripe after the core's previous unit that holds fewer than fanout_cap units for the
 *                   unit's destination rank.  Reading of Sec. 6.2 used: a core issues at most one unit per
 *                   stripe and may leave a stripe empty, and stripes are not limited in number, so the cap
 *                   F[stripe][dest] <= H_t is always met by a later stripe and never moves a unit to a
 *                   busier core: the lists and loads are those of plain LPT, the cap shows in task_stripe.
 * Unit ids enumerate (r, d, k) in that order. */
typedef struct {
    int64_t alpha;        /* fixed cost of a unit, 0 <= alpha < 2^30                      */
    int64_t beta;         /* bytes per cost unit, >= 1                                    */
    int64_t unit_rows;    /* S_t in rows, >= 1; unit_rows * row_bytes / beta < 2^36       */
    int32_t fanout_cap;   /* H_t >= 1                                                     */
    int32_t reserved;
} strata_tier;
typedef struct {
    int32_t n_tiers;      /* 1..3 */
    int32_t g0, g1;       /* ranks per innermost group and per middle group, >= 1         */
    int32_t reserved;
    strata_tier tiers[3];
} strata_partition_policy;
typedef struct {            /* all device pointers, caller-owned */
    int32_t *win_base;      /* [R,E]            first receive row of expert window (r,e)              */
    int32_t *unit_desc;     /* [max_units,4]    source rank, destination rank, first logical row, rows */
    int64_t *unit_cost;     /* [max_units]                                                            */
    int32_t *n_units;       /* [1]              number of units; -1 if they did not fit                */
    int32_t *task_offset;   /* [n_cores+1]      core c's list is task_unit[task_offset[c] .. [c+1])    */
    int32_t *task_unit;     /* [max_units]      unit ids, core-major, in issue order                   */
    int64_t *core_load;     /* [n_cores]        predicted load of each core                            */
    int32_t *scratch;       /* [max_units*(R+2)] working memory of the policy kernel                   */
    int32_t *task_stripe;   /* [max_units]      issue stripe of every entry of task_unit (strictly          */
                            /*                  increasing inside a core's list)                            */
} strata_partition_t;

/* Upper bound of the unit count for a shape and policy (host arithmetic only):
 * sum over tiers is bounded by N / min(unit_rows) + R*R. */
strata_status strata_moe_partition_max_units(const strata_moe_shape *shape, const strata_partition_policy *policy,
                                             size_t *max_units);
/* Generates the policy on the GPU (one launch, one CTA) from a layout that includes src_expert_count.
 * Limits: at most 8192 units and 1024 cores; more units raise STRATA_ERR_CAPACITY on the device status
 * and set *n_units = -1 (choose larger units).  Host errors: INVALID_ARG, SHAPE, WORKSPACE, CAPACITY. */
strata_status strata_moe_partition(strata_ctx *ctx, const strata_moe_layout_t *layout,
                                   const strata_partition_policy *policy, int32_t n_cores,
                                   const strata_partition_t *out, size_t max_units, void *stream);
/* Window-major bf16 dispatch: n_cores one-warp CTAs, CTA c copies the rows of the units in its task
 * list in order, one source row (found through layout->src_of_row, which must be present) per
 * receive row.  Writes exactly what strata_moe_dispatch writes.  Same registration, alignment and
 * capacity rules; rows of at most 16 KB. */
strata_status strata_moe_dispatch_windows(strata_ctx *ctx, const strata_moe_layout_t *layout,
                                          const strata_partition_t *partition, int32_t n_cores, const void *x,
                                          void *recv, size_t capacity_rows, void *stream);

/* Host helper: rank d's partition of the receive buffer, from a HOST copy of rank_offset[R+1]:
 * *rank_base = recv + rank_offset[d] * row_bytes, *rows = rank_offset[d+1] - rank_offset[d]. */
strata_status strata_moe_recv_view(strata_ctx *ctx, const int32_t *h_rank_offset, int rank,
                                   void *recv, void **rank_base, int64_t *rows);

/* Synchronises the stream, reads the device status word into *out and clears it. */
strata_status strata_device_status(strata_ctx *ctx, void *stream, strata_status *out);

/* Whole path from HOST buffers with identity experts (BF16 contexts only): copies ids, x and
 * gate weights to the device buffers given in `dev`, runs layout -> dispatch -> combine with
 * y = recv, copies out back and synchronises the stream.  Tokens travel in chunks of about 64 MB on
 * two internal copy streams, so the upload of one chunk, the kernels of the previous one and the
 * download of the one before overlap (streams and events are created on the first call; no device
 * memory is allocated).  h_* are host pointers (pinned memory
 * makes the copies asynchronous); every member of `dev` is a device pointer owned by the caller,
 * dev->recv inside a registered region with room for N rows.  Used for end-to-end timing and
 * smoke checks; the paper has no counterpart (its operators take device buffers). */
typedef struct {
    int32_t *ids;       /* [R,T,K] */
    void *x;            /* bf16 [R,T,H] */
    float *w;           /* [R,T,K] */
    void *recv;         /* bf16 [N,H] */
    void *out;          /* bf16 [R,T,H] */
    strata_moe_layout_t layout;
} strata_moe_device_buffers;
strata_status strata_moe_roundtrip_host(strata_ctx *ctx, const strata_moe_device_buffers *dev,
                                        const int32_t *h_ids, const void *h_x, const float *h_w,
                                        void *h_out, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* STRATA_MOE_H */
