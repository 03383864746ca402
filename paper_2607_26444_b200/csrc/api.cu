// C ABI: context, registration pool, argument validation and kernel launches.
// Host-side only; every device-side step lives in layout.cu / dispatch.cu / combine.cu.
#include <algorithm>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"

namespace strata {
cudaError_t configure_layout_kernels();
cudaError_t configure_dispatch_kernels();
cudaError_t configure_partition_kernels();
cudaError_t configure_collective_kernels();
}  // namespace strata

struct strata_region {
    uint64_t id;
    uintptr_t base;
    size_t bytes;
    size_t used;      // bump pointer of strata_pool_carve
};

struct strata_ctx {
    strata_moe_shape shape;
    int device;
    int n_sm;             // SMs the persistent kernels size their grids for (the device's, or the caller's budget)
    int n_sm_device;
    int x_early;          // the caller's promise about x (strata_ctx_set_x_early)
    int* ws;              // device workspace (header + tile counts)
    size_t ws_bytes;
    uint64_t next_region;
    uint64_t launches;
    strata::TraceBuf trace;
    // host round trip only: copy streams and events, created on first use (no device memory)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_done;
    cudaEvent_t ev_entry = nullptr, ev_out = nullptr;
    std::vector<strata_region> regions;
    std::mutex mu;
};

namespace {

using namespace strata;

strata_status check_shape(const strata_moe_shape* s)
{
    if (!s) return STRATA_ERR_INVALID_ARG;
    if (s->H <= 0 || s->H % 8 != 0) return STRATA_ERR_SHAPE;
    const strata_status st = check_layout_shape(*s);
    if (st != STRATA_OK) return st;
    if (s->dispatch_dtype != STRATA_BF16 && s->dispatch_dtype != STRATA_FP8_E4M3_B128) return STRATA_ERR_SHAPE;
    if (s->dispatch_dtype == STRATA_FP8_E4M3_B128 && s->H % 128 != 0) return STRATA_ERR_SHAPE;
    // Dispatch and combine number their work units (a token, or a column piece of one never shorter than
    // 1 KB) with 32-bit counters whose top values are reserved.
    if ((long long)s->R * s->T * (((long long)s->H * 2 + 1023) / 1024) >= (1ll << 32) - (1ll << 20)) return STRATA_ERR_SHAPE;
    return STRATA_OK;
}

size_t workspace_bytes(const strata_moe_shape& s)
{
    const LayoutGeom g = layout_geom(s);
    size_t b = (size_t)kWsHeaderBytes + (size_t)g.n_tiles * s.E * sizeof(int);
    return ((b + 255) & ~(size_t)255) + collective_table_bytes();
}

WorkQueue dispatch_queue(const strata_ctx* c) { return WorkQueue{reinterpret_cast<unsigned int*>(c->ws) + 2}; }
WorkQueue combine_queue(const strata_ctx* c) { return WorkQueue{reinterpret_cast<unsigned int*>(c->ws) + 4}; }
WorkQueue collective_queue(const strata_ctx* c) { return WorkQueue{reinterpret_cast<unsigned int*>(c->ws) + 6}; }

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

bool region_contains(const strata_ctx* c, const void* p, size_t bytes)
{
    const uintptr_t a = reinterpret_cast<uintptr_t>(p);
    for (const strata_region& r : c->regions)
        if (a >= r.base && bytes <= r.bytes && a - r.base <= r.bytes - bytes) return true;
    return false;
}

strata_status check_layout_ptrs(const strata_moe_layout_t* L, bool need_all)
{
    if (!L || !L->dst_row) return STRATA_ERR_INVALID_ARG;
    if (need_all && (!L->expert_count || !L->expert_offset || !L->rank_count || !L->rank_offset))
        return STRATA_ERR_INVALID_ARG;
    return STRATA_OK;
}

}  // namespace

extern "C" {

const char* strata_status_string(strata_status s)
{
    switch (s) {
        case STRATA_OK: return "ok";
        case STRATA_ERR_INVALID_ARG: return "invalid argument";
        case STRATA_ERR_SHAPE: return "unsupported shape";
        case STRATA_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case STRATA_ERR_NOT_REGISTERED: return "buffer not inside a registered region";
        case STRATA_ERR_CAPACITY: return "capacity too small";
        case STRATA_ERR_BAD_EXPERT_ID: return "expert id out of range (item skipped)";
        case STRATA_ERR_WORKSPACE: return "no workspace set";
        case STRATA_ERR_CUDA: return "CUDA runtime error";
        case STRATA_ERR_TIMEOUT: return "bounded device wait ran out";
        case STRATA_ERR_BAD_ROW: return "destination row out of range (row skipped)";
    }
    return "unknown status";
}

strata_status strata_ctx_create(strata_ctx** out, const strata_moe_shape* shape, int device)
{
    if (!out) return STRATA_ERR_INVALID_ARG;
    *out = nullptr;
    strata_status st = check_shape(shape);
    if (st != STRATA_OK) return st;
    int n_sm = 0;
    if (device != -1) {
        int n_dev = 0;
        if (cudaGetDeviceCount(&n_dev) != cudaSuccess) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
        if (device < 0 || device >= n_dev) return STRATA_ERR_INVALID_ARG;
        DeviceGuard g(device);
        if (!g.ok) return STRATA_ERR_CUDA;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
            return STRATA_ERR_CUDA;
        if (configure_layout_kernels() != cudaSuccess || configure_dispatch_kernels() != cudaSuccess ||
            configure_partition_kernels() != cudaSuccess || configure_collective_kernels() != cudaSuccess) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
    }
    strata_ctx* c = new (std::nothrow) strata_ctx();
    if (!c) return STRATA_ERR_INVALID_ARG;
    c->shape = *shape;
    c->device = device;
    c->n_sm = n_sm;
    c->n_sm_device = n_sm;
    c->x_early = 0;
    c->ws = nullptr;
    c->ws_bytes = 0;
    c->next_region = 1;
    c->launches = 0;
    c->trace = strata::TraceBuf{nullptr, 0, nullptr, 0, 0};
    *out = c;
    return STRATA_OK;
}

strata_status strata_ctx_destroy(strata_ctx* ctx)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    if (ctx->device >= 0 && (ctx->s_in || ctx->ev_entry)) {
        DeviceGuard g(ctx->device);
        for (cudaEvent_t e : ctx->ev_in) cudaEventDestroy(e);
        for (cudaEvent_t e : ctx->ev_done) cudaEventDestroy(e);
        if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
        if (ctx->ev_out) cudaEventDestroy(ctx->ev_out);
        if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
        if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
    }
    delete ctx;
    return STRATA_OK;
}

strata_status strata_moe_workspace_bytes(const strata_moe_shape* shape, size_t* bytes)
{
    if (!bytes) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_shape(shape);
    if (st != STRATA_OK) return st;
    *bytes = workspace_bytes(*shape);
    return STRATA_OK;
}

strata_status strata_moe_recv_rows(const strata_moe_shape* shape, size_t* rows)
{
    if (!rows) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_shape(shape);
    if (st != STRATA_OK) return st;
    *rows = (size_t)recv_rows(*shape);
    return STRATA_OK;
}

strata_status strata_ctx_set_workspace(strata_ctx* ctx, void* dptr, size_t bytes)
{
    if (!ctx || !dptr) return STRATA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(dptr) & 255u) != 0) return STRATA_ERR_ALIGNMENT;
    if (bytes < workspace_bytes(ctx->shape)) return STRATA_ERR_CAPACITY;
    if (ctx->device < 0) {               // host-only context: record, never touch
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->ws = static_cast<int*>(dptr);
        ctx->ws_bytes = bytes;
        return STRATA_OK;
    }
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    if (cudaMemset(dptr, 0, workspace_bytes(ctx->shape)) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) {
        cudaGetLastError();
        return STRATA_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lk(ctx->mu);
    ctx->ws = static_cast<int*>(dptr);
    ctx->ws_bytes = bytes;
    return STRATA_OK;
}

strata_status strata_ctx_launch_count(strata_ctx* ctx, uint64_t* count)
{
    if (!ctx || !count) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    *count = ctx->launches;
    return STRATA_OK;
}

strata_status strata_ctx_set_sm_budget(strata_ctx* ctx, int32_t n_sm)
{
    if (!ctx || n_sm < 0) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    ctx->n_sm = (n_sm == 0 || n_sm > ctx->n_sm_device) ? ctx->n_sm_device : n_sm;
    return STRATA_OK;
}

strata_status strata_ctx_set_x_early(strata_ctx* ctx, int32_t on)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    ctx->x_early = on ? 1 : 0;
    return STRATA_OK;
}

strata_status strata_ctx_set_trace(strata_ctx* ctx, uint64_t* dptr, size_t capacity_ctas)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    if (dptr && (reinterpret_cast<uintptr_t>(dptr) & 7u) != 0) return STRATA_ERR_ALIGNMENT;
    if (dptr && (capacity_ctas == 0 || capacity_ctas > (size_t)1 << 24)) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    ctx->trace.slots = reinterpret_cast<unsigned long long*>(dptr);
    ctx->trace.capacity = dptr ? (int)capacity_ctas : 0;
    return STRATA_OK;
}

strata_status strata_ctx_set_timeline(strata_ctx* ctx, uint64_t* buf, size_t n_ctas, size_t events_per_cta)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    if (buf && (reinterpret_cast<uintptr_t>(buf) & 7u) != 0) return STRATA_ERR_ALIGNMENT;
    if (buf && (n_ctas == 0 || n_ctas > (size_t)1 << 24 || events_per_cta == 0 || events_per_cta > (size_t)1 << 24))
        return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    ctx->trace.tl = reinterpret_cast<unsigned long long*>(buf);
    ctx->trace.tl_ctas = buf ? (int)n_ctas : 0;
    ctx->trace.tl_cap = buf ? (int)events_per_cta : 0;
    return STRATA_OK;
}

strata_status strata_timeline_decode(const uint64_t* host_buf, size_t n_ctas, size_t events_per_cta,
                                     strata_span* spans, size_t max_spans, size_t* n_spans, size_t* dropped)
{
    if (!host_buf || !n_spans || !dropped || (!spans && max_spans > 0)) return STRATA_ERR_INVALID_ARG;
    size_t found = 0, lost = 0;
    struct Open { uint8_t kernel, stage; uint64_t t; };
    std::vector<Open> stack;
    auto emit = [&](uint32_t cta, uint8_t kernel, uint8_t stage, uint16_t flags, uint64_t b, uint64_t e) {
        if (found < max_spans) spans[found] = strata_span{cta, kernel, stage, flags, b, e};
        ++found;
    };
    for (size_t b = 0; b < n_ctas; ++b) {
        const uint64_t* slice = host_buf + b * (events_per_cta + 1);
        const uint64_t counted = slice[0];
        const size_t n = counted < events_per_cta ? (size_t)counted : events_per_cta;
        lost += (size_t)(counted - n);
        stack.clear();
        uint64_t wraps = 0, prev = 0;
        for (size_t i = 0; i < n; ++i) {
            const uint64_t ev = slice[1 + i];
            uint64_t t = ev & 0xffffffffffffull;
            if (i > 0 && t + wraps < prev && prev - (t + wraps) > (1ull << 47)) wraps += 1ull << 48;   // timer wrapped
            t += wraps;
            prev = t;
            const uint8_t stage = (uint8_t)((ev >> 48) & 0xff), kernel = (uint8_t)(ev >> 57);
            if (((ev >> 56) & 1) == 0) {
                stack.push_back(Open{kernel, stage, t});
                continue;
            }
            // an end closes the innermost open begin of the same kernel and stage
            size_t k = stack.size();
            while (k > 0 && !(stack[k - 1].kernel == kernel && stack[k - 1].stage == stage)) --k;
            if (k == 0) {
                emit((uint32_t)b, kernel, stage, 2, t, t);           // an end without a begin
                continue;
            }
            emit((uint32_t)b, kernel, stage, 0, stack[k - 1].t, t);
            stack.erase(stack.begin() + (long)(k - 1));
        }
        for (const Open& o : stack) emit((uint32_t)b, o.kernel, o.stage, 1, o.t, o.t);   // never closed
    }
    *n_spans = found;
    *dropped = lost;
    return STRATA_OK;
}

// ---- pool -------------------------------------------------------------------------

strata_status strata_pool_register(strata_ctx* ctx, void* dbase, size_t bytes, uint64_t* region_id)
{
    if (!ctx || !dbase || !region_id || bytes == 0) return STRATA_ERR_INVALID_ARG;
    if (!aligned16(dbase)) return STRATA_ERR_ALIGNMENT;
    const uintptr_t a = reinterpret_cast<uintptr_t>(dbase);
    if (a + bytes < a) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    for (const strata_region& r : ctx->regions)
        if (a < r.base + r.bytes && r.base < a + bytes) return STRATA_ERR_INVALID_ARG;   // overlap
    strata_region r{ctx->next_region++, a, bytes, 0};
    ctx->regions.push_back(r);
    *region_id = r.id;
    return STRATA_OK;
}

strata_status strata_pool_is_ready(strata_ctx* ctx, const void* dptr, size_t bytes)
{
    if (!ctx || !dptr) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    return region_contains(ctx, dptr, bytes) ? STRATA_OK : STRATA_ERR_NOT_REGISTERED;
}

strata_status strata_pool_unregister(strata_ctx* ctx, uint64_t region_id)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    for (size_t i = 0; i < ctx->regions.size(); ++i)
        if (ctx->regions[i].id == region_id) {
            ctx->regions.erase(ctx->regions.begin() + (long)i);
            return STRATA_OK;
        }
    return STRATA_ERR_NOT_REGISTERED;
}

strata_status strata_pool_carve(strata_ctx* ctx, uint64_t region_id, size_t bytes, size_t align, void** dptr)
{
    if (!ctx || !dptr || align == 0 || (align & (align - 1)) != 0) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    for (strata_region& r : ctx->regions)
        if (r.id == region_id) {
            const uintptr_t cur = r.base + r.used;
            const uintptr_t al = (cur + (align - 1)) & ~(uintptr_t)(align - 1);
            const size_t start = al - r.base;
            if (start > r.bytes || bytes > r.bytes - start) return STRATA_ERR_CAPACITY;
            r.used = start + bytes;
            *dptr = reinterpret_cast<void*>(al);
            return STRATA_OK;
        }
    return STRATA_ERR_NOT_REGISTERED;
}

strata_status strata_pool_reset(strata_ctx* ctx, uint64_t region_id)
{
    if (!ctx) return STRATA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lk(ctx->mu);
    for (strata_region& r : ctx->regions)
        if (r.id == region_id) {
            r.used = 0;
            return STRATA_OK;
        }
    return STRATA_ERR_NOT_REGISTERED;
}

// ---- hot path -----------------------------------------------------------------------

strata_status strata_moe_layout(strata_ctx* ctx, const int32_t* topk_ids, const strata_moe_layout_t* layout,
                                void* stream)
{
    if (!ctx || !topk_ids) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_layout_ptrs(layout, true);
    if (st != STRATA_OK) return st;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    int n = 0;
    cudaError_t err = launch_layout(ctx->shape, topk_ids, *layout, ctx->ws, ctx->ws + kWsHeaderBytes / sizeof(int),
                                    static_cast<cudaStream_t>(stream), &n);
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += (uint64_t)n;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_dispatch(strata_ctx* ctx, const strata_moe_layout_t* layout, const void* x, void* recv,
                                  float* recv_scale, size_t capacity_rows, void* stream)
{
    if (!ctx || !x || !recv) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_layout_ptrs(layout, false);
    if (st != STRATA_OK) return st;
    const strata_moe_shape& s = ctx->shape;
    const bool fp8 = s.dispatch_dtype == STRATA_FP8_E4M3_B128;
    if (fp8 != (recv_scale != nullptr)) return STRATA_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(recv)) return STRATA_ERR_ALIGNMENT;
    if (fp8 && (reinterpret_cast<uintptr_t>(recv_scale) & 3u) != 0) return STRATA_ERR_ALIGNMENT;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    const size_t n_rows = (size_t)recv_rows(s);
    if (capacity_rows < n_rows) return STRATA_ERR_CAPACITY;
    const size_t row_bytes = fp8 ? (size_t)s.H : (size_t)s.H * 2;
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        if (!region_contains(ctx, recv, capacity_rows * row_bytes)) return STRATA_ERR_NOT_REGISTERED;
        if (fp8 && !region_contains(ctx, recv_scale, capacity_rows * (size_t)(s.H / 128) * sizeof(float)))
            return STRATA_ERR_NOT_REGISTERED;
    }
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err =
        fp8 ? launch_dispatch_fp8(s, layout->dst_row, x, recv, recv_scale, capacity_rows, ctx->ws, dispatch_queue(ctx),
                                  ctx->n_sm, ctx->trace, ctx->x_early != 0, static_cast<cudaStream_t>(stream))
            : launch_dispatch_bf16(s, layout->dst_row, x, recv, capacity_rows, ctx->ws, dispatch_queue(ctx), ctx->n_sm,
                                   ctx->trace, ctx->x_early != 0, static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_combine(strata_ctx* ctx, const strata_moe_layout_t* layout, const void* y, size_t y_rows,
                                 const float* topk_w, void* out, void* stream)
{
    if (!ctx || !y || !topk_w || !out) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_layout_ptrs(layout, false);
    if (st != STRATA_OK) return st;
    if (!aligned16(y) || !aligned16(out)) return STRATA_ERR_ALIGNMENT;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_combine(ctx->shape, layout->dst_row, y, y_rows, topk_w, out, ctx->ws, combine_queue(ctx),
                                     ctx->n_sm, ctx->trace, static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_expert_affine_inplace(strata_ctx* ctx, const strata_moe_layout_t* layout, void* recv,
                                               size_t capacity_rows, const float* scale, const float* bias,
                                               int32_t tile_rows, void* stream)
{
    if (!ctx || !layout || !recv || !scale || !bias) return STRATA_ERR_INVALID_ARG;
    if (!layout->expert_count || !layout->expert_offset) return STRATA_ERR_INVALID_ARG;
    const strata_moe_shape& s = ctx->shape;
    if (s.dispatch_dtype != STRATA_BF16 || s.slot_capacity > 0) return STRATA_ERR_SHAPE;
    const int align = s.segment_align > 1 ? s.segment_align : 1;
    if (tile_rows < 1 || align % tile_rows != 0) return STRATA_ERR_SHAPE;    // a tile must never hold two experts
    if (!aligned16(recv)) return STRATA_ERR_ALIGNMENT;
    const size_t n_rows = (size_t)recv_rows(s);
    if (capacity_rows < n_rows) return STRATA_ERR_CAPACITY;
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        if (!region_contains(ctx, recv, capacity_rows * (size_t)s.H * 2)) return STRATA_ERR_NOT_REGISTERED;
    }
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_expert_affine(s, *layout, recv, (long long)n_rows, scale, bias, tile_rows, ctx->n_sm,
                                           static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    if (err != cudaSuccess) cudaGetLastError();
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_mask_ragged(strata_ctx* ctx, const int32_t* tokens_per_rank, int32_t* topk_ids, void* stream)
{
    if (!ctx || !tokens_per_rank || !topk_ids) return STRATA_ERR_INVALID_ARG;
    if ((ctx->shape.flags & STRATA_FLAG_ALLOW_UNROUTED) == 0) return STRATA_ERR_SHAPE;   // -1 must be a legal id
    if (((reinterpret_cast<uintptr_t>(tokens_per_rank) | reinterpret_cast<uintptr_t>(topk_ids)) & 3u) != 0)
        return STRATA_ERR_ALIGNMENT;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_mask_ragged(ctx->shape, tokens_per_rank, topk_ids, ctx->n_sm_device,
                                         static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_row_experts(strata_ctx* ctx, const strata_moe_layout_t* layout, int32_t* row_expert,
                                     size_t capacity_rows, void* stream)
{
    if (!ctx || !row_expert) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_layout_ptrs(layout, true);
    if (st != STRATA_OK) return st;
    const strata_moe_shape& s = ctx->shape;
    if (s.slot_capacity > 0 && !layout->src_expert_count) return STRATA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(row_expert) & 3u) != 0) return STRATA_ERR_ALIGNMENT;
    const size_t n_rows = (size_t)recv_rows(s);
    if (capacity_rows < n_rows) return STRATA_ERR_CAPACITY;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_row_experts(s, *layout, row_expert, (long long)n_rows, static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

namespace {
strata_status check_policy(const strata_moe_shape& s, const strata_partition_policy* pol)
{
    if (!pol) return STRATA_ERR_INVALID_ARG;
    if (pol->n_tiers < 1 || pol->n_tiers > 3 || pol->g0 < 1 || pol->g1 < 1) return STRATA_ERR_INVALID_ARG;
    for (int t = 0; t < pol->n_tiers; ++t) {
        const strata_tier& q = pol->tiers[t];
        if (q.alpha < 0 || q.alpha >= (1ll << 30) || q.beta < 1 || q.unit_rows < 1 || q.fanout_cap < 1)
            return STRATA_ERR_INVALID_ARG;
        if (q.unit_rows > (1ll << 31)) return STRATA_ERR_INVALID_ARG;
        if (q.unit_rows * ((long long)s.H * 2) / q.beta >= (1ll << 36)) return STRATA_ERR_INVALID_ARG;
    }
    return STRATA_OK;
}
}  // namespace

strata_status strata_moe_partition_max_units(const strata_moe_shape* shape, const strata_partition_policy* policy,
                                             size_t* max_units)
{
    if (!max_units) return STRATA_ERR_INVALID_ARG;
    strata_status st = check_shape(shape);
    if (st != STRATA_OK) return st;
    st = check_policy(*shape, policy);
    if (st != STRATA_OK) return st;
    long long smin = policy->tiers[0].unit_rows;
    for (int t = 1; t < policy->n_tiers; ++t) smin = std::min<long long>(smin, policy->tiers[t].unit_rows);
    const long long n = (long long)shape->R * shape->T * shape->K;
    *max_units = (size_t)(n / smin + (long long)shape->R * shape->R);
    return STRATA_OK;
}

strata_status strata_moe_partition(strata_ctx* ctx, const strata_moe_layout_t* layout,
                                   const strata_partition_policy* policy, int32_t n_cores,
                                   const strata_partition_t* out, size_t max_units, void* stream)
{
    if (!ctx || !layout || !out) return STRATA_ERR_INVALID_ARG;
    if (!layout->src_expert_count || !layout->expert_offset) return STRATA_ERR_INVALID_ARG;
    if (!out->task_stripe) return STRATA_ERR_INVALID_ARG;
    if (!out->win_base || !out->unit_desc || !out->unit_cost || !out->n_units || !out->task_offset ||
        !out->task_unit || !out->core_load || !out->scratch)
        return STRATA_ERR_INVALID_ARG;
    strata_status st = check_policy(ctx->shape, policy);
    if (st != STRATA_OK) return st;
    if (ctx->shape.slot_capacity > 0) return STRATA_ERR_SHAPE;      // windows assume packed/aligned segments
    if (n_cores < 1 || n_cores > partition_max_cores_supported()) return STRATA_ERR_SHAPE;
    if (max_units < 1 || max_units > (size_t)1 << 20) return STRATA_ERR_CAPACITY;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_partition(ctx->shape, *layout, *policy, n_cores, *out, max_units, ctx->ws,
                                       static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_moe_dispatch_windows(strata_ctx* ctx, const strata_moe_layout_t* layout,
                                          const strata_partition_t* partition, int32_t n_cores, const void* x,
                                          void* recv, size_t capacity_rows, void* stream)
{
    if (!ctx || !layout || !partition || !x || !recv) return STRATA_ERR_INVALID_ARG;
    if (!layout->src_expert_count || !layout->src_of_row) return STRATA_ERR_INVALID_ARG;
    if (!partition->win_base || !partition->unit_desc || !partition->task_offset || !partition->task_unit ||
        !partition->n_units)
        return STRATA_ERR_INVALID_ARG;
    const strata_moe_shape& s = ctx->shape;
    if (s.dispatch_dtype != STRATA_BF16 || (uint32_t)s.H * 2u > windows_max_row_bytes() || s.slot_capacity > 0)
        return STRATA_ERR_SHAPE;
    if (n_cores < 1 || n_cores > partition_max_cores_supported()) return STRATA_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(recv)) return STRATA_ERR_ALIGNMENT;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    const size_t n_rows = (size_t)recv_rows(s);
    if (capacity_rows < n_rows) return STRATA_ERR_CAPACITY;
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        if (!region_contains(ctx, recv, capacity_rows * (size_t)s.H * 2)) return STRATA_ERR_NOT_REGISTERED;
    }
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_dispatch_windows(s, *layout, *partition, n_cores, x, recv, capacity_rows, ctx->ws,
                                              ctx->trace, static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

// ---- full-mesh collectives over emulated ranks ------------------------------------------------

namespace {
constexpr int kMaxCollectiveRanks = 1024;

// checks shared by the five operators
strata_status collective_prologue(strata_ctx* ctx, int32_t R, const void* in, void* out)
{
    if (!ctx || !in || !out) return STRATA_ERR_INVALID_ARG;
    if (R < 1 || R > kMaxCollectiveRanks) return STRATA_ERR_INVALID_ARG;
    if (!aligned16(in) || !aligned16(out)) return STRATA_ERR_ALIGNMENT;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    return STRATA_OK;
}

strata_status run_copy(strata_ctx* ctx, const void* in, void* out, unsigned long long n_slices,
                       unsigned long long slice_bytes, unsigned int inner, unsigned long long stride_a,
                       unsigned long long stride_b, int fan, unsigned long long fan_stride, void* stream)
{
    if (slice_bytes % 16 != 0) return STRATA_ERR_SHAPE;
    if (slice_bytes == 0) return STRATA_OK;
    const unsigned long long chunk = collective_chunk_bytes();
    const unsigned long long cps = (slice_bytes + chunk - 1) / chunk;
    if (cps > 0xfffffffeull / n_slices) return STRATA_ERR_SHAPE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_slice_copy(in, out, n_slices, slice_bytes, inner, stride_a, stride_b, fan, fan_stride,
                                        ctx->ws, collective_queue(ctx), ctx->n_sm, ctx->trace,
                                        static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status run_reduce(strata_ctx* ctx, const void* in, void* out, unsigned long long elems, int R, int fan,
                         void* stream)
{
    if (elems % 8 != 0) return STRATA_ERR_SHAPE;
    if (elems == 0) return STRATA_OK;
    const unsigned long long n_vec = elems / 8;
    if (n_vec / 128 >= 0xfffffffeull) return STRATA_ERR_SHAPE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_slice_reduce(in, out, n_vec, R, fan, collective_queue(ctx), ctx->n_sm, ctx->trace,
                                          static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 1;
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}
}  // namespace

strata_status strata_allgather(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t bytes_per_rank,
                               void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    // slice p = rank p's input; copy f lands in rank f's output at offset p*M
    return run_copy(ctx, in, out, (unsigned long long)R, bytes_per_rank, 1u, bytes_per_rank, 0ull, R,
                    (unsigned long long)R * bytes_per_rank, stream);
}

strata_status strata_alltoall(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t bytes_per_slice,
                              void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    // slice s = p*R + r (sender p, receiver r) lands at (r*R + p)*S
    return run_copy(ctx, in, out, (unsigned long long)R * R, bytes_per_slice, (unsigned int)R, bytes_per_slice,
                    (unsigned long long)R * bytes_per_slice, 1, 0ull, stream);
}

strata_status strata_broadcast(strata_ctx* ctx, int32_t R, int32_t root, const void* in, void* out, size_t bytes,
                               void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    if (root < 0 || root >= R) return STRATA_ERR_INVALID_ARG;
    return run_copy(ctx, static_cast<const unsigned char*>(in) + (size_t)root * bytes, out, 1ull, bytes, 1u, 0ull, 0ull,
                    R, bytes, stream);
}

strata_status strata_p2p(strata_ctx* ctx, int32_t R, int32_t src_rank, int32_t dst_rank, const void* in, void* out,
                         size_t bytes, void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    if (src_rank < 0 || src_rank >= R || dst_rank < 0 || dst_rank >= R) return STRATA_ERR_INVALID_ARG;
    return run_copy(ctx, static_cast<const unsigned char*>(in) + (size_t)src_rank * bytes,
                    static_cast<unsigned char*>(out) + (size_t)dst_rank * bytes, 1ull, bytes, 1u, 0ull, 0ull, 1, 0ull,
                    stream);
}

strata_status strata_alltoallv(strata_ctx* ctx, int32_t R, const void* in, size_t in_stride_bytes, void* out,
                               size_t out_stride_bytes, const int64_t* send_bytes, const int64_t* send_offset,
                               const int64_t* recv_offset, void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    if (!send_bytes || !send_offset || !recv_offset) return STRATA_ERR_INVALID_ARG;
    if (R > collective_max_v_ranks()) return STRATA_ERR_SHAPE;
    if (in_stride_bytes == 0 || out_stride_bytes == 0 || in_stride_bytes % 16 != 0 || out_stride_bytes % 16 != 0)
        return STRATA_ERR_SHAPE;
    // every sender's chunks fit the unit counter whatever the counts turn out to be
    const unsigned long long chunk = collective_chunk_bytes();
    if (((unsigned long long)in_stride_bytes / chunk + (unsigned long long)R) * (unsigned long long)R > 0x7fffffffull)
        return STRATA_ERR_SHAPE;
    if (((reinterpret_cast<uintptr_t>(send_bytes) | reinterpret_cast<uintptr_t>(send_offset) |
          reinterpret_cast<uintptr_t>(recv_offset)) & 7u) != 0)
        return STRATA_ERR_ALIGNMENT;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaError_t err = launch_slice_copyv(in, in_stride_bytes, out, out_stride_bytes,
                                         reinterpret_cast<const long long*>(send_bytes),
                                         reinterpret_cast<const long long*>(send_offset),
                                         reinterpret_cast<const long long*>(recv_offset), R,
                                         reinterpret_cast<unsigned char*>(ctx->ws) + workspace_bytes(ctx->shape) -
                                             collective_table_bytes(),
                                         ctx->ws,
                                         collective_queue(ctx), ctx->n_sm, ctx->trace, static_cast<cudaStream_t>(stream));
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        ctx->launches += 2;                // table kernel + copy kernel
    }
    return err == cudaSuccess ? STRATA_OK : STRATA_ERR_CUDA;
}

strata_status strata_reducescatter(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t elems_per_slice,
                                   void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    if (elems_per_slice % 8 != 0) return STRATA_ERR_SHAPE;
    // out, flat over [R][S], is the sum over the peers of their flat [R][S] inputs
    return run_reduce(ctx, in, out, (unsigned long long)R * elems_per_slice, R, 1, stream);
}

strata_status strata_allreduce(strata_ctx* ctx, int32_t R, const void* in, void* out, size_t elems, void* stream)
{
    strata_status st = collective_prologue(ctx, R, in, out);
    if (st != STRATA_OK) return st;
    return run_reduce(ctx, in, out, elems, R, R, stream);
}

strata_status strata_moe_recv_view(strata_ctx* ctx, const int32_t* h_rank_offset, int rank, void* recv,
                                   void** rank_base, int64_t* rows)
{
    if (!ctx || !h_rank_offset || !recv || !rank_base || !rows) return STRATA_ERR_INVALID_ARG;
    const strata_moe_shape& s = ctx->shape;
    if (rank < 0 || rank >= s.R) return STRATA_ERR_INVALID_ARG;
    const int64_t lo = h_rank_offset[rank], hi = h_rank_offset[rank + 1];
    if (lo < 0 || hi < lo) return STRATA_ERR_INVALID_ARG;
    const size_t row_bytes = s.dispatch_dtype == STRATA_FP8_E4M3_B128 ? (size_t)s.H : (size_t)s.H * 2;
    *rank_base = static_cast<unsigned char*>(recv) + (size_t)lo * row_bytes;
    *rows = hi - lo;
    return STRATA_OK;
}

strata_status strata_device_status(strata_ctx* ctx, void* stream, strata_status* out)
{
    if (!ctx || !out) return STRATA_ERR_INVALID_ARG;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyAsync(&word, ctx->ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return STRATA_ERR_CUDA;
    }
    if (word != 0) {
        // clear the status word; after an error also the ticket and the work-claim counters, which a
        // kernel that gave up may have left non-zero (header words 0..7)
        if (cudaMemsetAsync(ctx->ws, 0, 8 * sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
    }
    *out = static_cast<strata_status>(word);
    return STRATA_OK;
}

strata_status strata_moe_roundtrip_host(strata_ctx* ctx, const strata_moe_device_buffers* dev, const int32_t* h_ids,
                                        const void* h_x, const float* h_w, void* h_out, void* stream)
{
    if (!ctx || !dev || !h_ids || !h_x || !h_w || !h_out) return STRATA_ERR_INVALID_ARG;
    if (!dev->ids || !dev->x || !dev->w || !dev->recv || !dev->out) return STRATA_ERR_INVALID_ARG;
    strata_status rc = check_layout_ptrs(&dev->layout, true);
    if (rc != STRATA_OK) return rc;
    const strata_moe_shape& s = ctx->shape;
    if (s.dispatch_dtype != STRATA_BF16) return STRATA_ERR_SHAPE;
    if (!aligned16(dev->x) || !aligned16(dev->recv) || !aligned16(dev->out)) return STRATA_ERR_ALIGNMENT;
    if (!ctx->ws) return STRATA_ERR_WORKSPACE;
    const size_t n_tok = (size_t)s.R * s.T, n = n_tok * s.K, row_bytes = (size_t)s.H * 2;
    const size_t n_recv = (size_t)recv_rows(s);
    {
        std::lock_guard<std::mutex> lk(ctx->mu);
        if (!region_contains(ctx, dev->recv, n_recv * row_bytes)) return STRATA_ERR_NOT_REGISTERED;
    }
    if (ctx->device < 0) return STRATA_ERR_CUDA;
    DeviceGuard g(ctx->device);
    if (!g.ok) return STRATA_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // Token chunks of about 64 MB of x: chunk c+1 travels to the device while chunk c is dispatched
    // and combined and chunk c-1 travels back (the two copy directions use separate engines).
    const size_t chunk_tok = std::max<size_t>(1, std::min(n_tok, ((size_t)64 << 20) / row_bytes));
    const size_t n_chunks = (n_tok + chunk_tok - 1) / chunk_tok;
#define STRATA_TRY(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return STRATA_ERR_CUDA; } } while (0)
    if (!ctx->s_in) {
        STRATA_TRY(cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking));
        STRATA_TRY(cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking));
        STRATA_TRY(cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming));
        STRATA_TRY(cudaEventCreateWithFlags(&ctx->ev_out, cudaEventDisableTiming));
    }
    while (ctx->ev_in.size() < n_chunks) {
        cudaEvent_t a = nullptr, b = nullptr;
        STRATA_TRY(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
        ctx->ev_in.push_back(a);
        STRATA_TRY(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
        ctx->ev_done.push_back(b);
    }

    // The copy-in stream starts where the caller's stream is now.  The small copies go first: copies
    // in one direction are served in the order they were issued, whatever their stream.
    STRATA_TRY(cudaEventRecord(ctx->ev_entry, st));
    STRATA_TRY(cudaMemcpyAsync(dev->ids, h_ids, n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    STRATA_TRY(cudaMemcpyAsync(dev->w, h_w, n * sizeof(float), cudaMemcpyHostToDevice, st));
    rc = strata_moe_layout(ctx, dev->ids, &dev->layout, stream);
    if (rc != STRATA_OK) return rc;
    STRATA_TRY(cudaStreamWaitEvent(ctx->s_in, ctx->ev_entry, 0));
    const unsigned char* hx = static_cast<const unsigned char*>(h_x);
    unsigned char* dx = static_cast<unsigned char*>(dev->x);
    for (size_t c = 0; c < n_chunks; ++c) {
        const size_t a = c * chunk_tok, cnt = std::min(chunk_tok, n_tok - a);
        STRATA_TRY(cudaMemcpyAsync(dx + a * row_bytes, hx + a * row_bytes, cnt * row_bytes, cudaMemcpyHostToDevice,
                                   ctx->s_in));
        STRATA_TRY(cudaEventRecord(ctx->ev_in[c], ctx->s_in));
    }

    unsigned char* dout = static_cast<unsigned char*>(dev->out);
    unsigned char* hout = static_cast<unsigned char*>(h_out);
    for (size_t c = 0; c < n_chunks; ++c) {
        const size_t a = c * chunk_tok, cnt = std::min(chunk_tok, n_tok - a);
        strata_moe_shape sub = s;             // the chunk as a one-rank batch of cnt tokens
        sub.R = 1;
        sub.T = (int32_t)cnt;
        STRATA_TRY(cudaStreamWaitEvent(st, ctx->ev_in[c], 0));
        WorkQueue dq, cq;
        {
            std::lock_guard<std::mutex> lk(ctx->mu);
            dq = dispatch_queue(ctx);
            cq = combine_queue(ctx);
        }
        cudaError_t err = launch_dispatch_bf16(sub, dev->layout.dst_row + a * s.K, dx + a * row_bytes, dev->recv, n_recv,
                                               ctx->ws, dq, ctx->n_sm, TraceBuf{nullptr, 0, nullptr, 0, 0}, false, st);
        if (err == cudaSuccess)
            err = launch_combine(sub, dev->layout.dst_row + a * s.K, dev->recv, n_recv, dev->w + a * s.K,
                                 dout + a * row_bytes, ctx->ws, cq, ctx->n_sm, TraceBuf{nullptr, 0, nullptr, 0, 0}, st);
        {
            std::lock_guard<std::mutex> lk(ctx->mu);
            ctx->launches += 2;
        }
        if (err != cudaSuccess) {
            cudaGetLastError();
            return STRATA_ERR_CUDA;
        }
        STRATA_TRY(cudaEventRecord(ctx->ev_done[c], st));
        STRATA_TRY(cudaStreamWaitEvent(ctx->s_out, ctx->ev_done[c], 0));
        STRATA_TRY(cudaMemcpyAsync(hout + a * row_bytes, dout + a * row_bytes, cnt * row_bytes, cudaMemcpyDeviceToHost,
                                   ctx->s_out));
    }
    STRATA_TRY(cudaEventRecord(ctx->ev_out, ctx->s_out));
    STRATA_TRY(cudaStreamWaitEvent(st, ctx->ev_out, 0));
    STRATA_TRY(cudaStreamSynchronize(st));
#undef STRATA_TRY
    return STRATA_OK;
}

}  // extern "C"
