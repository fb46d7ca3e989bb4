// C ABI of libwash.so: argument checks, the context's tables, and the launches.
// The entry points are documented in include/wash.h.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/wash.h"
#include "wash_internal.h"

namespace wash {
uint64_t launch_count();
}

using wash::SegEntry;

namespace {

thread_local std::string g_last_error = "";

int fail(int code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_last_error = buf;
    return code;
}

int cuda_fail(cudaError_t err, const char *what)
{
    return fail(WASH_ERR_CUDA, "%s: %s", what, cudaGetErrorString(err));
}

constexpr int kSlots = 4;   // pinned staging slots for table uploads
constexpr double kEarlyShare = 0.3;   // expected share of selected coordinates from which the streaming kernel's early flavour is launched (N > 16)
constexpr int kPipeChunks = 32;   // wash_step_host cuts a large population into at most this many coordinate ranges

// makes `device` current for the lifetime of the guard
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int device)
    {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != device) {
            err = cudaSetDevice(device);
            switched = (err == cudaSuccess);
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

}  // namespace

struct wash_ctx {
    int N = 0, layout = 0, device = 0, n_seg = 0;
    std::vector<int64_t> numel, offset, coord_begin;
    std::vector<uint32_t> tensor_id;
    int64_t padded_P = 0;
    uint32_t n_groups = 0, n_tiles = 0;

    std::vector<SegEntry> seg_host;        // thresholds as last uploaded
    bool seg_uploaded = false;
    SegEntry *seg_dev = nullptr;
    uint32_t *tile_first_dev = nullptr;
    SegEntry *seg_pinned[kSlots] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t slot_event[kSlots] = {nullptr, nullptr, nullptr, nullptr};
    bool slot_used[kSlots] = {false, false, false, false};
    int next_slot = 0;

    void *stack_ptr[2] = {nullptr, nullptr};
    int stack_dtype[2] = {0, 0};

    uint32_t *status_dev = nullptr;
    wash_stats *stats_dev = nullptr;       // for wash_step_host
    wash::StatSlot *stat_slots_dev = nullptr;
    double *sq_slots_dev = nullptr;        // partial sums of wash_shuffle_consensus, allocated on first use, zero between calls
    double expected_selected = 0.0;        // sum over tensors of numel * thr / 2^32, for the current thresholds
    void *avg_dev = nullptr;               // for wash_step_host, allocated on first use
    size_t avg_bytes = 0;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;   // for wash_step_host's pipeline, created on first use
    cudaEvent_t pipe_event[2 * kPipeChunks + 2] = {};

    int mode = WASH_MODE_STREAM;
    wash::LaunchShape shape{0, 0, 148};

    // one model per device (wash_exchange_*)
    int x_self = -1;
    void *x_row[2] = {nullptr, nullptr};
    int x_dtype[2] = {0, 0};
    uint32_t *x_mask = nullptr;            // a byte per group, whole warp tiles
    uint32_t *x_warp_total = nullptr;      // [x_blocks * kExchangeWarps][N + 1]
    uint32_t *x_block_total = nullptr;     // [x_blocks][N + 1]
    uint32_t x_wtiles = 0, x_blocks = 0;
    void **x_staging[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // [parity][stack]: device array of N pointers
    int64_t x_capacity[2][2] = {{0, 0}, {0, 0}};
    void *x_own[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};        // staging buffers this library allocated
    std::vector<void *> x_opened;          // peers' buffers mapped by wash_exchange_staging_open
    bool x_opened_set[2][2] = {{false, false}, {false, false}};   // [parity][stack]: that set's peers are mapped
    bool x_planned = false;
    uint64_t x_step = 0, x_seed = 0;
};

namespace {

void release(wash_ctx *ctx)
{
    if (!ctx) return;
    DeviceGuard guard(ctx->device);
    if (ctx->seg_dev) cudaFree(ctx->seg_dev);
    if (ctx->tile_first_dev) cudaFree(ctx->tile_first_dev);
    if (ctx->status_dev) cudaFree(ctx->status_dev);
    if (ctx->stats_dev) cudaFree(ctx->stats_dev);
    if (ctx->stat_slots_dev) cudaFree(ctx->stat_slots_dev);
    if (ctx->sq_slots_dev) cudaFree(ctx->sq_slots_dev);
    if (ctx->avg_dev) cudaFree(ctx->avg_dev);
    if (ctx->x_mask) cudaFree(ctx->x_mask);
    if (ctx->x_warp_total) cudaFree(ctx->x_warp_total);
    if (ctx->x_block_total) cudaFree(ctx->x_block_total);
    for (auto &set : ctx->x_staging)
        for (void **ptrs : set)
            if (ptrs) cudaFree(ptrs);
    for (void *peer : ctx->x_opened) cudaIpcCloseMemHandle(peer);
    for (auto &set : ctx->x_own)
        for (void *own : set)
            if (own) cudaFree(own);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    for (cudaEvent_t e : ctx->pipe_event)
        if (e) cudaEventDestroy(e);
    for (int s = 0; s < kSlots; ++s) {
        if (ctx->seg_pinned[s]) cudaFreeHost(ctx->seg_pinned[s]);
        if (ctx->slot_event[s]) cudaEventDestroy(ctx->slot_event[s]);
    }
    delete ctx;
}

wash::PopView view_of(const wash_ctx *ctx)
{
    wash::PopView v;
    v.N = ctx->N;
    v.layout = ctx->layout;
    v.padded_P = ctx->padded_P;
    v.n_groups = ctx->n_groups;
    v.n_seg = ctx->n_seg;
    v.seg = ctx->seg_dev;
    v.tile_first = ctx->tile_first_dev;
    return v;
}

size_t elem_bytes(int dtype) { return dtype == WASH_BF16 ? 2 : 4; }

// floor(p * 2^32) for p in [0, 1]; the product is exact in binary64
uint64_t threshold_of(double p) { return static_cast<uint64_t>(std::floor(p * 4294967296.0)); }

// Brings the device copy of the segment table up to date with the call's
// probabilities (uploaded, in stream order, only when they changed).
int sync_table(wash_ctx *ctx, double p, const double *p_layer, cudaStream_t stream)
{
    // every probability is checked before the first threshold of the host mirror changes: a
    // rejected call must leave the mirror equal to the device table
    for (int s = 0; s < ctx->n_seg; ++s) {
        const double ps = p_layer ? p_layer[s] : p;
        if (!(ps >= 0.0 && ps <= 1.0)) return fail(WASH_ERR_ARG, "probability of tensor %d is %g, not in [0,1]", s, ps);
    }
    bool changed = !ctx->seg_uploaded;
    for (int s = 0; s < ctx->n_seg; ++s) {
        const uint64_t thr = threshold_of(p_layer ? p_layer[s] : p);
        if (thr != ctx->seg_host[s].thr) {
            ctx->seg_host[s].thr = thr;
            changed = true;
        }
    }
    if (!changed) return WASH_OK;
    ctx->seg_uploaded = false;   // until the copy below is queued, the mirror is ahead of the device table
    ctx->expected_selected = 0.0;
    for (int s = 0; s < ctx->n_seg; ++s)
        ctx->expected_selected += static_cast<double>(ctx->seg_host[s].numel) * static_cast<double>(ctx->seg_host[s].thr) / 4294967296.0;
    const int slot = ctx->next_slot;
    ctx->next_slot = (slot + 1) % kSlots;
    if (ctx->slot_used[slot]) {   // the copy that last read this slot must be done
        cudaError_t err = cudaEventSynchronize(ctx->slot_event[slot]);
        if (err != cudaSuccess) return cuda_fail(err, "cudaEventSynchronize(table slot)");
    }
    const size_t bytes = sizeof(SegEntry) * static_cast<size_t>(ctx->n_seg);
    std::memcpy(ctx->seg_pinned[slot], ctx->seg_host.data(), bytes);
    cudaError_t err = cudaMemcpyAsync(ctx->seg_dev, ctx->seg_pinned[slot], bytes, cudaMemcpyHostToDevice, stream);
    if (err != cudaSuccess) return cuda_fail(err, "cudaMemcpyAsync(segment table)");
    err = cudaEventRecord(ctx->slot_event[slot], stream);
    if (err != cudaSuccess) return cuda_fail(err, "cudaEventRecord(table slot)");
    ctx->slot_used[slot] = true;
    ctx->seg_uploaded = true;
    return WASH_OK;
}

int ensure_table(wash_ctx *ctx, cudaStream_t stream)
{
    if (ctx->seg_uploaded) return WASH_OK;
    std::vector<double> zeros(static_cast<size_t>(ctx->n_seg), 0.0);
    return sync_table(ctx, 0.0, zeros.data(), stream);
}

// which: 0 = parameters, 1 = optimizer state, 2 = both
int shuffle_impl(wash_ctx *ctx, int which, uint64_t step, double p, const double *p_layer, uint64_t seed,
                 void *stream_v, wash_stats *stats, uint32_t group_lo = 0, uint32_t group_hi = 0xFFFFFFFFu,
                 const wash::SqArgs *sq = nullptr, double *sq_out = nullptr)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (step >> 56) return fail(WASH_ERR_ARG, "step must be below 2^56");
    if (!p_layer && !(p >= 0.0 && p <= 1.0)) return fail(WASH_ERR_ARG, "p is %g, not in [0,1]", p);
    void *a = nullptr, *b = nullptr;
    int a_dtype = wash::kDtypeNone, b_dtype = wash::kDtypeNone;
    if (which == 0 || which == 2) {
        a = ctx->stack_ptr[WASH_STACK_PARAMS];
        a_dtype = ctx->stack_dtype[WASH_STACK_PARAMS];
        if (!a) return fail(WASH_ERR_STATE, "parameter stack is not bound");
    }
    if (which == 1 || which == 2) {
        void *o = ctx->stack_ptr[WASH_STACK_OPT];
        if (!o) return fail(WASH_ERR_STATE, "optimizer-state stack is not bound");
        if (which == 1) { a = o; a_dtype = ctx->stack_dtype[WASH_STACK_OPT]; }
        else { b = o; b_dtype = ctx->stack_dtype[WASH_STACK_OPT]; }
    }
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int rc = sync_table(ctx, p, p_layer, stream);
    if (rc != WASH_OK) return rc;

    wash::ShuffleArgs args;
    args.pop = view_of(ctx);
    args.a = a;
    args.b = b;
    args.group_lo = group_lo;
    args.group_hi = group_hi < ctx->n_groups ? group_hi : ctx->n_groups;
    args.keys = wash::philox_keys(seed);
    args.step_lo = static_cast<uint32_t>(step);
    args.step_hi8 = static_cast<uint32_t>(step >> 32) << 8;
    args.stats = reinterpret_cast<unsigned long long *>(stats);
    int mode = ctx->mode;
    // Counters: blocks that selected something add to the caller's two words directly when
    // that stays well below one atomic per nanosecond on one address (measured limit);
    // otherwise through the partial-sum slots and a small flush kernel.
    {
        const double bytes = static_cast<double>(ctx->N) * static_cast<double>(ctx->padded_P) *
                             (elem_bytes(a_dtype) + (b ? elem_bytes(b_dtype) : 0));
        const double kernel_ns = bytes / 6000.0 + 2000.0;
        const double reporting_blocks = std::fmin(ctx->expected_selected, static_cast<double>(ctx->n_groups) / 64.0);
        args.stat_slots = (2.0 * reporting_blocks / kernel_ns > 0.35) ? ctx->stat_slots_dev : nullptr;
        // WASH_MODE_AUTO: the expected share of selected coordinates decides
        if (ctx->mode == WASH_MODE_AUTO) {
            double coordinates = 0.0;
            for (int s = 0; s < ctx->n_seg; ++s) coordinates += static_cast<double>(ctx->seg_host[s].numel);
            // measured crossovers of the two kernels (fp32, 2^25-2^26 coordinates): serving a coordinate costs a
            // 128-byte DRAM access per model and stack in [N][P], one or two for all N models in [P][N]; and a
            // small population leaves the streaming kernel bound by issue slots, not by the stack's bytes.
            // [N][P]: N = 2 17 %, 4 10 %, 8 4 %, 16 2.5 %, 32 3-5 %; [P][N]: N <= 8 above 30 %, 16 10 %, 32 12 %
            const double share = ctx->layout == WASH_LAYOUT_PN ? (ctx->N <= 8 ? 0.30 : 0.10) : std::fmax(0.03, 0.35 / ctx->N);
            mode = ctx->expected_selected < share * coordinates ? WASH_MODE_SPARSE : WASH_MODE_STREAM;
        }
        double coordinates = 0.0;
        for (int s = 0; s < ctx->n_seg; ++s) coordinates += static_cast<double>(ctx->seg_host[s].numel);
        // [P][N], even N: the streaming kernel pads its shared-memory image against bank conflicts
        // once a fifth of the coordinates is expected to be served from it
        args.expected_share = coordinates > 0.0 ? static_cast<float>(ctx->expected_selected / coordinates) : 0.f;
        if (ctx->layout == WASH_LAYOUT_PN && !(ctx->N & 1)) args.pn_pad = ctx->expected_selected >= 0.2 * coordinates ? 4u : 0u;
        // The streaming kernel's early flavour (permutations drawn while the copies are in flight, dense
        // serving for N > 16) costs registers and, for N > 16, three more permutation columns of shared
        // memory per thread: measured, it pays only for large populations of which most coordinates are
        // served (N = 32, p = 1: 15.7 -> 10.4 ms, [P][N] 29.8 -> 13.3 ms; slower by 0-15 % everywhere else).
        args.early = ctx->N > 16 && ctx->expected_selected >= kEarlyShare * coordinates;
        if (ctx->shape.blocks_per_sm == -2) args.early = false;   // tuning override (wash_set_launch)
        if (ctx->shape.blocks_per_sm == -3) args.early = true;
        if (sq) {   // the statistic is gathered by the streaming kernel only
            mode = WASH_MODE_STREAM;
            args.stat_slots = ctx->stat_slots_dev;
            args.sq = *sq;
        }
        if (mode == WASH_MODE_SPARSE) args.stat_slots = nullptr;   // one wave of large blocks: a few hundred atomics at most
    }
    args.status = ctx->status_dev;
    bool supported = false;
    cudaError_t err = wash::launch_shuffle(args, a_dtype, b_dtype, mode, ctx->shape, stream, &supported);
    if (err != cudaSuccess) return cuda_fail(err, "shuffle kernel launch");
    if (!supported) return fail(WASH_ERR_UNSUPPORTED, "no shuffle kernel for dtypes (%d, %d)", a_dtype, b_dtype);
    if (sq && (err = wash::launch_sq_flush(*sq, ctx->N, sq_out, stream)) != cudaSuccess) return cuda_fail(err, "consensus flush launch");
    return WASH_OK;
}

int reduce_impl(wash_ctx *ctx, int op, int stack, void *out, int out_dtype, float alpha, int tensor_lo,
                int tensor_hi, double *sq_out, void *stream_v, uint32_t group_lo = 0, uint32_t group_hi = 0xFFFFFFFFu)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (!ctx->stack_ptr[stack]) return fail(WASH_ERR_STATE, "stack %d is not bound", stack);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int rc = ensure_table(ctx, stream);
    if (rc != WASH_OK) return rc;
    wash::ReduceArgs args;
    args.pop = view_of(ctx);
    args.stack = ctx->stack_ptr[stack];
    args.out = out;
    args.alpha = alpha;
    args.one_minus_alpha = 1.0f - alpha;
    args.group_lo = ctx->seg_host[static_cast<size_t>(tensor_lo)].group_begin;
    args.group_hi = ctx->seg_host[static_cast<size_t>(tensor_hi) - 1].group_end;
    if (group_lo > args.group_lo) args.group_lo = group_lo;   // optional narrowing to a range of groups
    if (group_hi < args.group_hi) args.group_hi = group_hi;
    if (args.group_lo >= args.group_hi) return WASH_OK;
    args.sq_out = sq_out;
    args.status = ctx->status_dev;
    bool supported = false;
    cudaError_t err = wash::launch_reduce(args, op, ctx->stack_dtype[stack], out_dtype, ctx->shape, stream, &supported);
    if (err != cudaSuccess) return cuda_fail(err, "kernel launch");
    if (!supported) return fail(WASH_ERR_UNSUPPORTED, "no kernel for dtype %d -> %d", ctx->stack_dtype[stack], out_dtype);
    return WASH_OK;
}

}  // namespace

extern "C" {

int wash_create_segments(wash_ctx **out, int32_t N, int32_t n_segments, const int64_t *numel,
                         const uint32_t *tensor_id, const int64_t *coord_begin, int32_t layout, int32_t device)
{
    if (!out) return fail(WASH_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (N < 2 || N > WASH_MAX_N) return fail(WASH_ERR_ARG, "N = %d, must be in [2, %d]", N, WASH_MAX_N);
    if (n_segments < 1 || !numel) return fail(WASH_ERR_ARG, "need at least one tensor");
    if (layout != WASH_LAYOUT_NP && layout != WASH_LAYOUT_PN) return fail(WASH_ERR_ARG, "unknown layout %d", layout);
    if (device < 0) return fail(WASH_ERR_ARG, "device = %d", device);

    wash_ctx *ctx = new (std::nothrow) wash_ctx;
    if (!ctx) return fail(WASH_ERR_ALLOC, "out of host memory");
    ctx->N = N;
    ctx->layout = layout;
    ctx->device = device;
    ctx->n_seg = n_segments;
    int64_t cur = 0;
    for (int s = 0; s < n_segments; ++s) {
        const int64_t d = numel[s];
        const int64_t cb = coord_begin ? coord_begin[s] : 0;
        if (d <= 0 || d >= (int64_t(1) << 32)) { delete ctx; return fail(WASH_ERR_ARG, "numel[%d] = %lld, must be in (0, 2^32)", s, (long long)d); }
        if (cb < 0 || (cb & 3) || cb + d > (int64_t(1) << 32)) { delete ctx; return fail(WASH_ERR_ARG, "coord_begin[%d] = %lld must be a multiple of 4 with coord_begin + numel <= 2^32", s, (long long)cb); }
        ctx->numel.push_back(d);
        ctx->offset.push_back(cur);
        ctx->coord_begin.push_back(cb);
        ctx->tensor_id.push_back(tensor_id ? tensor_id[s] : static_cast<uint32_t>(s));
        cur += (d + WASH_ALIGN_ELEMS - 1) / WASH_ALIGN_ELEMS * WASH_ALIGN_ELEMS;
        if (cur / 4 >= (int64_t(1) << 31)) { delete ctx; return fail(WASH_ERR_ARG, "row too long: more than 2^33 elements"); }
    }
    ctx->padded_P = cur;
    ctx->n_groups = static_cast<uint32_t>(cur / 4);
    ctx->n_tiles = (ctx->n_groups + (1u << wash::kTileShift) - 1) >> wash::kTileShift;

    ctx->seg_host.resize(static_cast<size_t>(n_segments));
    for (int s = 0; s < n_segments; ++s) {
        SegEntry &e = ctx->seg_host[static_cast<size_t>(s)];
        e.group_begin = static_cast<uint32_t>(ctx->offset[s] / 4);
        e.group_end = static_cast<uint32_t>((s + 1 < n_segments ? ctx->offset[s + 1] : cur) / 4);
        e.tensor_id = ctx->tensor_id[s];
        e.cgroup_begin = static_cast<uint32_t>(ctx->coord_begin[s] / 4);
        e.numel = static_cast<uint32_t>(ctx->numel[s]);
        e.reserved = 0;
        e.thr = 0;
    }
    std::vector<uint32_t> tile_first(ctx->n_tiles);
    {
        uint32_t s = 0;
        for (uint32_t t = 0; t < ctx->n_tiles; ++t) {
            const uint32_t g = t << wash::kTileShift;
            while (g >= ctx->seg_host[s].group_end) ++s;
            tile_first[t] = s;
        }
    }

    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) { delete ctx; return cuda_fail(guard.err, "cudaSetDevice"); }
    cudaError_t err = cudaSuccess;
    int sm_count = 0;
    err = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device);
    if (err != cudaSuccess) { delete ctx; return cuda_fail(err, "cudaDeviceGetAttribute"); }
    ctx->shape.sm_count = sm_count;
    const size_t seg_bytes = sizeof(SegEntry) * static_cast<size_t>(n_segments);
    if ((err = cudaMalloc(&ctx->seg_dev, seg_bytes)) != cudaSuccess ||
        (err = cudaMalloc(&ctx->tile_first_dev, sizeof(uint32_t) * ctx->n_tiles)) != cudaSuccess ||
        (err = cudaMalloc(&ctx->status_dev, sizeof(uint32_t))) != cudaSuccess ||
        (err = cudaMalloc(&ctx->stats_dev, sizeof(wash_stats))) != cudaSuccess ||
        (err = cudaMalloc(&ctx->stat_slots_dev, sizeof(wash::StatSlot) * wash::kStatSlots)) != cudaSuccess) {
        release(ctx);
        cudaGetLastError();
        return fail(WASH_ERR_ALLOC, "device allocation failed: %s", cudaGetErrorString(err));
    }
    for (int s = 0; s < kSlots; ++s) {
        if ((err = cudaMallocHost(&ctx->seg_pinned[s], seg_bytes)) != cudaSuccess ||
            (err = cudaEventCreateWithFlags(&ctx->slot_event[s], cudaEventDisableTiming)) != cudaSuccess) {
            release(ctx);
            cudaGetLastError();
            return fail(WASH_ERR_ALLOC, "pinned allocation failed: %s", cudaGetErrorString(err));
        }
    }
    if ((err = cudaMemcpy(ctx->tile_first_dev, tile_first.data(), sizeof(uint32_t) * ctx->n_tiles, cudaMemcpyHostToDevice)) != cudaSuccess ||
        (err = cudaMemset(ctx->status_dev, 0, sizeof(uint32_t))) != cudaSuccess ||
        (err = cudaMemset(ctx->stats_dev, 0, sizeof(wash_stats))) != cudaSuccess ||
        (err = cudaMemset(ctx->stat_slots_dev, 0, sizeof(wash::StatSlot) * wash::kStatSlots)) != cudaSuccess) {
        release(ctx);
        return cuda_fail(err, "table upload");
    }
    *out = ctx;
    return WASH_OK;
}

int wash_create(wash_ctx **out, int32_t N, int32_t n_tensors, const int64_t *numel, int32_t layout, int32_t device)
{
    return wash_create_segments(out, N, n_tensors, numel, nullptr, nullptr, layout, device);
}

int wash_destroy(wash_ctx *ctx)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    release(ctx);
    return WASH_OK;
}

int wash_stack_elems(const wash_ctx *ctx, int64_t *padded_P, int64_t *offsets)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (padded_P) *padded_P = ctx->padded_P;
    if (offsets)
        for (int s = 0; s < ctx->n_seg; ++s) offsets[s] = ctx->offset[s];
    return WASH_OK;
}

int wash_bind(wash_ctx *ctx, int32_t stack, int32_t dtype, void *dev_ptr, int64_t n_elems)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (!dev_ptr) { ctx->stack_ptr[stack] = nullptr; return WASH_OK; }
    if (dtype != WASH_F32 && dtype != WASH_BF16) return fail(WASH_ERR_ARG, "unknown dtype %d", dtype);
    if (n_elems != static_cast<int64_t>(ctx->N) * ctx->padded_P)
        return fail(WASH_ERR_ARG, "stack has %lld elements, population needs N * padded_P = %lld", (long long)n_elems,
                    (long long)(static_cast<int64_t>(ctx->N) * ctx->padded_P));
    if (reinterpret_cast<uintptr_t>(dev_ptr) & 15) return fail(WASH_ERR_ARG, "stack pointer must be 16-byte aligned");
    ctx->stack_ptr[stack] = dev_ptr;
    ctx->stack_dtype[stack] = dtype;
    return WASH_OK;
}

int wash_set_mode(wash_ctx *ctx, int32_t mode)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (mode != WASH_MODE_STREAM && mode != WASH_MODE_SPARSE && mode != WASH_MODE_AUTO) return fail(WASH_ERR_ARG, "unknown mode %d", mode);
    ctx->mode = mode;
    return WASH_OK;
}

int wash_set_launch(wash_ctx *ctx, int32_t threads, int32_t blocks_per_sm)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (threads != 0 && (threads < 32 || threads > 256 || (threads & 31))) return fail(WASH_ERR_ARG, "threads = %d: need 0 or a multiple of 32 in [32, 256]", threads);
    ctx->shape.threads = threads;
    ctx->shape.blocks_per_sm = blocks_per_sm;
    return WASH_OK;
}

int wash_layer_probs(int32_t L, double p, int32_t schedule, double *out)
{
    if (L < 1 || !out) return fail(WASH_ERR_ARG, "need L >= 1 and an output array");
    if (!(p >= 0.0 && p <= 1.0)) return fail(WASH_ERR_ARG, "p is %g, not in [0,1]", p);
    if (schedule < WASH_SCHEDULE_DECREASING || schedule > WASH_SCHEDULE_INCREASING) return fail(WASH_ERR_ARG, "unknown schedule %d", schedule);
    for (int l = 0; l < L; ++l) {
        if (L == 1 || schedule == WASH_SCHEDULE_CONSTANT) { out[l] = p; continue; }
        const double depth = static_cast<double>(l) / static_cast<double>(L - 1);
        out[l] = schedule == WASH_SCHEDULE_DECREASING ? p * (1.0 - depth) : p * depth;
    }
    return WASH_OK;
}

int wash_shuffle(wash_ctx *ctx, uint64_t step, double p, const double *p_layer, uint64_t seed, void *stream, wash_stats *stats)
{
    return shuffle_impl(ctx, 0, step, p, p_layer, seed, stream, stats);
}

int wash_shuffle_opt_state(wash_ctx *ctx, uint64_t step, double p, const double *p_layer, uint64_t seed, void *stream, wash_stats *stats)
{
    return shuffle_impl(ctx, 1, step, p, p_layer, seed, stream, stats);
}

int wash_shuffle_both(wash_ctx *ctx, uint64_t step, double p, const double *p_layer, uint64_t seed, void *stream, wash_stats *stats)
{
    return shuffle_impl(ctx, 2, step, p, p_layer, seed, stream, stats);
}

int wash_shuffle_consensus(wash_ctx *ctx, int32_t stacks, uint64_t step, double p, const double *p_layer, uint64_t seed,
                           void *stream, wash_stats *stats, int32_t n_ranges, const int32_t *tensor_bounds, double *dev_sq_out)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stacks != WASH_STACK_PARAMS && stacks != WASH_STACK_OPT && stacks != WASH_STACK_BOTH) return fail(WASH_ERR_ARG, "stacks must be WASH_STACK_PARAMS, WASH_STACK_OPT or WASH_STACK_BOTH");
    if (n_ranges < 1 || n_ranges > WASH_MAX_CONSENSUS_RANGES) return fail(WASH_ERR_ARG, "n_ranges = %d, must be in [1, %d]", n_ranges, WASH_MAX_CONSENSUS_RANGES);
    if (!tensor_bounds || !dev_sq_out) return fail(WASH_ERR_ARG, "tensor_bounds and dev_sq_out must not be NULL");
    wash::SqArgs sq;
    for (int r = 0; r <= n_ranges; ++r) {
        const int32_t b = tensor_bounds[r];
        if (b < 0 || b > ctx->n_seg || (r > 0 && b < tensor_bounds[r - 1]))
            return fail(WASH_ERR_ARG, "tensor_bounds must ascend within [0, %d]; entry %d is %d", ctx->n_seg, r, b);
        sq.seg_bound[r] = static_cast<uint32_t>(b);
    }
    for (int r = n_ranges + 1; r <= wash::kMaxSqRanges; ++r) sq.seg_bound[r] = sq.seg_bound[n_ranges];
    sq.n_ranges = n_ranges;
    sq.inv_n = 1.0 / static_cast<double>(ctx->N);
    if (!ctx->sq_slots_dev) {
        DeviceGuard guard(ctx->device);
        if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
        const size_t bytes = sizeof(double) * wash::kSqSlots * wash::kMaxSqRanges * static_cast<size_t>(ctx->N);
        cudaError_t err = cudaMalloc(&ctx->sq_slots_dev, bytes);
        if (err != cudaSuccess) {
            cudaGetLastError();
            ctx->sq_slots_dev = nullptr;
            return fail(WASH_ERR_ALLOC, "device allocation of the consensus partial sums failed: %s", cudaGetErrorString(err));
        }
        if ((err = cudaMemset(ctx->sq_slots_dev, 0, bytes)) != cudaSuccess) return cuda_fail(err, "cudaMemset(consensus partial sums)");
    }
    sq.slots = ctx->sq_slots_dev;
    return shuffle_impl(ctx, stacks, step, p, p_layer, seed, stream, stats, 0, 0xFFFFFFFFu, &sq, dev_sq_out);
}

int papa_ema(wash_ctx *ctx, int32_t stack, float alpha, void *stream)
{
    if (!(alpha > 0.0f && alpha < 1.0f)) return fail(WASH_ERR_ARG, "alpha is %g, must be in (0,1)", (double)alpha);
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    return reduce_impl(ctx, wash::kOpEma, stack, nullptr, WASH_F32, alpha, 0, ctx->n_seg, nullptr, stream);
}

int population_average(wash_ctx *ctx, int32_t stack, void *dev_out, int32_t out_dtype, void *stream)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (!dev_out || (reinterpret_cast<uintptr_t>(dev_out) & 15)) return fail(WASH_ERR_ARG, "dev_out must be a 16-byte aligned device pointer");
    if (out_dtype != WASH_F32 && out_dtype != WASH_BF16) return fail(WASH_ERR_ARG, "unknown out_dtype %d", out_dtype);
    return reduce_impl(ctx, wash::kOpAverage, stack, dev_out, out_dtype, 0.0f, 0, ctx->n_seg, nullptr, stream);
}

int papa_all(wash_ctx *ctx, int32_t stack, void *stream)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    return reduce_impl(ctx, wash::kOpPapaAll, stack, nullptr, WASH_F32, 0.0f, 0, ctx->n_seg, nullptr, stream);
}

int wash_consensus_sq(wash_ctx *ctx, int32_t stack, int32_t tensor_lo, int32_t tensor_hi, double *dev_sq_out, void *stream)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (!dev_sq_out) return fail(WASH_ERR_ARG, "dev_sq_out is NULL");
    if (tensor_lo < 0 || tensor_hi > ctx->n_seg || tensor_lo > tensor_hi) return fail(WASH_ERR_ARG, "tensor range [%d, %d) is not within [0, %d]", tensor_lo, tensor_hi, ctx->n_seg);
    if (tensor_lo == tensor_hi) return WASH_OK;
    return reduce_impl(ctx, wash::kOpConsensus, stack, nullptr, WASH_F32, 0.0f, tensor_lo, tensor_hi, dev_sq_out, stream);
}

int wash_step_host(wash_ctx *ctx, int32_t ops, void *host_params, void *host_opt, void *host_avg, uint64_t step,
                   double p, const double *p_layer, uint64_t seed, float alpha, void *stream_v, wash_stats *host_stats)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (!host_params) return fail(WASH_ERR_ARG, "host_params is NULL");
    if (ops & ~(WASH_OP_SHUFFLE | WASH_OP_EMA | WASH_OP_AVERAGE)) return fail(WASH_ERR_ARG, "unknown bits in ops");
    if ((ops & WASH_OP_AVERAGE) && !host_avg) return fail(WASH_ERR_ARG, "host_avg is NULL but WASH_OP_AVERAGE is set");
    if (!ctx->stack_ptr[WASH_STACK_PARAMS]) return fail(WASH_ERR_STATE, "parameter stack is not bound");
    if (host_opt && !ctx->stack_ptr[WASH_STACK_OPT]) return fail(WASH_ERR_STATE, "optimizer-state stack is not bound");
    if ((ops & WASH_OP_EMA) && !(alpha > 0.0f && alpha < 1.0f)) return fail(WASH_ERR_ARG, "alpha is %g, must be in (0,1)", (double)alpha);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int pd = ctx->stack_dtype[WASH_STACK_PARAMS];
    const size_t n_elems = static_cast<size_t>(ctx->N) * static_cast<size_t>(ctx->padded_P);
    const size_t p_bytes = n_elems * elem_bytes(pd);
    const size_t o_bytes = host_opt ? n_elems * elem_bytes(ctx->stack_dtype[WASH_STACK_OPT]) : 0;
    const size_t avg_bytes = static_cast<size_t>(ctx->padded_P) * elem_bytes(pd);
    cudaError_t err;
    if ((ops & WASH_OP_AVERAGE) && ctx->avg_bytes < avg_bytes) {
        if (ctx->avg_dev) cudaFree(ctx->avg_dev);
        ctx->avg_dev = nullptr;
        ctx->avg_bytes = 0;
        if ((err = cudaMalloc(&ctx->avg_dev, avg_bytes)) != cudaSuccess) {
            cudaGetLastError();
            return fail(WASH_ERR_ALLOC, "device allocation of the average row failed: %s", cudaGetErrorString(err));
        }
        ctx->avg_bytes = avg_bytes;
    }
    int rc;
    wash_stats st = {0, 0};
    // Large populations go through in kPipeChunks coordinate ranges so that the copy of one
    // range to the device, the kernels on the previous one and the copy of the one before
    // back to the host overlap (the PCIe link is full duplex, and the draws are keyed by
    // global coordinates, so a range can be processed on its own).
    if (ctx->n_groups >= (1u << 18)) {
        if (!ctx->copy_in) {
            if ((err = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking)) != cudaSuccess ||
                (err = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking)) != cudaSuccess)
                return cuda_fail(err, "cudaStreamCreate");
            for (cudaEvent_t &e : ctx->pipe_event)
                if ((err = cudaEventCreateWithFlags(&e, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(err, "cudaEventCreate");
        }
        // Once a copy is queued on the side streams, an error must not leave them running into the
        // caller's host buffers: the pipeline runs inside a lambda and every exit waits for all
        // three streams (their own status is ignored then; the first error is what is returned).
        auto pipeline = [&]() -> int {
            cudaEvent_t *ev_in = ctx->pipe_event, *ev_done = ctx->pipe_event + kPipeChunks;
            cudaEvent_t ev_start = ctx->pipe_event[2 * kPipeChunks], ev_out = ctx->pipe_event[2 * kPipeChunks + 1];
            if ((ops & WASH_OP_SHUFFLE) && (err = cudaMemsetAsync(ctx->stats_dev, 0, sizeof(wash_stats), stream)) != cudaSuccess) return cuda_fail(err, "cudaMemsetAsync(stats)");
            if ((ops & WASH_OP_AVERAGE) && (err = cudaMemsetAsync(ctx->avg_dev, 0, avg_bytes, stream)) != cudaSuccess) return cuda_fail(err, "cudaMemsetAsync(average row)");
            // the copy streams start after whatever the caller's stream has queued so far
            if ((err = cudaEventRecord(ev_start, stream)) != cudaSuccess ||
                (err = cudaStreamWaitEvent(ctx->copy_in, ev_start, 0)) != cudaSuccess ||
                (err = cudaStreamWaitEvent(ctx->copy_out, ev_start, 0)) != cudaSuccess) return cuda_fail(err, "pipeline set-up");
            // ranges of about 32 MiB of stack (8 at least, kPipeChunks at most): the first range's copy in and
            // the last range's copy out are the part of the transfers that nothing overlaps
            const size_t stack_bytes = p_bytes + o_bytes;
            int chunks = static_cast<int>(stack_bytes >> 25);
            chunks = chunks < 8 ? 8 : (chunks > kPipeChunks ? kPipeChunks : chunks);
            const uint32_t per = ((ctx->n_groups + chunks - 1) / chunks + 255u) & ~255u;   // groups per range
            // moves the elements [e0, e0 + count) of every model between a host and the device stack
            auto copy_range = [&](void *dst, const void *src, int dtype, size_t e0, size_t count, cudaMemcpyKind kind, cudaStream_t s) {
                const size_t eb = elem_bytes(dtype);
                if (ctx->layout == WASH_LAYOUT_NP) {
                    const size_t pitch = static_cast<size_t>(ctx->padded_P) * eb;
                    return cudaMemcpy2DAsync(static_cast<char *>(dst) + e0 * eb, pitch, static_cast<const char *>(src) + e0 * eb, pitch,
                                             count * eb, static_cast<size_t>(ctx->N), kind, s);
                }
                const size_t off = e0 * ctx->N * eb;
                return cudaMemcpyAsync(static_cast<char *>(dst) + off, static_cast<const char *>(src) + off, count * ctx->N * eb, kind, s);
            };
            const int od = ctx->stack_dtype[WASH_STACK_OPT];
            for (int k = 0; k < kPipeChunks; ++k) {
                const uint32_t g0 = static_cast<uint32_t>(k) * per;
                if (g0 >= ctx->n_groups) break;
                const uint32_t g1 = g0 + per < ctx->n_groups ? g0 + per : ctx->n_groups;
                const size_t e0 = 4ull * g0, count = 4ull * (g1 - g0);
                if ((err = copy_range(ctx->stack_ptr[WASH_STACK_PARAMS], host_params, pd, e0, count, cudaMemcpyHostToDevice, ctx->copy_in)) != cudaSuccess)
                    return cuda_fail(err, "copy of a parameter range to the device");
                if (host_opt && (err = copy_range(ctx->stack_ptr[WASH_STACK_OPT], host_opt, od, e0, count, cudaMemcpyHostToDevice, ctx->copy_in)) != cudaSuccess)
                    return cuda_fail(err, "copy of an optimizer-state range to the device");
                if ((err = cudaEventRecord(ev_in[k], ctx->copy_in)) != cudaSuccess || (err = cudaStreamWaitEvent(stream, ev_in[k], 0)) != cudaSuccess)
                    return cuda_fail(err, "pipeline event");
                if (ops & WASH_OP_SHUFFLE) {
                    rc = shuffle_impl(ctx, host_opt ? 2 : 0, step, p, p_layer, seed, stream, ctx->stats_dev, g0, g1);
                    if (rc != WASH_OK) return rc;
                }
                if (ops & WASH_OP_EMA) {
                    rc = reduce_impl(ctx, wash::kOpEma, WASH_STACK_PARAMS, nullptr, WASH_F32, alpha, 0, ctx->n_seg, nullptr, stream, g0, g1);
                    if (rc != WASH_OK) return rc;
                }
                if (ops & WASH_OP_AVERAGE) {
                    rc = reduce_impl(ctx, wash::kOpAverage, WASH_STACK_PARAMS, ctx->avg_dev, pd, 0.0f, 0, ctx->n_seg, nullptr, stream, g0, g1);
                    if (rc != WASH_OK) return rc;
                }
                if ((err = cudaEventRecord(ev_done[k], stream)) != cudaSuccess || (err = cudaStreamWaitEvent(ctx->copy_out, ev_done[k], 0)) != cudaSuccess)
                    return cuda_fail(err, "pipeline event");
                if ((err = copy_range(host_params, ctx->stack_ptr[WASH_STACK_PARAMS], pd, e0, count, cudaMemcpyDeviceToHost, ctx->copy_out)) != cudaSuccess)
                    return cuda_fail(err, "copy of a parameter range to the host");
                if (host_opt && (err = copy_range(host_opt, ctx->stack_ptr[WASH_STACK_OPT], od, e0, count, cudaMemcpyDeviceToHost, ctx->copy_out)) != cudaSuccess)
                    return cuda_fail(err, "copy of an optimizer-state range to the host");
                if ((ops & WASH_OP_AVERAGE) &&
                    (err = cudaMemcpyAsync(static_cast<char *>(host_avg) + e0 * elem_bytes(pd), static_cast<char *>(ctx->avg_dev) + e0 * elem_bytes(pd),
                                           count * elem_bytes(pd), cudaMemcpyDeviceToHost, ctx->copy_out)) != cudaSuccess)
                    return cuda_fail(err, "copy of an average range to the host");
            }
            // the caller's stream continues only when the last range is back on the host
            if ((err = cudaEventRecord(ev_out, ctx->copy_out)) != cudaSuccess || (err = cudaStreamWaitEvent(stream, ev_out, 0)) != cudaSuccess)
                return cuda_fail(err, "pipeline event");
            if ((ops & WASH_OP_SHUFFLE) && (err = cudaMemcpyAsync(&st, ctx->stats_dev, sizeof st, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
                return cuda_fail(err, "copy of the counters to the host");
            if ((err = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(err, "cudaStreamSynchronize");
            if (host_stats) *host_stats = st;
            return WASH_OK;
        };
        const int prc = pipeline();
        if (prc != WASH_OK) {
            const std::string first = g_last_error;
            cudaStreamSynchronize(ctx->copy_in);
            cudaStreamSynchronize(stream);
            cudaStreamSynchronize(ctx->copy_out);
            cudaGetLastError();
            g_last_error = first;
        }
        return prc;
    }
    if ((err = cudaMemcpyAsync(ctx->stack_ptr[WASH_STACK_PARAMS], host_params, p_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the parameter stack to the device");
    if (host_opt && (err = cudaMemcpyAsync(ctx->stack_ptr[WASH_STACK_OPT], host_opt, o_bytes, cudaMemcpyHostToDevice, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the optimizer-state stack to the device");
    if (ops & WASH_OP_SHUFFLE) {
        if ((err = cudaMemsetAsync(ctx->stats_dev, 0, sizeof(wash_stats), stream)) != cudaSuccess) return cuda_fail(err, "cudaMemsetAsync(stats)");
        rc = shuffle_impl(ctx, host_opt ? 2 : 0, step, p, p_layer, seed, stream, ctx->stats_dev);
        if (rc != WASH_OK) return rc;
    }
    if (ops & WASH_OP_EMA) {
        rc = papa_ema(ctx, WASH_STACK_PARAMS, alpha, stream);
        if (rc != WASH_OK) return rc;
    }
    if (ops & WASH_OP_AVERAGE) {
        if (avg_bytes % 16) { /* padded_P is a multiple of 8 elements, so this cannot happen */ }
        // padding of the row is never written by the kernel: give it a defined value
        if ((err = cudaMemsetAsync(ctx->avg_dev, 0, avg_bytes, stream)) != cudaSuccess) return cuda_fail(err, "cudaMemsetAsync(average row)");
        rc = population_average(ctx, WASH_STACK_PARAMS, ctx->avg_dev, pd, stream);
        if (rc != WASH_OK) return rc;
    }
    if ((err = cudaMemcpyAsync(host_params, ctx->stack_ptr[WASH_STACK_PARAMS], p_bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the parameter stack to the host");
    if (host_opt && (err = cudaMemcpyAsync(host_opt, ctx->stack_ptr[WASH_STACK_OPT], o_bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the optimizer-state stack to the host");
    if ((ops & WASH_OP_AVERAGE) && (err = cudaMemcpyAsync(host_avg, ctx->avg_dev, avg_bytes, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the average to the host");
    if ((ops & WASH_OP_SHUFFLE) && (err = cudaMemcpyAsync(&st, ctx->stats_dev, sizeof st, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(err, "copy of the counters to the host");
    if ((err = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(err, "cudaStreamSynchronize");
    if (host_stats) *host_stats = st;
    return WASH_OK;
}

// ---- one model per device ------------------------------------------------------------

}  // extern "C"

namespace {

// kernel arguments of the planned step; `need_rows`: at least one row must be bound
int exchange_args(wash_ctx *ctx, wash::ExchangeArgs *out)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (ctx->x_self < 0) return fail(WASH_ERR_STATE, "wash_exchange_bind has not been called");
    wash::ExchangeArgs &a = *out;
    a.pop = view_of(ctx);
    a.self = ctx->x_self;
    a.n_wtiles = ctx->x_wtiles;
    a.n_blocks = ctx->x_blocks;
    a.keys = wash::philox_keys(ctx->x_seed);
    a.step_lo = static_cast<uint32_t>(ctx->x_step);
    a.step_hi8 = static_cast<uint32_t>(ctx->x_step >> 32) << 8;
    a.mask = ctx->x_mask;
    a.warp_total = ctx->x_warp_total;
    a.block_total = ctx->x_block_total;
    const int parity = static_cast<int>(ctx->x_step & 1u);
    for (int k = 0; k < 2; ++k) {
        a.row[k] = ctx->x_row[k];
        a.dtype[k] = ctx->x_dtype[k];
        const int set = ctx->x_staging[parity][k] ? parity : 0;
        a.staging[k] = ctx->x_staging[set][k];
        a.capacity[k] = ctx->x_capacity[set][k];
    }
    a.stats = nullptr;
    a.status = ctx->status_dev;
    return WASH_OK;
}

int exchange_ready(const wash_ctx *ctx, const wash::ExchangeArgs &a)
{
    if (!ctx->x_planned) return fail(WASH_ERR_STATE, "no step has been planned (wash_exchange_plan)");
    if (!a.row[0] && !a.row[1]) return fail(WASH_ERR_STATE, "no model row is bound");
    for (int k = 0; k < 2; ++k)
        if (a.row[k] && !a.staging[k]) return fail(WASH_ERR_STATE, "stack %d has no staging buffers (wash_exchange_staging)", k);
    return WASH_OK;
}

}  // namespace

extern "C" {

int wash_exchange_bind(wash_ctx *ctx, int32_t self, int32_t stack, int32_t dtype, void *dev_row, int64_t n_elems)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (self < 0 || self >= ctx->N) return fail(WASH_ERR_ARG, "self = %d, must be in [0, %d)", self, ctx->N);
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (ctx->padded_P >= (int64_t(1) << 32)) return fail(WASH_ERR_UNSUPPORTED, "rows of 2^32 elements and more cannot be exchanged");
    if (ctx->x_self >= 0 && ctx->x_self != self) return fail(WASH_ERR_STATE, "context already is worker %d", ctx->x_self);
    if (dev_row) {
        if (dtype != WASH_F32 && dtype != WASH_BF16) return fail(WASH_ERR_ARG, "unknown dtype %d", dtype);
        if (n_elems != ctx->padded_P) return fail(WASH_ERR_ARG, "row has %lld elements, a model needs padded_P = %lld", (long long)n_elems, (long long)ctx->padded_P);
        if (reinterpret_cast<uintptr_t>(dev_row) & 15) return fail(WASH_ERR_ARG, "row pointer must be 16-byte aligned");
    }
    if (!ctx->x_mask) {
        DeviceGuard guard(ctx->device);
        if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
        // the grid: kExchangeBlocksPerSm blocks per SM, fewer for short rows; its
        // warps share the warp tiles evenly
        const uint32_t wtiles = (ctx->n_groups + wash::kExchangeTileGroups - 1) / wash::kExchangeTileGroups;
        const uint32_t max_blocks = static_cast<uint32_t>(ctx->shape.sm_count > 0 ? ctx->shape.sm_count : 148) * static_cast<uint32_t>(wash::kExchangeBlocksPerSm);
        const uint32_t want = (wtiles + wash::kExchangeWarps - 1) / wash::kExchangeWarps;
        const uint32_t blocks = want < max_blocks ? want : max_blocks;
        const size_t columns = static_cast<size_t>(ctx->N) + 1;
        cudaError_t err;
        if ((err = cudaMalloc(&ctx->x_mask, sizeof(uint32_t) * 32u * static_cast<size_t>(wtiles))) != cudaSuccess ||
            (err = cudaMalloc(&ctx->x_warp_total, sizeof(uint32_t) * columns * blocks * wash::kExchangeWarps)) != cudaSuccess ||
            (err = cudaMalloc(&ctx->x_block_total, sizeof(uint32_t) * columns * blocks)) != cudaSuccess) {
            cudaGetLastError();
            if (ctx->x_mask) cudaFree(ctx->x_mask);
            if (ctx->x_warp_total) cudaFree(ctx->x_warp_total);
            ctx->x_mask = nullptr;
            ctx->x_warp_total = nullptr;
            return fail(WASH_ERR_ALLOC, "device allocation of the exchange tables failed: %s", cudaGetErrorString(err));
        }
        ctx->x_wtiles = wtiles;
        ctx->x_blocks = blocks;
    }
    ctx->x_self = self;
    ctx->x_row[stack] = dev_row;
    ctx->x_dtype[stack] = dtype;
    return WASH_OK;
}

int wash_exchange_staging(wash_ctx *ctx, int32_t stack, int32_t parity, void *const *buffers, int64_t capacity_elems)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (parity != 0 && parity != 1) return fail(WASH_ERR_ARG, "parity must be 0 or 1");
    if (!buffers) return fail(WASH_ERR_ARG, "buffers is NULL");
    if (capacity_elems < 0) return fail(WASH_ERR_ARG, "capacity_elems = %lld", (long long)capacity_elems);
    for (int n = 0; n < ctx->N; ++n)
        if (!buffers[n] || (reinterpret_cast<uintptr_t>(buffers[n]) & 3)) return fail(WASH_ERR_ARG, "buffers[%d] must be a 4-byte aligned device-accessible pointer", n);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaError_t err;
    if (!ctx->x_staging[parity][stack] &&
        (err = cudaMalloc(reinterpret_cast<void **>(&ctx->x_staging[parity][stack]), sizeof(void *) * static_cast<size_t>(ctx->N))) != cudaSuccess) {
        cudaGetLastError();
        return fail(WASH_ERR_ALLOC, "device allocation of the pointer table failed: %s", cudaGetErrorString(err));
    }
    // synchronous: earlier steps that read the table are complete when it is replaced
    if ((err = cudaDeviceSynchronize()) != cudaSuccess) return cuda_fail(err, "cudaDeviceSynchronize");
    if ((err = cudaMemcpy(ctx->x_staging[parity][stack], buffers, sizeof(void *) * static_cast<size_t>(ctx->N), cudaMemcpyHostToDevice)) != cudaSuccess)
        return cuda_fail(err, "upload of the staging pointers");
    ctx->x_capacity[parity][stack] = capacity_elems;
    return WASH_OK;
}

int wash_exchange_staging_create(wash_ctx *ctx, int32_t stack, int32_t parity, int64_t capacity_elems, void *handle_out)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (parity != 0 && parity != 1) return fail(WASH_ERR_ARG, "parity must be 0 or 1");
    if (capacity_elems < 1) return fail(WASH_ERR_ARG, "capacity_elems = %lld", (long long)capacity_elems);
    if (!handle_out) return fail(WASH_ERR_ARG, "handle_out is NULL");
    if (ctx->x_self < 0 || !ctx->x_row[stack]) return fail(WASH_ERR_STATE, "bind the row of stack %d first (wash_exchange_bind)", stack);
    if (ctx->x_own[parity][stack]) return fail(WASH_ERR_STATE, "staging set %d of stack %d already exists", parity, stack);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    void *buf = nullptr;
    cudaError_t err = cudaMalloc(&buf, static_cast<size_t>(capacity_elems) * elem_bytes(ctx->x_dtype[stack]));
    if (err != cudaSuccess) {
        cudaGetLastError();
        return fail(WASH_ERR_ALLOC, "device allocation of the staging buffer failed: %s", cudaGetErrorString(err));
    }
    cudaIpcMemHandle_t handle;
    if ((err = cudaIpcGetMemHandle(&handle, buf)) != cudaSuccess) {
        cudaFree(buf);
        return cuda_fail(err, "cudaIpcGetMemHandle");
    }
    static_assert(sizeof handle == WASH_IPC_HANDLE_BYTES, "handle size");
    std::memcpy(handle_out, &handle, sizeof handle);
    ctx->x_own[parity][stack] = buf;
    ctx->x_capacity[parity][stack] = capacity_elems;
    return WASH_OK;
}

int wash_exchange_staging_open(wash_ctx *ctx, int32_t stack, int32_t parity, const void *handles)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (stack != WASH_STACK_PARAMS && stack != WASH_STACK_OPT) return fail(WASH_ERR_ARG, "stack must be 0 or 1");
    if (parity != 0 && parity != 1) return fail(WASH_ERR_ARG, "parity must be 0 or 1");
    if (!handles) return fail(WASH_ERR_ARG, "handles is NULL");
    if (!ctx->x_own[parity][stack]) return fail(WASH_ERR_STATE, "create this worker's buffer first (wash_exchange_staging_create)");
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    if (ctx->x_opened_set[parity][stack]) return fail(WASH_ERR_STATE, "the peers' buffers of staging set %d of stack %d are already open", parity, stack);
    std::vector<void *> buffers(static_cast<size_t>(ctx->N), nullptr);
    std::vector<void *> mapped;   // what this call opened: closed again if it fails part-way
    auto roll_back = [&]() {
        for (void *peer : mapped) cudaIpcCloseMemHandle(peer);
        cudaGetLastError();
    };
    for (int n = 0; n < ctx->N; ++n) {
        if (n == ctx->x_self) { buffers[n] = ctx->x_own[parity][stack]; continue; }
        cudaIpcMemHandle_t handle;
        std::memcpy(&handle, static_cast<const char *>(handles) + static_cast<size_t>(n) * WASH_IPC_HANDLE_BYTES, sizeof handle);
        cudaError_t err = cudaIpcOpenMemHandle(&buffers[n], handle, cudaIpcMemLazyEnablePeerAccess);
        if (err != cudaSuccess) {
            roll_back();
            return cuda_fail(err, "cudaIpcOpenMemHandle (is worker's buffer in another process on a device this one can reach?)");
        }
        mapped.push_back(buffers[n]);
    }
    const int rc = wash_exchange_staging(ctx, stack, parity, buffers.data(), ctx->x_capacity[parity][stack]);
    if (rc != WASH_OK) {
        const std::string first = g_last_error;
        roll_back();
        g_last_error = first;
        return rc;
    }
    ctx->x_opened.insert(ctx->x_opened.end(), mapped.begin(), mapped.end());
    ctx->x_opened_set[parity][stack] = true;
    return WASH_OK;
}

int wash_exchange_plan(wash_ctx *ctx, uint64_t step, double p, const double *p_layer, uint64_t seed, void *stream_v)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (ctx->x_self < 0) return fail(WASH_ERR_STATE, "wash_exchange_bind has not been called");
    if (step >> 56) return fail(WASH_ERR_ARG, "step must be below 2^56");
    if (!p_layer && !(p >= 0.0 && p <= 1.0)) return fail(WASH_ERR_ARG, "p is %g, not in [0,1]", p);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int rc = sync_table(ctx, p, p_layer, stream);
    if (rc != WASH_OK) return rc;
    ctx->x_step = step;
    ctx->x_seed = seed;
    wash::ExchangeArgs args;
    if ((rc = exchange_args(ctx, &args)) != WASH_OK) return rc;
    cudaError_t err = wash::launch_exchange_plan(args, stream);
    if (err != cudaSuccess) return cuda_fail(err, "exchange plan launch");
    ctx->x_planned = true;
    return WASH_OK;
}

int wash_exchange_send(wash_ctx *ctx, void *stream_v)
{
    wash::ExchangeArgs args;
    int rc = exchange_args(ctx, &args);
    if (rc != WASH_OK || (rc = exchange_ready(ctx, args)) != WASH_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaError_t err = wash::launch_exchange_send(args, static_cast<cudaStream_t>(stream_v));
    if (err != cudaSuccess) return cuda_fail(err, "exchange send launch");
    return WASH_OK;
}

int wash_exchange_receive(wash_ctx *ctx, void *stream_v, wash_stats *stats)
{
    wash::ExchangeArgs args;
    int rc = exchange_args(ctx, &args);
    if (rc != WASH_OK || (rc = exchange_ready(ctx, args)) != WASH_OK) return rc;
    args.stats = reinterpret_cast<unsigned long long *>(stats);
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaError_t err = wash::launch_exchange_receive(args, static_cast<cudaStream_t>(stream_v));
    if (err != cudaSuccess) return cuda_fail(err, "exchange receive launch");
    return WASH_OK;
}

int wash_exchange_counts(wash_ctx *ctx, uint64_t *host_need, uint64_t *host_selected, void *stream_v)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    if (!ctx->x_planned) return fail(WASH_ERR_STATE, "no step has been planned (wash_exchange_plan)");
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t columns = static_cast<size_t>(ctx->N) + 1;
    std::vector<uint32_t> per_block(columns * ctx->x_blocks);
    cudaError_t err = cudaMemcpyAsync(per_block.data(), ctx->x_block_total, sizeof(uint32_t) * per_block.size(), cudaMemcpyDeviceToHost, stream);
    if (err == cudaSuccess) err = cudaStreamSynchronize(stream);
    if (err != cudaSuccess) return cuda_fail(err, "reading the plan's totals");
    std::vector<uint64_t> total(columns, 0);
    for (size_t b = 0; b < ctx->x_blocks; ++b)
        for (size_t col = 0; col < columns; ++col) total[col] += per_block[b * columns + col];
    if (host_need)
        for (int n = 0; n < ctx->N; ++n) host_need[n] = total[static_cast<size_t>(n)];
    if (host_selected) *host_selected = total[static_cast<size_t>(ctx->N)];
    return WASH_OK;
}

int wash_check(wash_ctx *ctx, void *stream_v)
{
    if (!ctx) return fail(WASH_ERR_ARG, "ctx is NULL");
    DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    uint32_t status = 0;
    cudaError_t err = cudaMemcpyAsync(&status, ctx->status_dev, sizeof status, cudaMemcpyDeviceToHost, stream);
    if (err == cudaSuccess) err = cudaStreamSynchronize(stream);
    if (err != cudaSuccess) return cuda_fail(err, "reading the status word");
    if (status) {
        cudaMemsetAsync(ctx->status_dev, 0, sizeof(uint32_t), stream);
        return fail(WASH_ERR_DEVICE_CHECK, "device status 0x%x:%s%s", status,
                    (status & 1u) ? " a group outside its segment table;" : "",
                    (status & 4u) ? " an exchange step needed more slots than the staging buffers hold;" : "");
    }
    return WASH_OK;
}

int wash_philox_probe(uint64_t n_blocks, uint64_t seed, uint32_t *dev_checksum, int32_t device, void *stream_v)
{
    if (device < 0) return fail(WASH_ERR_ARG, "device = %d", device);
    DeviceGuard guard(device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err, "cudaSetDevice");
    cudaError_t err = wash::launch_philox_probe(n_blocks, seed, dev_checksum, static_cast<cudaStream_t>(stream_v));
    if (err != cudaSuccess) return cuda_fail(err, "philox probe launch");
    return WASH_OK;
}

const char *wash_last_error(void) { return g_last_error.c_str(); }

uint64_t wash_launch_count(void) { return wash::launch_count(); }

}  // extern "C"
