// wash_shuffle_noalloc: the shuffling step for callers that must not allocate.
//
// Every other entry point works through a wash_ctx whose lookup tables were placed
// in device memory by cudaMalloc at wash_create time.  Some callers cannot do that:
// a training process whose framework has already claimed all of the GPU's memory for
// its own pool (a cudaMalloc from a library would fail, or would have to be carved out
// of the pool by hand), and loops in which the implicit device-wide synchronisation of
// cudaMalloc / cudaFree would stall kernels that other streams have in flight (each call
// here still makes two small pageable host-to-device copies, ordered on its stream).  For them the same kernel is launched with its tables in a fixed array
// that is part of the library image: it exists on every GPU that loads libwash.so, from
// load to exit, and costs kScratchBytes there whether or not this entry point is used.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/wash.h"
#include "wash_internal.h"

using wash::SegEntry;

namespace {

constexpr int kMaxTensors = WASH_NOALLOC_MAX_TENSORS;
constexpr long long kMaxRowElems = WASH_NOALLOC_MAX_ROW_ELEMS;
constexpr size_t kMaxTiles = static_cast<size_t>(kMaxRowElems / 4) >> wash::kTileShift;
constexpr size_t kSegBytes = sizeof(SegEntry) * kMaxTensors;          // 32 KiB
constexpr size_t kTileBytes = sizeof(uint32_t) * kMaxTiles;           // 256 KiB
constexpr size_t kSlotBytes = sizeof(wash::StatSlot) * wash::kStatSlots;   // 8 KiB
constexpr size_t kScratchBytes = kSegBytes + kTileBytes + kSlotBytes;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// lookup -- it is NOT a device address and must never be passed to a kernel; the device
// address is obtained per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char *g_scratch_addr[kMaxDevices] = {};   // device address of the array, per device
int g_sm_count[kMaxDevices] = {};

thread_local char g_msg[256];

int fail(int code, const char *msg)
{
    snprintf(g_msg, sizeof g_msg, "%s", msg);
    return code;
}

}  // namespace

// wash_last_error() reports errors of the context-based calls; this entry point keeps
// its own message so that it does not touch their state.
extern "C" const char *wash_noalloc_last_error(void) { return g_msg; }

extern "C" int wash_shuffle_noalloc(int32_t N, int32_t n_tensors, const int64_t *numel, int32_t layout,
                                    int32_t dtype, void *dev_stack, int64_t n_elems, uint64_t step, double p,
                                    const double *p_layer, uint64_t seed, int32_t device, void *stream_v,
                                    wash_stats *stats)
{
    g_msg[0] = 0;
    if (N < 2 || N > WASH_MAX_N) return fail(WASH_ERR_ARG, "N must be in [2, WASH_MAX_N]");
    if (n_tensors < 1 || !numel) return fail(WASH_ERR_ARG, "need at least one tensor");
    if (n_tensors > kMaxTensors) return fail(WASH_ERR_ARG, "too many tensors for the built-in scratch (limit WASH_NOALLOC_MAX_TENSORS = 1024); use wash_create + wash_shuffle");
    if (layout != WASH_LAYOUT_NP && layout != WASH_LAYOUT_PN) return fail(WASH_ERR_ARG, "unknown layout");
    if (dtype != WASH_F32 && dtype != WASH_BF16) return fail(WASH_ERR_ARG, "unknown dtype");
    if (!dev_stack || (reinterpret_cast<uintptr_t>(dev_stack) & 15)) return fail(WASH_ERR_ARG, "dev_stack must be a 16-byte aligned device pointer");
    if (step >> 56) return fail(WASH_ERR_ARG, "step must be below 2^56");
    if (device < 0 || device >= kMaxDevices) return fail(WASH_ERR_ARG, "device ordinal out of range");
    if (!p_layer && !(p >= 0.0 && p <= 1.0)) return fail(WASH_ERR_ARG, "p must be in [0,1]");

    // row geometry, the same rule as wash_create: tensors start on multiples of 8 elements
    std::vector<SegEntry> seg(static_cast<size_t>(n_tensors));
    long long cur = 0;
    for (int t = 0; t < n_tensors; ++t) {
        const long long d = numel[t];
        if (d <= 0 || d >= (1ll << 32)) return fail(WASH_ERR_ARG, "numel[t] must be in (0, 2^32)");
        const double pt = p_layer ? p_layer[t] : p;
        if (!(pt >= 0.0 && pt <= 1.0)) return fail(WASH_ERR_ARG, "p_layer[t] must be in [0,1]");
        SegEntry &e = seg[static_cast<size_t>(t)];
        e.group_begin = static_cast<uint32_t>(cur / 4);
        cur += (d + WASH_ALIGN_ELEMS - 1) / WASH_ALIGN_ELEMS * WASH_ALIGN_ELEMS;
        if (cur > kMaxRowElems) return fail(WASH_ERR_ARG, "row too long for the built-in scratch (limit WASH_NOALLOC_MAX_ROW_ELEMS = 2^26 padded elements per model); use wash_create + wash_shuffle");
        e.group_end = static_cast<uint32_t>(cur / 4);
        e.tensor_id = static_cast<uint32_t>(t);
        e.cgroup_begin = 0;
        e.numel = static_cast<uint32_t>(d);
        e.reserved = 0;
        e.thr = static_cast<uint64_t>(std::floor(pt * 4294967296.0));
    }
    const long long padded_P = cur;
    if (n_elems != static_cast<int64_t>(N) * padded_P) return fail(WASH_ERR_ARG, "n_elems must equal N * padded_P");
    const uint32_t n_groups = static_cast<uint32_t>(padded_P / 4);
    const uint32_t n_tiles = (n_groups + (1u << wash::kTileShift) - 1) >> wash::kTileShift;
    std::vector<uint32_t> tile_first(n_tiles);
    for (uint32_t tile = 0, s = 0; tile < n_tiles; ++tile) {
        const uint32_t g = tile << wash::kTileShift;
        while (g >= seg[s].group_end) ++s;
        tile_first[tile] = s;
    }

    int prev = -1;
    cudaError_t err = cudaGetDevice(&prev);
    if (err != cudaSuccess) return fail(WASH_ERR_CUDA, cudaGetErrorString(err));
    if (prev != device && (err = cudaSetDevice(device)) != cudaSuccess) return fail(WASH_ERR_CUDA, cudaGetErrorString(err));
    int rc = WASH_OK;
    unsigned char *scratch = nullptr;
    int sm_count = 0;
    {
        // set-up, once per device, with that device current: ask the runtime where this
        // device's copy of the array lives
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[device]) {
            void *addr = nullptr;
            err = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
            if (err == cudaSuccess) err = cudaDeviceGetAttribute(&g_sm_count[device], cudaDevAttrMultiProcessorCount, device);
            if (err != cudaSuccess || !addr) rc = fail(WASH_ERR_CUDA, err != cudaSuccess ? cudaGetErrorString(err) : "cudaGetSymbolAddress returned NULL");
            else g_scratch_addr[device] = static_cast<unsigned char *>(addr);
        }
        scratch = g_scratch_addr[device];
        sm_count = g_sm_count[device];
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    if (rc == WASH_OK) {
        // the table uploads below read host arrays that die with this call: a captured copy
        // would read freed memory at replay
        cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
        err = cudaStreamIsCapturing(stream, &capture);
        if (err != cudaSuccess) rc = fail(WASH_ERR_CUDA, cudaGetErrorString(err));
        else if (capture != cudaStreamCaptureStatusNone) rc = fail(WASH_ERR_STATE, "the stream is in capture mode: wash_shuffle_noalloc copies its tables from host arrays that do not outlive the call");
    }
    if (rc == WASH_OK) {
        SegEntry *seg_dev = reinterpret_cast<SegEntry *>(scratch);
        uint32_t *tile_dev = reinterpret_cast<uint32_t *>(scratch + kSegBytes);
        // Both tables are rewritten in full and the counters' partial sums are zeroed, in
        // stream order, before the kernel runs; nothing is carried over from the previous call.
        err = cudaMemcpyAsync(seg_dev, seg.data(), sizeof(SegEntry) * seg.size(), cudaMemcpyHostToDevice, stream);
        if (err == cudaSuccess) err = cudaMemcpyAsync(tile_dev, tile_first.data(), sizeof(uint32_t) * n_tiles, cudaMemcpyHostToDevice, stream);
        // the partial sums of the statistics must start at zero
        wash::StatSlot *slots_dev = reinterpret_cast<wash::StatSlot *>(scratch + kSegBytes + kTileBytes);
        if (err == cudaSuccess && stats) err = cudaMemsetAsync(slots_dev, 0, kSlotBytes, stream);
        if (err != cudaSuccess) rc = fail(WASH_ERR_CUDA, cudaGetErrorString(err));
        if (rc == WASH_OK) {
            wash::ShuffleArgs args;
            args.pop.N = N;
            args.pop.layout = layout;
            args.pop.padded_P = padded_P;
            args.pop.n_groups = n_groups;
            args.pop.n_seg = n_tensors;
            args.pop.seg = seg_dev;
            args.pop.tile_first = tile_dev;
            args.a = dev_stack;
            args.b = nullptr;
            args.group_lo = 0;
            args.group_hi = n_groups;
            args.keys = wash::philox_keys(seed);
            args.step_lo = static_cast<uint32_t>(step);
            args.step_hi8 = static_cast<uint32_t>(step >> 32) << 8;
            args.stats = reinterpret_cast<unsigned long long *>(stats);
            args.stat_slots = slots_dev;
            args.status = nullptr;
            const wash::LaunchShape shape{0, 0, sm_count};
            bool supported = false;
            err = wash::launch_shuffle(args, dtype, wash::kDtypeNone, wash::kModeStream, shape, stream, &supported);
            if (err != cudaSuccess) rc = fail(WASH_ERR_CUDA, cudaGetErrorString(err));
            else if (!supported) rc = fail(WASH_ERR_UNSUPPORTED, "no kernel for this dtype");
        }
    }
    if (prev != device) cudaSetDevice(prev);
    return rc;
}
