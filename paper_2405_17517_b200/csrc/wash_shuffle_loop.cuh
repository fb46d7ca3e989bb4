// Streaming shuffle for populations whose group of all models is small (N * 16 bytes in fp32):
// a resident grid of one-warp blocks, each walking tiles of 32 * G groups with two shared-memory
// stages.
//
// With one group per thread and one trip per thread (wash_shuffle_async.cuh) a thread spends a
// few hundred instructions around its single group -- block start, table lookup, the copies'
// addresses, the statistics' block reduction -- which is nothing beside 320 bytes of a ten-model
// group but fills the issue slots at 40 % of the memory bandwidth when the group has 32 bytes.
// Here a warp stays: the copies of its next tile are started, the mask of the current tile is
// drawn while they travel, the current tile (whose copies were started one trip earlier) is
// served, and the table entry, the counters and the launch constants live in registers across
// trips.  Tiles are dealt round-robin over the blocks, so the blocks resident at one moment read
// neighbouring addresses.
//
// The image of a stage is the one-trip kernel's block image with T = 32 (the block is one warp,
// so every helper of that kernel -- copies, serving, padding rule -- is used as it is).
#pragma once
#define WASH_SERVING_ONLY
#include "wash_shuffle_async.cuh"

namespace wash {

__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int K>
__device__ __forceinline__ void cp_async_wait_all_but_latest()   // all groups of copies but the K latest
{
    asm volatile("cp.async.wait_group %0;" ::"n"(K) : "memory");
}

// The table entry of the lane's previous group; a group of the same segment needs no lookup.
struct SegCache {
    uint32_t begin, end;   // groups [begin, end) of the row
    uint32_t tensor_id, cgroup_begin, numel, seg;
    uint32_t thr_lo;       // the threshold's low word
    uint32_t thr_hi;       // 1: the threshold is 2^32 (every coordinate selected)
    uint32_t plain;        // groups of the segment that hold four coordinates, 0 unless 0 < threshold < 2^32
};

__device__ __forceinline__ GroupInfo find_group_cached(const PopView &pop, SegCache &sc, uint32_t g, uint32_t *status)
{
    if (g - sc.begin >= sc.end - sc.begin) {
        uint32_t s = __ldg(pop.tile_first + (g >> kTileShift));
        const uint32_t last = static_cast<uint32_t>(pop.n_seg) - 1u;
        while (s < last && g >= __ldg(&pop.seg[s].group_end)) ++s;
        const uint4 lo = __ldg(reinterpret_cast<const uint4 *>(pop.seg + s));
        const uint4 hi = __ldg(reinterpret_cast<const uint4 *>(pop.seg + s) + 1);
        if (g < lo.x || g >= lo.y) {   // table inconsistent with the row: report, touch nothing
            if (status) atomicOr(status, 1u);
            return GroupInfo{0, 0, 0, 0, s};
        }
        const bool drawn = hi.w == 0 && hi.z != 0;   // 0 < threshold < 2^32: the mask words decide
        sc = SegCache{lo.x, lo.y, lo.z, lo.w, hi.x, s, hi.z, hi.w, drawn ? min(hi.x >> 2, lo.y - lo.x) : 0u};
    }
    const uint32_t local = g - sc.begin;
    GroupInfo gi;
    gi.seg = sc.seg;
    gi.tensor_id = sc.tensor_id;
    gi.cgroup = sc.cgroup_begin + local;
    gi.thr = static_cast<uint64_t>(sc.thr_lo) | (static_cast<uint64_t>(sc.thr_hi) << 32);
    // coordinates of the tensor from this group on; the segment may end in a group of padding only
    const long long left = static_cast<long long>(sc.numel) - 4ll * local;
    gi.valid = left >= 4 ? 4 : (left > 0 ? static_cast<int>(left) : 0);
    return gi;
}

// Starts the copies of the full tile of 32 * G groups that begins at group g_first into a stage.
// fp32 only: [N][P]: lane l copies the vector of every model for its G groups; [P][N] without
// padding: the tile's bytes are contiguous and are copied as they lie, 512 bytes per warp and copy.
template <int LAYOUT, int G>
__device__ __forceinline__ void fetch_full_tile_f32(uint32_t image, uint32_t image_stride, const void *base, const PopView &pop,
                                                    uint32_t g_first, int n_models)
{
    const uint32_t lane = threadIdx.x;
    if (LAYOUT == kLayoutNP) {
        const size_t row_bytes = static_cast<size_t>(pop.padded_P) * 4;
        const char *src0 = static_cast<const char *>(base) + (static_cast<size_t>(g_first) + lane) * 16;
        uint32_t dst0 = image + lane * 16;
#pragma unroll
        for (int i = 0; i < G; ++i, src0 += 512, dst0 += image_stride) {
            const char *src = src0;
            uint32_t dst = dst0;
            for (int j = 0; j < n_models; ++j, src += row_bytes, dst += 512) cp_async<16>(dst, src);
        }
    } else {
        const char *src = static_cast<const char *>(base) + (static_cast<size_t>(g_first) * n_models + lane) * 16;
        uint32_t dst0 = image + lane * 16;
#pragma unroll
        for (int i = 0; i < G; ++i, dst0 += image_stride) {
            uint32_t dst = dst0;
            for (int j = 0; j < n_models; ++j, src += 512, dst += 512) cp_async<16>(dst, src);
        }
    }
}

template <class TA, class TB, int LAYOUT, int G, int S>
__global__ void __launch_bounds__(32, 32) shuffle_loop_kernel(const __grid_constant__ ShuffleArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    constexpr uint32_t T_ = 32;   // the launch has one warp per block
    const int n_models = a.pop.N;
    const size_t group_elems = LAYOUT == kLayoutPN ? pn_group_elems(n_models, a.pn_pad) : 4u * static_cast<size_t>(n_models);
    const uint32_t a_bytes = static_cast<uint32_t>(group_elems * T_ * TA::kBytes);
    const uint32_t b_bytes = kHasB ? static_cast<uint32_t>(group_elems * T_ * TB::kBytes) : 0u;
    const uint32_t stage_bytes = G * (a_bytes + b_bytes);
    uint8_t *s_list = smem_raw + S * stage_bytes;   // 128 bytes: the warp's list of selected coordinates
    uint8_t *s_perm = s_list + 128 + threadIdx.x;   // a column [n][T] of bytes, used when N > 16

    // group indices fit 32 bits (the table holds them so); a tile index therefore too
    const uint32_t n_tiles = static_cast<uint32_t>((a.group_hi - a.group_lo + T_ * G - 1) / (T_ * G));
    const uint32_t full_tiles = static_cast<uint32_t>((a.group_hi - a.group_lo) / (T_ * G));   // the tiles before the ragged one
    const uint32_t group_lo = static_cast<uint32_t>(a.group_lo);
    const uint32_t image0 = smem_addr(smem_raw);
    // starts the copies of a tile into a stage (nothing beyond the last tile) and closes their group
    auto fetch = [&](uint32_t tile, uint32_t stage) {
        const uint32_t g_first = group_lo + tile * (T_ * G);
        constexpr bool kFastA = TA::kBytes == 4, kFastB = !kHasB || TB::kBytes == 4;
        const bool linear = LAYOUT == kLayoutNP || a.pn_pad == 0;
        if (tile < full_tiles && linear && (kFastA || kFastB)) {
            const uint32_t image_a = image0 + stage * stage_bytes;
            if constexpr (kFastA) fetch_full_tile_f32<LAYOUT, G>(image_a, a_bytes + b_bytes, a.a, a.pop, g_first, n_models);
            if constexpr (kHasB && TB::kBytes == 4) fetch_full_tile_f32<LAYOUT, G>(image_a + a_bytes, a_bytes + b_bytes, a.b, a.pop, g_first, n_models);
        }
        if (tile < n_tiles && !(tile < full_tiles && linear && kFastA && kFastB)) {
#pragma unroll
            for (int i = 0; i < G; ++i) {
                const uint64_t g_block = static_cast<uint64_t>(g_first) + static_cast<uint64_t>(i) * T_;
                if (g_block >= a.group_hi) break;
                const uint32_t in_tile = static_cast<uint32_t>(min(static_cast<uint64_t>(T_), a.group_hi - g_block));
                const uint32_t image_a = image0 + stage * stage_bytes + i * (a_bytes + b_bytes);
                if (!(tile < full_tiles && linear && kFastA)) async_fetch<TA, LAYOUT>(image_a, a.a, a.pop, g_block, in_tile, n_models, a.pn_pad);
                if constexpr (kHasB)
                    if (!(tile < full_tiles && linear && TB::kBytes == 4)) async_fetch<TB, LAYOUT>(image_a + a_bytes, a.b, a.pop, g_block, in_tile, n_models, a.pn_pad);
            }
        }
        cp_async_commit();
    };

    uint32_t selected = 0, moved = 0, stage = 0;
    SegCache sc{0, 0, 0, 0, 0, 0, 0, 0, 0};
    uint32_t tile = blockIdx.x;
    // S - 1 tiles in flight ahead of the one that is served; beyond the last tile (also when the
    // index wraps) a fetch copies nothing
    uint32_t ahead = tile, ahead_stage = 0;
#pragma unroll
    for (int k = 0; k < S - 1; ++k) {
        fetch(ahead, ahead_stage);
        ahead = ahead + gridDim.x >= ahead ? ahead + gridDim.x : n_tiles;
        ahead_stage = ahead_stage + 1 == S ? 0 : ahead_stage + 1;
    }
    for (; tile < n_tiles; tile += gridDim.x, stage = stage + 1 == S ? 0 : stage + 1) {
        fetch(ahead, ahead_stage);
        ahead = ahead + gridDim.x >= ahead ? ahead + gridDim.x : n_tiles;
        ahead_stage = ahead_stage + 1 == S ? 0 : ahead_stage + 1;
        const uint32_t g_first = group_lo + tile * (T_ * G);
        uint32_t sel[G];
        GroupInfo gi[G];
        // the usual tile: full, every lane's G groups whole and in the segment of its previous
        // group, thresholds that the mask words decide -- then nothing is looked up or predicated
        const uint32_t local = g_first + threadIdx.x - sc.begin;
        const bool plain = tile < full_tiles && __all_sync(0xFFFFFFFFu, local < sc.plain && local + (G - 1) * T_ < sc.plain);
        if (plain) {
#pragma unroll
            for (int i = 0; i < G; ++i) {
                gi[i].seg = sc.seg;
                gi[i].tensor_id = sc.tensor_id;
                gi[i].cgroup = sc.cgroup_begin + local + i * T_;
                gi[i].valid = 4;
                gi[i].thr = sc.thr_lo;
                const Philox4 w = philox4x32_10(gi[i].cgroup, sc.tensor_id, a.step_lo, a.step_hi8, a.keys);
                sel[i] = (w.x < sc.thr_lo ? 1u : 0u) | (w.y < sc.thr_lo ? 2u : 0u) | (w.z < sc.thr_lo ? 4u : 0u) | (w.w < sc.thr_lo ? 8u : 0u);
            }
        } else {
#pragma unroll
            for (int i = 0; i < G; ++i) {
                sel[i] = 0;
                gi[i] = GroupInfo{0, 0, 0, 0, 0};
                const uint64_t g = static_cast<uint64_t>(g_first) + static_cast<uint64_t>(i) * T_ + threadIdx.x;
                if (g < a.group_hi) {
                    gi[i] = find_group_cached(a.pop, sc, static_cast<uint32_t>(g), a.status);
                    if (gi[i].thr != 0 && gi[i].valid != 0) {
                        uint32_t m = 0xFu;   // a threshold of 2^32 selects whatever the word is
                        if ((gi[i].thr >> 32) == 0) {
                            const Philox4 w = philox4x32_10(gi[i].cgroup, gi[i].tensor_id, a.step_lo, a.step_hi8, a.keys);
                            const uint32_t thr_lo = static_cast<uint32_t>(gi[i].thr);
                            m = (w.x < thr_lo ? 1u : 0u) | (w.y < thr_lo ? 2u : 0u) | (w.z < thr_lo ? 4u : 0u) | (w.w < thr_lo ? 8u : 0u);
                        }
                        sel[i] = m & ((1u << gi[i].valid) - 1u);
                    }
                }
            }
        }
        uint32_t any = 0;
#pragma unroll
        for (int i = 0; i < G; ++i) any |= sel[i];
        cp_async_wait_all_but_latest<S - 1>();   // this tile's copies; the next tiles' stay in flight
        __syncwarp();
        if (__any_sync(0xFFFFFFFFu, any != 0)) {
#pragma unroll
            for (int i = 0; i < G; ++i) {
                const unsigned char *image_a = smem_raw + stage * stage_bytes + i * (a_bytes + b_bytes);
                serve_tile<TA, TB, LAYOUT>(a, image_a, image_a + a_bytes, s_list, s_perm,
                                           static_cast<uint64_t>(g_first) + static_cast<uint64_t>(i) * T_, sel[i], gi[i], selected, moved);
            }
            __syncwarp();   // the stage is overwritten by the copies the next trip starts
        }
    }
    cp_async_wait_all();
    publish_block_stats(a.stats, a.stat_slots, selected, moved);
}

template <class TA, class TB, int G, int S>
cudaError_t launch_shuffle_loop_tiles(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const size_t group_elems = 4 * static_cast<size_t>(args.pop.N) + (args.pop.layout == kLayoutPN ? args.pn_pad : 0);
    const size_t image = group_elems * (TA::kBytes + (kHasB ? TB::kBytes : 0)) * 32;
    const size_t smem = (S * G * image + 128 + (args.pop.N > 16 ? 32 * static_cast<size_t>(args.pop.N) : 0) + 15) & ~static_cast<size_t>(15);
    const bool np = args.pop.layout == kLayoutNP;
    auto kernel = np ? shuffle_loop_kernel<TA, TB, kLayoutNP, G, S> : shuffle_loop_kernel<TA, TB, kLayoutPN, G, S>;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), 32, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    const uint64_t per_tile = 32ull * G;
    const uint64_t n_tiles = (static_cast<uint64_t>(args.group_hi - args.group_lo) + per_tile - 1) / per_tile;
    if (n_tiles == 0) return cudaSuccess;
    const uint64_t resident = static_cast<uint64_t>(shape.sm_count > 0 ? shape.sm_count : 148) * fit.occupancy;
    const uint64_t grid = n_tiles < resident ? n_tiles : resident;
    kernel<<<static_cast<unsigned>(grid), 32, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

template <class TA, class TB>
cudaError_t launch_shuffle_loop_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    // Two groups per lane and tile, two stages.  Measured on 2^27 coordinates (N = 2, fp32, p = 1e-4 .. 0.1):
    // one group per lane leaves too few bytes in flight (0.215 against 0.174 ms at p = 1e-4), four make a
    // trip that serves anything long and cost resident warps (0.294 against 0.217 ms at p = 1e-3), a third
    // stage changes nothing (0.226 against 0.219 ms).
    return launch_shuffle_loop_tiles<TA, TB, 2, 2>(args, shape, stream);
}

inline cudaError_t launch_shuffle_loop(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                       cudaStream_t stream, bool *supported)
{
    *supported = true;
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeNone) return launch_shuffle_loop_typed<F32, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeNone) return launch_shuffle_loop_typed<BF16, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeF32) return launch_shuffle_loop_typed<F32, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeF32) return launch_shuffle_loop_typed<BF16, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeBF16) return launch_shuffle_loop_typed<BF16, BF16>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeBF16) return launch_shuffle_loop_typed<F32, BF16>(args, shape, stream);
    *supported = false;
    return cudaSuccess;
}

}  // namespace wash
