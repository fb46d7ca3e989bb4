// Sparse shuffle (WASH_MODE_SPARSE): the mask is drawn first, without touching the stacks, and
// only the selected coordinates are loaded, permuted and stored -- the paper's point that a
// step moves p d values, not d, carried onto one GPU.  The kernel is bound by the integer
// pipes (one Philox block per 4 coordinates), not by memory.
//
// Work is cut into warp tiles (wash_warp_tiles.cuh): a lane draws the masks of four consecutive
// groups at once; a warp walks a contiguous range of tiles, queues the selected coordinates in
// a ring in shared memory and serves them 32 at a time, one per lane, so that the permutation
// draws and the N loads of a coordinate run on full warps although selected coordinates are
// rare and scattered.  The exchange is in place: a lane first loads the coordinate's N values
// into its column of shared memory, then stores the ones that move.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"
#include "wash_warp_tiles.cuh"
#include "wash_permutation.cuh"

namespace wash {

constexpr int kSparseWarps = 8;
constexpr int kSparseThreads = 32 * kSparseWarps;

struct SparseArgs {
    ShuffleArgs s;
    uint32_t n_wtiles;   // warp tiles in [group_lo, group_hi)
    uint32_t n_blocks;   // grid; its warps share the warp tiles evenly, in order
};

template <class TA, class TB, int LAYOUT>
__global__ void __launch_bounds__(kSparseThreads, 4) shuffle_sparse_kernel(const __grid_constant__ SparseArgs p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const ShuffleArgs &a = p.s;
    const int n_models = a.pop.N;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    // [a ring per warp][a column of N words per thread][a column of N bytes per thread, N > 16]
    uint32_t *ring = reinterpret_cast<uint32_t *>(smem_raw) + warp * kXRing;
    uint32_t *s_col = reinterpret_cast<uint32_t *>(smem_raw) + kSparseWarps * kXRing + threadIdx.x;
    uint8_t *s_perm = smem_raw + 4u * (kSparseWarps * kXRing + static_cast<uint32_t>(n_models) * kSparseThreads) + threadIdx.x;

    // this warp's tiles: t0 .. t1-1, tile t = groups group_lo + 128 t ..
    const uint64_t range = blockIdx.x * kSparseWarps + warp, ranges = static_cast<uint64_t>(p.n_blocks) * kSparseWarps;
    const uint32_t t0 = static_cast<uint32_t>(range * p.n_wtiles / ranges), t1 = static_cast<uint32_t>((range + 1) * p.n_wtiles / ranges);
    const uint64_t range_group = static_cast<uint64_t>(a.group_lo) + static_cast<uint64_t>(t0) * kWarpTileGroups;
    uint32_t cursor = (t0 < t1 && range_group < a.group_hi) ? __ldg(a.pop.tile_first + (range_group >> kTileShift)) : 0u;

    uint32_t selected = 0, moved = 0, head = 0, tail = 0;
    // one round: lane j takes entry head + j
    auto serve = [&](uint32_t count) {
        if (lane < count) {
            const long long e = 4ll * static_cast<long long>(range_group) + ring[(head + lane) % kXRing];
            const GroupInfo gi = find_group(a.pop, static_cast<uint32_t>(e >> 2), a.status);
            const uint32_t coord = 4u * gi.cgroup + static_cast<uint32_t>(e & 3);
            uint64_t perm = 0;
            if (n_models <= 16) perm = draw_permutation_packed(n_models, coord, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
            else draw_permutation_u8(s_perm, kSparseThreads, n_models, coord, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
            // nibble n of `perm` (N <= 16) or byte n of the column is the model whose value model n takes
            auto source_of = [&](int n, uint64_t rest) -> int {
                return n_models <= 16 ? static_cast<int>(static_cast<uint32_t>(rest) & 15u) : static_cast<int>(s_perm[n * kSparseThreads]);
            };
            // all N old values first (the exchange is in place), then the moved ones back
            for (int n = 0; n < n_models; ++n) s_col[n * kSparseThreads] = TA::load_elem(a.a, elem_index<LAYOUT>(a.pop, n, e));
            uint64_t rest = perm;
            for (int n = 0; n < n_models; ++n, rest >>= 4) {
                const int src = source_of(n, rest);
                if (src == n) continue;
                TA::store_elem(a.a, elem_index<LAYOUT>(a.pop, n, e), s_col[src * kSparseThreads]);
                ++moved;
            }
            if constexpr (kHasB) {
                for (int n = 0; n < n_models; ++n) s_col[n * kSparseThreads] = TB::load_elem(a.b, elem_index<LAYOUT>(a.pop, n, e));
                rest = perm;
                for (int n = 0; n < n_models; ++n, rest >>= 4) {
                    const int src = source_of(n, rest);
                    if (src != n) TB::store_elem(a.b, elem_index<LAYOUT>(a.pop, n, e), s_col[src * kSparseThreads]);
                }
            }
            ++selected;
        }
        __syncwarp();
        head += count;
    };
    LaneSegment ls{1, 0, 0, 0, 0};
    const uint32_t whole_tiles = (a.group_hi - a.group_lo) / kWarpTileGroups;   // tiles with all 128 groups inside the range
    for (uint32_t t = t0; t < t1; ++t) {
        uint32_t sel4 = 0;
        const uint32_t g0 = a.group_lo + t * kWarpTileGroups + 4u * lane;   // meaningful (no wrap) when t < whole_tiles
        if (!(t < whole_tiles && lane_masks_fast(a, g0, ls, &sel4))) {
            const uint64_t g0_wide = static_cast<uint64_t>(a.group_lo) + static_cast<uint64_t>(t) * kWarpTileGroups + 4u * lane;
            // ranges end on multiples of 4 groups: a lane's groups are all inside or all outside
            if (g0_wide < a.group_hi) sel4 = lane_masks_general(a, static_cast<uint32_t>(g0_wide), ls, cursor);
        }
        if (__any_sync(kFull, sel4 != 0)) {
            tail = ring_append(ring, tail, sel4, t - t0);
            while (tail - head >= 32u) serve(32u);
        }
    }
    if (tail != head) serve(tail - head);
    publish_block_stats(a.stats, a.stat_slots, selected, moved);
}

template <class TA, class TB>
cudaError_t launch_shuffle_sparse_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    if (args.group_hi <= args.group_lo) return cudaSuccess;
    SparseArgs p;
    p.s = args;
    p.n_wtiles = (args.group_hi - args.group_lo + kWarpTileGroups - 1) / kWarpTileGroups;
    const size_t n = static_cast<size_t>(args.pop.N);
    const size_t smem = 4 * (static_cast<size_t>(kSparseWarps) * kXRing + n * kSparseThreads) + (n > 16 ? n * kSparseThreads : 0);
    auto kernel = args.pop.layout == kLayoutNP ? shuffle_sparse_kernel<TA, TB, kLayoutNP> : shuffle_sparse_kernel<TA, TB, kLayoutPN>;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), kSparseThreads, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    // one resident wave of blocks, fewer for short rows; the warps share the tiles evenly
    const uint32_t resident = static_cast<uint32_t>(shape.sm_count > 0 ? shape.sm_count : 148) * static_cast<uint32_t>(fit.occupancy);
    const uint32_t want = (p.n_wtiles + kSparseWarps - 1) / kSparseWarps;
    // Grid: one resident wave when a warp expects few selected coordinates; up to four waves when it
    // expects many.  A warp serves its queue in full rounds and once at the end of its range, so with
    // one wave every warp reaches its (latency-bound) last round at the same time, after the
    // (multiply-bound) mask; with shorter ranges in several waves the block scheduler overlaps one
    // wave's serving with the next one's mask and evens out ranges that select unequally (per-layer p).
    // Measured (1 / 2 / 4 waves): cfg2 21.3 / 26.6 / 35.7 us at 2.4 coordinates a warp, cfg3 77.3 / 71.0 /
    // 75.6 us at 11, cfg4 104.1 / 94.4 / 89.4 us at 27.  A warp keeps at least two tiles.
    const double per_warp = static_cast<double>(args.expected_share) * 4.0 * static_cast<double>(args.group_hi - args.group_lo) /
                            (static_cast<double>(resident) * kSparseWarps);
    uint32_t waves = per_warp <= 8.0 ? 1u : (per_warp <= 20.0 ? 2u : 4u);
    while (waves > 1 && p.n_wtiles < 2ull * waves * resident * kSparseWarps) waves >>= 1;
    const uint32_t cap = resident * waves;
    p.n_blocks = want < cap ? want : cap;
    kernel<<<p.n_blocks, kSparseThreads, smem, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

inline cudaError_t launch_shuffle_sparse_tiles(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                               cudaStream_t stream, bool *supported)
{
    *supported = true;
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeNone) return launch_shuffle_sparse_typed<F32, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeNone) return launch_shuffle_sparse_typed<BF16, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeF32) return launch_shuffle_sparse_typed<F32, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeF32) return launch_shuffle_sparse_typed<BF16, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeBF16) return launch_shuffle_sparse_typed<BF16, BF16>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeBF16) return launch_shuffle_sparse_typed<F32, BF16>(args, shape, stream);
    *supported = false;
    return cudaSuccess;
}

}  // namespace wash
