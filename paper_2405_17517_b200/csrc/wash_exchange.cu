// The shuffling step with one model per device: the worker form of Eq. 3.
//
// Every worker draws the same mask and the same permutations from the shared (seed, step),
// so only values cross the link.  Worker n owns a staging buffer; the selected coordinates
// with pi_i(n) != n take its slots in coordinate order and worker pi_i(n) stores its own
// value of the coordinate straight into the slot (a peer store when the buffer lives on
// another device).  After all workers have sent, each one copies its slots into its model.
//
// Work is cut into warp tiles of 128 groups (512 coordinates: a lane owns four consecutive
// groups, so its four Philox draws overlap and its four mask bytes move as one word).  A
// warp owns a contiguous range of warp tiles and visits them in order, which turns "the
// slot of a coordinate" into a running count: no per-tile offsets are stored, only one
// total per warp and per block, and the kernels need no block-wide barrier inside the loop.
//   plan     draws the mask and, for selected coordinates, the permutation; writes a byte per
//            group (low nibble: selected coordinates, high nibble: those whose new value comes
//            from another worker) and, per warp and per block, how many slots of every
//            worker's buffer its range takes (+ the selected count)
//   send     adds up the totals of the blocks and warps before it (its first slots), then
//            replays its range: redraws the permutations of the selected coordinates, numbers
//            every worker's slots with warp votes and stores this worker's value where
//            pi_i(n) is this worker
//   receive  the same replay for its own buffer only, from the high nibbles: no draw at all
// The plan reads no model data; send and receive touch only selected coordinates.
// All three kernels must be launched with the same grid (n_blocks).
#include "wash_device.cuh"
#include "wash_launch.cuh"
#include "wash_warp_tiles.cuh"
#include "wash_permutation.cuh"

namespace wash {

constexpr int kXThreads = 32 * kExchangeWarps;
static_assert(kExchangeTileGroups == kWarpTileGroups, "the exchange works on warp tiles");
constexpr uint32_t kNoDestination = 0xFFu;

// pi of the coordinate stored at row element `elem`, as {need: bit n set iff pi(n) != n,
// dest: the n != self with pi(n) == self, if any}
__device__ __forceinline__ void routes_of(const ExchangeArgs &a, uint32_t elem, uint8_t *s_perm,
                                          unsigned long long *need, uint32_t *dest)
{
    const int n_models = a.pop.N;
    const GroupInfo gi = find_group(a.pop, elem >> 2, a.status);
    const uint32_t coord = 4u * gi.cgroup + (elem & 3u);
    uint64_t packed = 0;
    if (n_models <= 16) packed = draw_permutation_packed(n_models, coord, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
    else draw_permutation_u8(s_perm, kXThreads, n_models, coord, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
    unsigned long long nd = 0;
    uint32_t d = kNoDestination;
    for (int n = 0; n < n_models; ++n) {
        const int src = n_models <= 16 ? static_cast<int>((packed >> (4 * n)) & 15ull) : static_cast<int>(s_perm[n * kXThreads]);
        if (src == n) continue;
        nd |= 1ull << n;
        if (src == a.self) d = static_cast<uint32_t>(n);
    }
    *need = nd;
    *dest = d;
}

// first and one-past-last warp tile of this warp (the n_wtiles tiles are dealt out evenly,
// in order, to the grid's warps), and the cursor into the segment table for the first
__device__ __forceinline__ void warp_range(const ExchangeArgs &a, uint32_t *t0, uint32_t *t1, uint32_t *cursor)
{
    const uint64_t range = blockIdx.x * kExchangeWarps + (threadIdx.x >> 5);
    const uint64_t ranges = static_cast<uint64_t>(a.n_blocks) * kExchangeWarps;
    *t0 = static_cast<uint32_t>(range * a.n_wtiles / ranges);
    *t1 = static_cast<uint32_t>((range + 1) * a.n_wtiles / ranges);
    const uint32_t g = *t0 * kExchangeTileGroups;
    *cursor = (*t0 < *t1 && g < a.pop.n_groups) ? __ldg(a.pop.tile_first + (g >> kTileShift)) : 0u;
}

__global__ void __launch_bounds__(kXThreads, kExchangeBlocksPerSm) exchange_plan_kernel(const __grid_constant__ ExchangeArgs a)
{
    extern __shared__ uint8_t s_perm_all[];   // column per thread (kMaxN * kXThreads bytes) when N > 16, else nothing
    __shared__ uint32_t s_count[kExchangeWarps][kMaxN + 1];
    __shared__ uint32_t s_ring[kExchangeWarps][kXRing];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const int n_models = a.pop.N, columns = n_models + 1;
    for (int col = lane; col < columns; col += 32) s_count[warp][col] = 0;
    __syncwarp();
    uint32_t t0, t1, cursor;
    warp_range(a, &t0, &t1, &cursor);
    uint32_t head = 0, tail = 0;   // ring positions served / queued so far
    const uint32_t range_elem = 4u * kExchangeTileGroups * t0;   // first row element of the warp's range (rows are shorter than 2^32)
    // one round: lane j takes entry head + j; counts every worker's slots and marks the
    // coordinates this worker receives in the (already written) mask words
    auto serve = [&](uint32_t count) {
        if (lane < count) {
            const uint32_t elem = range_elem + s_ring[warp][(head + lane) % kXRing];
            unsigned long long need;
            uint32_t dest;
            routes_of(a, elem, s_perm_all + threadIdx.x, &need, &dest);
            for (unsigned long long left = need; left; left &= left - 1ull) atomicAdd(&s_count[warp][__ffsll(static_cast<long long>(left)) - 1], 1u);
            atomicAdd(&s_count[warp][n_models], 1u);
            if ((need >> a.self) & 1ull) {
                const uint32_t g = elem >> 2;   // byte g % 4 of word g / 4, bit 4 + c
                atomicOr(&a.mask[g >> 2], 16u << ((elem & 3u) + 8u * (g & 3u)));
            }
        }
        __syncwarp();
        head += count;
    };
    LaneSegment ls{1, 0, 0, 0, 0};
    const uint32_t whole_tiles = a.pop.n_groups / kExchangeTileGroups;   // tiles with all 128 groups inside the row
    for (uint32_t t = t0; t < t1; ++t) {
        const uint32_t g0 = t * kExchangeTileGroups + 4u * lane;   // rows are shorter than 2^32 elements: no wrap
        uint32_t sel4 = 0;
        if (!(t < whole_tiles && lane_masks_fast(a, g0, ls, &sel4))) sel4 = lane_masks_general(a, g0, ls, cursor);
        a.mask[static_cast<size_t>(t) * 32u + lane] = sel4;
        if (__any_sync(kFull, sel4 != 0)) {
            tail = ring_append(s_ring[warp], tail, sel4, t - t0);   // orders the mask stores before the rounds' atomics, too
            while (tail - head >= 32u) serve(32u);
        }
    }
    if (tail != head) serve(tail - head);
    const uint32_t range = blockIdx.x * kExchangeWarps + warp;
    for (int col = lane; col < columns; col += 32) a.warp_total[static_cast<size_t>(range) * columns + col] = s_count[warp][col];
    __syncthreads();
    if (threadIdx.x < static_cast<uint32_t>(columns)) {
        uint32_t sum = 0;
#pragma unroll
        for (int w = 0; w < kExchangeWarps; ++w) sum += s_count[w][threadIdx.x];
        a.block_total[static_cast<size_t>(blockIdx.x) * columns + threadIdx.x] = sum;
    }
}

__device__ __forceinline__ void copy_element(void *dst, long long dst_idx, const void *src, long long src_idx, int dtype)
{
    if (dtype == kDtypeF32) static_cast<uint32_t *>(dst)[dst_idx] = static_cast<const uint32_t *>(src)[src_idx];
    else static_cast<uint16_t *>(dst)[dst_idx] = static_cast<const uint16_t *>(src)[src_idx];
}

// Sum over the blocks before this one of column `col` of block_total, by one warp.
__device__ __forceinline__ uint32_t blocks_before(const ExchangeArgs &a, int col)
{
    const uint32_t lane = threadIdx.x & 31u;
    const int columns = a.pop.N + 1;
    uint32_t sum = 0;
    for (uint32_t b = lane; b < blockIdx.x; b += 32) sum += a.block_total[static_cast<size_t>(b) * columns + col];
    return __reduce_add_sync(kFull, sum);
}

__global__ void __launch_bounds__(kXThreads) exchange_send_kernel(const __grid_constant__ ExchangeArgs a)
{
    extern __shared__ uint8_t s_perm_all[];
    __shared__ uint32_t s_base[kMaxN];
    __shared__ uint32_t s_ring[kExchangeWarps][kXRing];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const int n_models = a.pop.N, columns = n_models + 1;
    // slots of every worker's buffer taken before this block, then before this warp
    for (int col = warp; col < n_models; col += kExchangeWarps) {
        const uint32_t sum = blocks_before(a, col);
        if (lane == 0) s_base[col] = sum;
    }
    __syncthreads();
    uint32_t run[2] = {0, 0};   // next slot of worker lane (run[0]) and worker lane + 32 (run[1])
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int col = static_cast<int>(lane) + 32 * h;
        if (col >= n_models) continue;
        uint32_t sum = s_base[col];
        for (uint32_t w = 0; w < warp; ++w) sum += a.warp_total[static_cast<size_t>(blockIdx.x * kExchangeWarps + w) * columns + col];
        run[h] = sum;
    }
    uint32_t t0, t1, cursor;
    warp_range(a, &t0, &t1, &cursor);
    uint32_t head = 0, tail = 0;
    const uint32_t range_elem = 4u * kExchangeTileGroups * t0;
    // one round: lane j takes entry head + j (coordinate order along the lanes); the warp votes
    // worker by worker to number the slots, then every lane with a destination copies its value
    auto serve = [&](uint32_t count) {
        unsigned long long need = 0;
        uint32_t dest = kNoDestination, elem = 0;
        if (lane < count) {
            elem = range_elem + s_ring[warp][(head + lane) % kXRing];
            routes_of(a, elem, s_perm_all + threadIdx.x, &need, &dest);
        }
        uint32_t slot = 0;
        for (int n = 0; n < n_models; ++n) {
            const uint32_t votes = __ballot_sync(kFull, (need >> n) & 1ull);
            const uint32_t next = __shfl_sync(kFull, n < 32 ? run[0] : run[1], n & 31);
            if (dest == static_cast<uint32_t>(n)) slot = next + __popc(votes & ((1u << lane) - 1u));
            if (lane == static_cast<uint32_t>(n & 31)) {
                if (n < 32) run[0] += __popc(votes);
                else run[1] += __popc(votes);
            }
        }
        if (dest != kNoDestination) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (!a.row[k]) continue;
                if (static_cast<long long>(slot) < a.capacity[k]) copy_element(a.staging[k][dest], slot, a.row[k], elem, a.dtype[k]);
                else atomicOr(a.status, 4u);   // staging buffer too small: nothing is written beyond it
            }
        }
        __syncwarp();
        head += count;
    };
    for (uint32_t t = t0; t < t1; ++t) {
        const uint32_t sel4 = a.mask[static_cast<size_t>(t) * 32u + lane] & 0x0F0F0F0Fu;
        if (!__any_sync(kFull, sel4 != 0)) continue;
        tail = ring_append(s_ring[warp], tail, sel4, t - t0);
        while (tail - head >= 32u) serve(32u);
    }
    if (tail != head) serve(tail - head);
}

__global__ void __launch_bounds__(kXThreads) exchange_receive_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ uint32_t s_part[kExchangeWarps];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const int columns = a.pop.N + 1;
    if (a.stats && blockIdx.x == 0 && warp < 2) {   // the step's totals: selected coordinates, values this worker receives
        const int col = warp == 0 ? a.pop.N : a.self;
        uint32_t sum = 0;
        for (uint32_t b = lane; b < a.n_blocks; b += 32) sum += a.block_total[static_cast<size_t>(b) * columns + col];
        sum = __reduce_add_sync(kFull, sum);
        if (lane == 0) atomicAdd(a.stats + warp, static_cast<unsigned long long>(sum));
    }
    // slots of this worker's buffer taken before this block (all warps share the sum), then before this warp
    {
        uint32_t sum = 0;
        for (uint32_t b = threadIdx.x; b < blockIdx.x; b += kXThreads) sum += a.block_total[static_cast<size_t>(b) * columns + a.self];
        sum = __reduce_add_sync(kFull, sum);
        if (lane == 0) s_part[warp] = sum;
    }
    __syncthreads();
    uint32_t run = 0;
#pragma unroll
    for (int w = 0; w < kExchangeWarps; ++w) run += s_part[w];
    for (uint32_t w = 0; w < warp; ++w) run += a.warp_total[static_cast<size_t>(blockIdx.x * kExchangeWarps + w) * columns + a.self];
    uint32_t t0, t1, cursor;
    warp_range(a, &t0, &t1, &cursor);
    const void *src[2] = {a.row[0] ? a.staging[0][a.self] : nullptr, a.row[1] ? a.staging[1][a.self] : nullptr};
    for (uint32_t t = t0; t < t1; ++t) {
        const uint32_t take4 = (a.mask[static_cast<size_t>(t) * 32u + lane] >> 4) & 0x0F0F0F0Fu;
        if (!__any_sync(kFull, take4 != 0)) continue;
        uint32_t total = 0;
        uint32_t slot = run + warp_exclusive_scan(__popc(take4), &total);
        run += total;
        const long long lane_elem = 4ll * (static_cast<long long>(t) * kExchangeTileGroups + 4u * lane);
        for (uint32_t left = take4; left; left &= left - 1u, ++slot) {
            const int bit = __ffs(left) - 1;   // byte q = bit / 8, coordinate c = bit % 8
            const long long elem = lane_elem + 4 * (bit >> 3) + (bit & 7);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (!a.row[k]) continue;
                if (static_cast<long long>(slot) < a.capacity[k]) copy_element(a.row[k], elem, src[k], slot, a.dtype[k]);
                else atomicOr(a.status, 4u);
            }
        }
    }
}

// Populations above 16 models keep their permutations in a column of bytes per thread: with
// the kernels' static shared memory that is more than the default 48 KiB per block, so the
// kernel's limit is raised first.
static cudaError_t perm_smem(const ExchangeArgs &args, const void *kernel, size_t *bytes)
{
    *bytes = args.pop.N > 16 ? static_cast<size_t>(kMaxN) * kXThreads : 0;
    if (*bytes == 0) return cudaSuccess;
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(*bytes));
}

cudaError_t launch_exchange_plan(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_blocks == 0) return cudaSuccess;
    size_t smem = 0;
    cudaError_t err = perm_smem(args, reinterpret_cast<const void *>(exchange_plan_kernel), &smem);
    if (err != cudaSuccess) return err;
    exchange_plan_kernel<<<args.n_blocks, kXThreads, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_exchange_send(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_blocks == 0) return cudaSuccess;
    size_t smem = 0;
    cudaError_t err = perm_smem(args, reinterpret_cast<const void *>(exchange_send_kernel), &smem);
    if (err != cudaSuccess) return err;
    exchange_send_kernel<<<args.n_blocks, kXThreads, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_exchange_receive(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_blocks == 0) return cudaSuccess;
    exchange_receive_kernel<<<args.n_blocks, kXThreads, 0, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

}  // namespace wash
