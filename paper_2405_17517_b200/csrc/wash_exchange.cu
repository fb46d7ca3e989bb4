// The shuffling step with one model per device: the worker form of Eq. 3.
//
// Every worker draws the same mask and the same permutations from the shared (seed, step),
// so only values cross the link.  Worker n owns a staging buffer; the selected coordinates
// with pi_i(n) != n take its slots in coordinate order and worker pi_i(n) stores its own
// value of the coordinate straight into the slot (a peer store when the buffer lives on
// another device).  After all workers have sent, each one copies its slots into its model.
//
// Three kernels and a small scan, all on tiles of 256 groups (1024 coordinates, one group
// per thread):
//   plan     draws the mask (one Philox block per group) and, for selected coordinates, the
//            permutation; writes one byte per group (low nibble: selected coordinates, high
//            nibble: those whose new value comes from another worker) and, per tile, how many
//            slots of every worker's buffer the tile takes (+ the selected count)
//   scan     turns each worker's column of tile counts into slot offsets (one block per column)
//   send     lists the tile's selected coordinates in order, redraws their permutations, and
//            lets thread n walk the list for worker n: it counts worker n's slots and stores
//            this worker's value where pi_i(n) is this worker
//   receive  reads the bytes, numbers its own slots with a block scan and copies them in
// The plan reads no model data; send and receive touch only selected coordinates.
#include "wash_device.cuh"
#include "wash_launch.cuh"
#include "wash_shuffle_tma.cuh"     // draw_permutation_u8
#include "wash_shuffle_async.cuh"   // draw_permutation_packed

namespace wash {

constexpr int kXThreads = kExchangeTileGroups;

// exclusive prefix sum of `mine` over the block's threads (in thread order); *total = block sum
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t mine, uint32_t *s_warp, uint32_t *total)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t upto = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, upto, d);
        if (lane >= static_cast<uint32_t>(d)) upto += v;
    }
    if (lane == 31) s_warp[warp] = upto;
    __syncthreads();
    uint32_t before = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < kXThreads / 32; ++w) {
        const uint32_t v = s_warp[w];
        if (static_cast<uint32_t>(w) < warp) before += v;
        sum += v;
    }
    *total = sum;
    return before + upto - mine;
}

// source model pi(n) out of either representation of the permutation
__device__ __forceinline__ int perm_source(int n_models, uint64_t packed, const uint8_t *s_perm, int n)
{
    return n_models <= 16 ? static_cast<int>((packed >> (4 * n)) & 15ull) : static_cast<int>(s_perm[n * kXThreads]);
}

__global__ void __launch_bounds__(kXThreads) exchange_plan_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ uint32_t s_count[kMaxN + 1];
    __shared__ uint8_t s_perm_all[kMaxN * kXThreads];   // column per thread, used when N > 16
    uint8_t *s_perm = s_perm_all + threadIdx.x;
    const int n_models = a.pop.N;
    if (threadIdx.x <= static_cast<uint32_t>(n_models)) s_count[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t g = blockIdx.x * kXThreads + threadIdx.x;
    if (g < a.pop.n_groups) {
        uint32_t byte = 0;
        const GroupInfo gi = find_group(a.pop, g, a.status);
        if (gi.thr != 0 && gi.valid != 0) {
            const Philox4 w = philox4x32_10(gi.cgroup, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
            const uint32_t thr_lo = static_cast<uint32_t>(gi.thr);
            const bool always = (gi.thr >> 32) != 0;
            uint32_t sel = 0;
            sel |= (w.x < thr_lo || always) ? 1u : 0u;
            sel |= (w.y < thr_lo || always) ? 2u : 0u;
            sel |= (w.z < thr_lo || always) ? 4u : 0u;
            sel |= (w.w < thr_lo || always) ? 8u : 0u;
            sel &= (1u << gi.valid) - 1u;
            byte = sel;
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                if (!((sel >> c) & 1u)) continue;
                uint64_t packed = 0;
                if (n_models <= 16) packed = draw_permutation_packed(n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
                else draw_permutation_u8(s_perm, kXThreads, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
                for (int n = 0; n < n_models; ++n)
                    if (perm_source(n_models, packed, s_perm, n) != n) {
                        atomicAdd(&s_count[n], 1u);
                        if (n == a.self) byte |= 16u << c;
                    }
                atomicAdd(&s_count[n_models], 1u);
            }
        }
        a.mask[g] = static_cast<uint8_t>(byte);
    }
    __syncthreads();
    if (threadIdx.x <= static_cast<uint32_t>(n_models))
        a.tile_count[static_cast<size_t>(threadIdx.x) * a.n_tiles + blockIdx.x] = s_count[threadIdx.x];
}

// One block per column: counts -> exclusive prefix sums in place, column total to a.total.
__global__ void __launch_bounds__(1024) exchange_scan_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ uint32_t s_warp[32];
    uint32_t *col = a.tile_count + static_cast<size_t>(blockIdx.x) * a.n_tiles;
    const uint32_t chunk = (a.n_tiles + 1023u) / 1024u;
    const uint32_t lo = min(threadIdx.x * chunk, a.n_tiles), hi = min(lo + chunk, a.n_tiles);
    uint32_t sum = 0;
    for (uint32_t t = lo; t < hi; ++t) sum += col[t];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t upto = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, upto, d);
        if (lane >= static_cast<uint32_t>(d)) upto += v;
    }
    if (lane == 31) s_warp[warp] = upto;
    __syncthreads();
    uint32_t before = 0, total = 0;
    for (uint32_t w = 0; w < 32; ++w) {
        const uint32_t v = s_warp[w];
        if (w < warp) before += v;
        total += v;
    }
    uint32_t run = before + upto - sum;
    for (uint32_t t = lo; t < hi; ++t) {
        const uint32_t v = col[t];
        col[t] = run;
        run += v;
    }
    if (threadIdx.x == 0) a.total[blockIdx.x] = total;
}

__device__ __forceinline__ void copy_element(void *dst, long long dst_idx, const void *src, long long src_idx, int dtype)
{
    if (dtype == kDtypeF32) static_cast<uint32_t *>(dst)[dst_idx] = static_cast<const uint32_t *>(src)[src_idx];
    else static_cast<uint16_t *>(dst)[dst_idx] = static_cast<const uint16_t *>(src)[src_idx];
}

__global__ void __launch_bounds__(kXThreads) exchange_send_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ unsigned long long s_need[4 * kXThreads];   // bit n: the coordinate takes a slot of worker n
    __shared__ unsigned long long s_mine[4 * kXThreads];   // bit n: ... and this worker fills it
    __shared__ uint16_t s_offset[4 * kXThreads];           // coordinate within the tile
    __shared__ uint32_t s_warp[kXThreads / 32];
    __shared__ uint8_t s_perm_all[kMaxN * kXThreads];
    uint8_t *s_perm = s_perm_all + threadIdx.x;
    const int n_models = a.pop.N;
    const uint32_t g = blockIdx.x * kXThreads + threadIdx.x;
    const uint32_t sel = g < a.pop.n_groups ? (a.mask[g] & 15u) : 0u;
    if (!__syncthreads_or(sel != 0)) return;   // at small p most tiles have nothing selected
    uint32_t listed = 0;
    uint32_t pos = block_exclusive_scan(__popc(sel), s_warp, &listed);
    if (sel) {
        const GroupInfo gi = find_group(a.pop, g, a.status);
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            if (!((sel >> c) & 1u)) continue;
            uint64_t packed = 0;
            if (n_models <= 16) packed = draw_permutation_packed(n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
            else draw_permutation_u8(s_perm, kXThreads, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
            unsigned long long need = 0, mine = 0;
            for (int n = 0; n < n_models; ++n) {
                const int src = perm_source(n_models, packed, s_perm, n);
                if (src == n) continue;
                need |= 1ull << n;
                if (src == a.self) mine |= 1ull << n;
            }
            s_need[pos] = need;
            s_mine[pos] = mine;
            s_offset[pos] = static_cast<uint16_t>(4u * threadIdx.x + c);
            ++pos;
        }
    }
    __syncthreads();
    const int n = static_cast<int>(threadIdx.x);   // this thread numbers worker n's slots
    if (n >= n_models || n == a.self) return;
    uint32_t slot = a.tile_count[static_cast<size_t>(n) * a.n_tiles + blockIdx.x];
    const long long tile_elem = 4ll * kXThreads * static_cast<long long>(blockIdx.x);
    void *dst[2] = {a.row[0] ? a.staging[0][n] : nullptr, a.row[1] ? a.staging[1][n] : nullptr};
    for (uint32_t e = 0; e < listed; ++e) {
        if (!((s_need[e] >> n) & 1ull)) continue;
        if ((s_mine[e] >> n) & 1ull) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (!a.row[k]) continue;
                if (static_cast<long long>(slot) < a.capacity[k]) copy_element(dst[k], slot, a.row[k], tile_elem + s_offset[e], a.dtype[k]);
                else atomicOr(a.status, 4u);   // staging buffer too small: nothing is written beyond it
            }
        }
        ++slot;
    }
}

__global__ void __launch_bounds__(kXThreads) exchange_receive_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ uint32_t s_warp[kXThreads / 32];
    if (a.stats && blockIdx.x == 0 && threadIdx.x == 0) {
        atomicAdd(a.stats, static_cast<unsigned long long>(a.total[a.pop.N]));
        atomicAdd(a.stats + 1, static_cast<unsigned long long>(a.total[a.self]));
    }
    const uint32_t g = blockIdx.x * kXThreads + threadIdx.x;
    const uint32_t take = g < a.pop.n_groups ? (a.mask[g] >> 4) : 0u;
    if (!__syncthreads_or(take != 0)) return;
    uint32_t total = 0;
    uint32_t slot = a.tile_count[static_cast<size_t>(a.self) * a.n_tiles + blockIdx.x] + block_exclusive_scan(__popc(take), s_warp, &total);
    if (!take) return;
    const void *src[2] = {a.row[0] ? a.staging[0][a.self] : nullptr, a.row[1] ? a.staging[1][a.self] : nullptr};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        if (!((take >> c) & 1u)) continue;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (!a.row[k]) continue;
            if (static_cast<long long>(slot) < a.capacity[k]) copy_element(a.row[k], 4ll * g + c, src[k], slot, a.dtype[k]);
            else atomicOr(a.status, 4u);
        }
        ++slot;
    }
}

cudaError_t launch_exchange_plan(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_tiles == 0) return cudaSuccess;
    exchange_plan_kernel<<<args.n_tiles, kXThreads, 0, stream>>>(args);
    count_launch();
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    exchange_scan_kernel<<<args.pop.N + 1, 1024, 0, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_exchange_send(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_tiles == 0) return cudaSuccess;
    exchange_send_kernel<<<args.n_tiles, kXThreads, 0, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_exchange_receive(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_tiles == 0) return cudaSuccess;
    exchange_receive_kernel<<<args.n_tiles, kXThreads, 0, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

}  // namespace wash
