// The shuffling step with one model per device: the worker form of Eq. 3.
//
// Every worker draws the same mask and the same permutations from the shared (seed, step),
// so only values cross the link.  Worker n owns a staging buffer; the selected coordinates
// with pi_i(n) != n take its slots in coordinate order and worker pi_i(n) stores its own
// value of the coordinate straight into the slot (a peer store when the buffer lives on
// another device).  After all workers have sent, each one copies its slots into its model.
//
// Three kernels and a small scan, all on tiles of 1024 groups (4096 coordinates; a block of
// 256 threads, four consecutive groups per thread so that the four Philox draws overlap):
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

constexpr int kXThreads = 256;
constexpr int kXPerThread = kExchangeTileGroups / kXThreads;   // consecutive groups per thread
static_assert(kXPerThread == 4, "a thread's mask bytes are moved as one 32-bit word");
constexpr int kXList = 1024;   // selected coordinates listed per pass of the send kernel

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

// the four groups of this thread: g0 .. g0+3
__device__ __forceinline__ uint32_t first_group() { return (blockIdx.x * kXThreads + threadIdx.x) * kXPerThread; }

// the mask of one group: bit c set iff coordinate c is selected
__device__ __forceinline__ uint32_t draw_mask(uint32_t cgroup, uint32_t tensor, uint64_t thr, int valid, const ExchangeArgs &a)
{
    const Philox4 w = philox4x32_10(cgroup, tensor, a.step_lo, a.step_hi8, a.key0, a.key1);
    const uint32_t thr_lo = static_cast<uint32_t>(thr);
    const bool always = (thr >> 32) != 0;
    uint32_t m = 0;
    m |= (w.x < thr_lo || always) ? 1u : 0u;
    m |= (w.y < thr_lo || always) ? 2u : 0u;
    m |= (w.z < thr_lo || always) ? 4u : 0u;
    m |= (w.w < thr_lo || always) ? 8u : 0u;
    return m & ((1u << valid) - 1u);
}

// Permutations of a group's selected coordinates: counts every worker's slots in s_count and
// returns the group's byte (low nibble sel, high nibble the coordinates this worker receives).
__device__ __forceinline__ uint32_t plan_selected(uint32_t sel, uint32_t cgroup, uint32_t tensor, uint8_t *s_perm,
                                                  uint32_t *s_count, const ExchangeArgs &a)
{
    const int n_models = a.pop.N;
    uint32_t byte = sel;
    for (uint32_t left = sel; left; left &= left - 1u) {
        const int c = __ffs(left) - 1;
        uint64_t packed = 0;
        if (n_models <= 16) packed = draw_permutation_packed(n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.key0, a.key1);
        else draw_permutation_u8(s_perm, kXThreads, n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.key0, a.key1);
        for (int n = 0; n < n_models; ++n)
            if (perm_source(n_models, packed, s_perm, n) != n) {
                atomicAdd(&s_count[n], 1u);
                if (n == a.self) byte |= 16u << c;
            }
        atomicAdd(&s_count[n_models], 1u);
    }
    return byte;
}

__global__ void __launch_bounds__(kXThreads, 5) exchange_plan_kernel(const __grid_constant__ ExchangeArgs a)
{
    extern __shared__ uint8_t s_perm_all[];   // column per thread (kMaxN * kXThreads bytes) when N > 16, else nothing
    __shared__ uint32_t s_count[kMaxN + 1];
    uint8_t *s_perm = s_perm_all + threadIdx.x;
    const int n_models = a.pop.N;
    if (threadIdx.x <= static_cast<uint32_t>(n_models)) s_count[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t g0 = first_group();
    uint32_t bytes = 0;
    if (g0 < a.pop.n_groups) {
        uint32_t cursor = __ldg(a.pop.tile_first + (g0 >> kTileShift));
        const GroupInfo gi0 = find_group_forward(a.pop.seg, a.pop.n_seg, cursor, g0, a.status);
        const uint32_t seg_end = a.pop.seg[cursor].group_end;
        if (g0 + kXPerThread <= seg_end) {
            // the usual case: the thread's four groups lie in one tensor -- one table lookup,
            // four independent Philox draws
            if (gi0.thr != 0 && gi0.valid != 0) {
                const long long left = static_cast<long long>(a.pop.seg[cursor].numel) - 4ll * (gi0.cgroup - a.pop.seg[cursor].cgroup_begin);
                uint32_t sel[kXPerThread];
#pragma unroll
                for (int q = 0; q < kXPerThread; ++q) {
                    const long long l = left - 4 * q;
                    const int valid = l >= 4 ? 4 : (l > 0 ? static_cast<int>(l) : 0);
                    sel[q] = draw_mask(gi0.cgroup + q, gi0.tensor_id, gi0.thr, valid, a);
                }
#pragma unroll
                for (int q = 0; q < kXPerThread; ++q)
                    if (sel[q]) bytes |= plan_selected(sel[q], gi0.cgroup + q, gi0.tensor_id, s_perm, s_count, a) << (8 * q);
            }
        } else {
#pragma unroll 1
            for (int q = 0; q < kXPerThread; ++q) {
                if (g0 + q >= a.pop.n_groups) break;
                const GroupInfo gi = find_group_forward(a.pop.seg, a.pop.n_seg, cursor, g0 + q, a.status);
                if (gi.thr == 0 || gi.valid == 0) continue;
                const uint32_t sel = draw_mask(gi.cgroup, gi.tensor_id, gi.thr, gi.valid, a);
                if (sel) bytes |= plan_selected(sel, gi.cgroup, gi.tensor_id, s_perm, s_count, a) << (8 * q);
            }
        }
    }
    reinterpret_cast<uint32_t *>(a.mask)[g0 / kXPerThread] = bytes;   // the array covers whole tiles
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

// A selected coordinate's value of this worker goes to at most one other worker: the n with
// pi(n) = self (pi is a permutation), unless pi(self) = self and it stays.
constexpr uint8_t kNoDestination = 0xFF;

__global__ void __launch_bounds__(kXThreads) exchange_send_kernel(const __grid_constant__ ExchangeArgs a)
{
    extern __shared__ uint8_t s_perm_all[];         // kMaxN * kXThreads bytes when N > 16, else nothing
    __shared__ unsigned long long s_need[kXList];   // bit n: the coordinate takes a slot of worker n
    __shared__ uint32_t s_slot[kXList];             // slot of the destination's buffer this worker fills
    __shared__ uint16_t s_offset[kXList];           // coordinate within the tile
    __shared__ uint8_t s_dest[kXList];              // the worker that receives this worker's value
    __shared__ uint32_t s_warp[kXThreads / 32];
    uint8_t *s_perm = s_perm_all + threadIdx.x;
    const int n_models = a.pop.N;
    const uint32_t g0 = first_group();
    const uint32_t bytes = reinterpret_cast<const uint32_t *>(a.mask)[g0 / kXPerThread];
    const uint32_t sel4 = bytes & 0x0F0F0F0Fu;
    if (!__syncthreads_or(sel4 != 0)) return;
    uint32_t listed = 0;
    const uint32_t first = block_exclusive_scan(__popc(sel4), s_warp, &listed);   // position of this thread's first entry
    // thread n numbers worker n's slots
    const int n = static_cast<int>(threadIdx.x);
    const bool walker = n < n_models && n != a.self;
    uint32_t slot = walker ? a.tile_count[static_cast<size_t>(n) * a.n_tiles + blockIdx.x] : 0u;
    const long long tile_elem = 4ll * kExchangeTileGroups * static_cast<long long>(blockIdx.x);
    uint32_t cursor = sel4 ? __ldg(a.pop.tile_first + (g0 >> kTileShift)) : 0u;
    // the list is served kXList entries at a time (one pass unless p is large)
    for (uint32_t base = 0; base < listed; base += kXList) {
        if (sel4) {
            uint32_t pos = first;
#pragma unroll 1
            for (int q = 0; q < kXPerThread; ++q) {
                const uint32_t sel = (sel4 >> (8 * q)) & 15u;
                if (!sel) continue;
                if (pos + 4 <= base || pos >= base + kXList) { pos += __popc(sel); continue; }   // not in this pass
                const GroupInfo gi = find_group_forward(a.pop.seg, a.pop.n_seg, cursor, g0 + q, a.status);
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    if (!((sel >> c) & 1u)) continue;
                    if (pos >= base && pos < base + kXList) {
                        uint64_t packed = 0;
                        if (n_models <= 16) packed = draw_permutation_packed(n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
                        else draw_permutation_u8(s_perm, kXThreads, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
                        unsigned long long need = 0;
                        uint8_t dest = kNoDestination;
                        for (int m = 0; m < n_models; ++m) {
                            const int src = perm_source(n_models, packed, s_perm, m);
                            if (src == m) continue;
                            need |= 1ull << m;
                            if (src == a.self) dest = static_cast<uint8_t>(m);
                        }
                        s_need[pos - base] = need;
                        s_dest[pos - base] = dest;
                        s_offset[pos - base] = static_cast<uint16_t>(4u * (kXPerThread * threadIdx.x + q) + c);
                    }
                    ++pos;
                }
            }
        }
        __syncthreads();
        const uint32_t count = min(listed - base, static_cast<uint32_t>(kXList));
        if (walker) {   // shared memory only: no load from the model sits in this serial loop
            for (uint32_t e = 0; e < count; ++e) {
                if (!((s_need[e] >> n) & 1ull)) continue;
                if (s_dest[e] == n) s_slot[e] = slot;
                ++slot;
            }
        }
        __syncthreads();
        // the copies, one entry per thread: all loads of the pass are in flight together
        for (uint32_t e = threadIdx.x; e < count; e += kXThreads) {
            const uint32_t dest = s_dest[e];
            if (dest == kNoDestination) continue;
            const long long to = s_slot[e];
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (!a.row[k]) continue;
                if (to < a.capacity[k]) copy_element(a.staging[k][dest], to, a.row[k], tile_elem + s_offset[e], a.dtype[k]);
                else atomicOr(a.status, 4u);   // staging buffer too small: nothing is written beyond it
            }
        }
        __syncthreads();   // the list is rewritten by the next pass
    }
}

__global__ void __launch_bounds__(kXThreads) exchange_receive_kernel(const __grid_constant__ ExchangeArgs a)
{
    __shared__ uint32_t s_warp[kXThreads / 32];
    if (a.stats && blockIdx.x == 0 && threadIdx.x == 0) {
        atomicAdd(a.stats, static_cast<unsigned long long>(a.total[a.pop.N]));
        atomicAdd(a.stats + 1, static_cast<unsigned long long>(a.total[a.self]));
    }
    const uint32_t g0 = first_group();
    const uint32_t take4 = (reinterpret_cast<const uint32_t *>(a.mask)[g0 / kXPerThread] >> 4) & 0x0F0F0F0Fu;
    if (!__syncthreads_or(take4 != 0)) return;
    uint32_t total = 0;
    uint32_t slot = a.tile_count[static_cast<size_t>(a.self) * a.n_tiles + blockIdx.x] + block_exclusive_scan(__popc(take4), s_warp, &total);
    if (!take4) return;
    const void *src[2] = {a.row[0] ? a.staging[0][a.self] : nullptr, a.row[1] ? a.staging[1][a.self] : nullptr};
#pragma unroll 1
    for (int q = 0; q < kXPerThread; ++q) {
        const uint32_t take = (take4 >> (8 * q)) & 15u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (!((take >> c) & 1u)) continue;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (!a.row[k]) continue;
                if (static_cast<long long>(slot) < a.capacity[k]) copy_element(a.row[k], 4ll * (g0 + q) + c, src[k], slot, a.dtype[k]);
                else atomicOr(a.status, 4u);
            }
            ++slot;
        }
    }
}

cudaError_t launch_exchange_plan(const ExchangeArgs &args, cudaStream_t stream)
{
    if (args.n_tiles == 0) return cudaSuccess;
    const size_t smem = args.pop.N > 16 ? static_cast<size_t>(kMaxN) * kXThreads : 0;
    exchange_plan_kernel<<<args.n_tiles, kXThreads, smem, stream>>>(args);
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
    const size_t smem = args.pop.N > 16 ? static_cast<size_t>(kMaxN) * kXThreads : 0;
    exchange_send_kernel<<<args.n_tiles, kXThreads, smem, stream>>>(args);
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
