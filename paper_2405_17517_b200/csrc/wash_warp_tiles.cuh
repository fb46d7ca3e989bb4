// Warp tiles: the work unit of the kernels that draw the mask without touching the stacks (the
// sparse shuffle and the one-model-per-device exchange).  A warp tile is 128 consecutive groups
// (512 coordinates); a lane owns four consecutive groups of it, so that its four Philox draws
// overlap, one table lookup serves all four, and its four mask nibbles fit one word.  A warp
// visits a contiguous range of warp tiles in order.
//
// `A` is the kernel's argument struct; it has the fields pop, keys, step_lo, step_hi8, status.
#pragma once
#include "wash_device.cuh"

namespace wash {

constexpr int kWarpTileGroups = 128;
constexpr uint32_t kFull = 0xFFFFFFFFu;

// What a lane knows about its four consecutive groups g0 .. g0+3.
struct LaneGroups {
    bool one_tensor;   // all four lie in one tensor (the usual case): described by the fields below
    uint32_t cgroup0, tensor;
    uint64_t thr;
    long long left;    // coordinates of the tensor from the first group on
};

template <class A>
__device__ __forceinline__ LaneGroups describe_groups(const A &a, uint32_t g0, uint32_t &cursor)
{
    LaneGroups lg{true, 0, 0, 0, 0};
    if (g0 >= a.pop.n_groups) return lg;   // thr == 0: nothing to draw
    const GroupInfo gi = find_group_forward(a.pop.seg, a.pop.n_seg, cursor, g0, a.status);
    const SegEntry &seg = a.pop.seg[cursor];
    lg.one_tensor = g0 + 4 <= seg.group_end;
    lg.cgroup0 = gi.cgroup;
    lg.tensor = gi.tensor_id;
    lg.thr = gi.thr;
    lg.left = static_cast<long long>(seg.numel) - 4ll * (gi.cgroup - seg.cgroup_begin);
    return lg;
}

// group q of the lane
template <class A>
__device__ __forceinline__ GroupInfo lane_group(const A &a, const LaneGroups &lg, uint32_t g0, int q)
{
    if (lg.one_tensor) {
        const long long l = lg.left - 4 * q;
        return GroupInfo{lg.tensor, lg.cgroup0 + q, l >= 4 ? 4 : (l > 0 ? static_cast<int>(l) : 0), lg.thr};
    }
    if (g0 + q >= a.pop.n_groups) return GroupInfo{0, 0, 0, 0};
    return find_group(a.pop, g0 + q, a.status);
}

// the mask of one group: bit c set iff coordinate c is selected
template <class A>
__device__ __forceinline__ uint32_t draw_mask(const GroupInfo &gi, const A &a)
{
    if (gi.thr == 0 || gi.valid == 0) return 0;
    const Philox4 w = philox4x32_10(gi.cgroup, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
    const uint32_t thr_lo = static_cast<uint32_t>(gi.thr);
    const bool always = (gi.thr >> 32) != 0;
    uint32_t m = 0;
    m |= (w.x < thr_lo || always) ? 1u : 0u;
    m |= (w.y < thr_lo || always) ? 2u : 0u;
    m |= (w.z < thr_lo || always) ? 4u : 0u;
    m |= (w.w < thr_lo || always) ? 8u : 0u;
    return m & ((1u << gi.valid) - 1u);
}

// The segment a lane's groups were last found in, kept in registers.  While the lane's four
// groups lie among that segment's whole groups a tile costs two compares, four Philox blocks
// and sixteen word compares (lane_masks_fast); everything else -- a tensor's end, its ragged
// last group, a threshold of 2^32 -- takes lane_masks_general, which also refreshes the
// registers.  Starts empty: {1, 0, 0, 0, 0}.
struct LaneSegment {
    uint32_t begin, full_end;   // the segment's whole groups (full_end = 0: none take the fast path)
    uint32_t cgroup_off;        // group index within the tensor = group + cgroup_off (modulo 2^32)
    uint32_t tensor, thr;
};

// The masks of groups g0 .. g0+3 (a nibble per byte) if they are whole groups of the lane's
// segment; false if the general path must take them.  g0 + 4 must not wrap.
template <class A>
__device__ __forceinline__ bool lane_masks_fast(const A &a, uint32_t g0, const LaneSegment &ls, uint32_t *sel4)
{
    if (g0 < ls.begin || g0 + 4u > ls.full_end) return false;
    uint32_t m4 = 0;
    if (ls.thr != 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const Philox4 w = philox4x32_10(g0 + ls.cgroup_off + q, ls.tensor, a.step_lo, a.step_hi8, a.keys);
            const uint32_t m = (w.x < ls.thr ? 1u : 0u) | (w.y < ls.thr ? 2u : 0u) | (w.z < ls.thr ? 4u : 0u) | (w.w < ls.thr ? 8u : 0u);
            m4 |= m << (8 * q);
        }
    }
    *sel4 = m4;
    return true;
}

// The same for any four groups of the row (those beyond its end select nothing).
template <class A>
__device__ __forceinline__ uint32_t lane_masks_general(const A &a, uint32_t g0, LaneSegment &ls, uint32_t &cursor)
{
    uint32_t sel4 = 0;
    const LaneGroups lg = describe_groups(a, g0, cursor);
    if (lg.one_tensor) {
        if (lg.thr != 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) sel4 |= draw_mask(lane_group(a, lg, g0, q), a) << (8 * q);
        }
    } else {
#pragma unroll 1
        for (int q = 0; q < 4; ++q) sel4 |= draw_mask(lane_group(a, lg, g0, q), a) << (8 * q);
    }
    const SegEntry &se = a.pop.seg[cursor];
    ls.begin = se.group_begin;
    ls.full_end = (se.thr >> 32) != 0 ? 0u : se.group_begin + se.numel / 4u;   // 2^32 selects always: general path
    ls.cgroup_off = se.cgroup_begin - se.group_begin;
    ls.tensor = se.tensor_id;
    ls.thr = static_cast<uint32_t>(se.thr);
    return sel4;
}

__device__ __forceinline__ uint32_t warp_exclusive_scan(uint32_t mine, uint32_t *total)
{
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t upto = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(kFull, upto, d);
        if (lane >= static_cast<uint32_t>(d)) upto += v;
    }
    *total = __shfl_sync(kFull, upto, 31);
    return upto - mine;
}

// The selected coordinates of a warp's range are few and scattered: serving each where it is
// found would leave 31 lanes idle.  Instead the warp queues them, in coordinate order, as
// row elements in a ring in shared memory and serves them 32 at a time, one per lane.
constexpr uint32_t kXRing = 1024;   // entries; a warp tile adds at most 512, a round removes 32

// appends the lane's selected coordinates of the warp's tile number t_rel (counted from the first
// tile of the warp's range); an entry is the coordinate's row element counted from the first
// element of that range.  sel4: a nibble per byte, one byte per group.
__device__ __forceinline__ uint32_t ring_append(uint32_t *ring, uint32_t tail, uint32_t sel4, uint32_t t_rel)
{
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t total = 0;
    uint32_t pos = tail + warp_exclusive_scan(__popc(sel4), &total);
    const uint32_t elem0 = 4u * (t_rel * kWarpTileGroups + 4u * lane);
    for (uint32_t left = sel4; left; left &= left - 1u, ++pos) {
        const uint32_t bit = static_cast<uint32_t>(__ffs(left) - 1);   // byte q = bit / 8, coordinate c = bit % 8
        ring[pos % kXRing] = elem0 + 4u * (bit >> 3) + (bit & 7u);
    }
    __syncwarp();
    return tail + total;
}

}  // namespace wash
