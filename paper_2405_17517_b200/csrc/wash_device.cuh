// Device-side building blocks: Philox4x32-10, element types, segment lookup.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "wash_internal.h"

namespace wash {

// ---- Philox4x32-10 (Salmon et al., SC'11) ------------------------------------------
// Ten rounds of two 32x32->64 multiplies; the key advances by the two Weyl constants
// after every round (the ten keys come ready-made from the host: PhiloxKeys).
struct Philox4 {
    uint32_t x, y, z, w;
};

__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys &keys)
{
    constexpr uint32_t kMul0 = 0xD2511F53u, kMul1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(kMul0, c0), lo0 = kMul0 * c0;
        const uint32_t hi1 = __umulhi(kMul1, c2), lo1 = kMul1 * c2;
        c0 = hi1 ^ c1 ^ keys.k[2 * r];
        c2 = hi0 ^ c3 ^ keys.k[2 * r + 1];
        c1 = lo1;
        c3 = lo0;
    }
    return Philox4{c0, c1, c2, c3};
}

// ---- element types -------------------------------------------------------------------
// A "group" is 4 consecutive elements: 16 bytes of fp32, 8 bytes of bf16.  Values are
// carried as raw bits (uint32 per element, bf16 in the low half).
struct F32 {
    using vec = uint4;
    static constexpr int kBytes = 4;
    static constexpr int kCode = kDtypeF32;
    static __device__ __forceinline__ vec load_group(const void *p)
    {
        vec v;
        asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
        return v;
    }
    static __device__ __forceinline__ void store_group(void *p, vec v) { *reinterpret_cast<vec *>(p) = v; }
    static __device__ __forceinline__ uint32_t get(const vec &v, int c)
    {
        return c == 0 ? v.x : c == 1 ? v.y : c == 2 ? v.z : v.w;
    }
    static __device__ __forceinline__ vec pack(uint32_t a, uint32_t b, uint32_t c, uint32_t d) { return make_uint4(a, b, c, d); }
    static __device__ __forceinline__ uint32_t load_elem(const void *base, long long idx) { return reinterpret_cast<const uint32_t *>(base)[idx]; }
    static __device__ __forceinline__ void store_elem(void *base, long long idx, uint32_t bits) { reinterpret_cast<uint32_t *>(base)[idx] = bits; }
    static __device__ __forceinline__ float to_float(uint32_t bits) { return __uint_as_float(bits); }
    static __device__ __forceinline__ uint32_t from_float(float f) { return __float_as_uint(f); }
    static __device__ __forceinline__ vec pack_floats(float a, float b, float c, float d)
    {
        return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
    }
};

struct BF16 {
    using vec = uint2;
    static constexpr int kBytes = 2;
    static constexpr int kCode = kDtypeBF16;
    static __device__ __forceinline__ vec load_group(const void *p)
    {
        vec v;
        asm volatile("ld.global.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
        return v;
    }
    static __device__ __forceinline__ void store_group(void *p, vec v) { *reinterpret_cast<vec *>(p) = v; }
    static __device__ __forceinline__ uint32_t get(const vec &v, int c)
    {
        return c == 0 ? (v.x & 0xFFFFu) : c == 1 ? (v.x >> 16) : c == 2 ? (v.y & 0xFFFFu) : (v.y >> 16);
    }
    static __device__ __forceinline__ vec pack(uint32_t a, uint32_t b, uint32_t c, uint32_t d) { return make_uint2(a | (b << 16), c | (d << 16)); }
    static __device__ __forceinline__ uint32_t load_elem(const void *base, long long idx) { return reinterpret_cast<const uint16_t *>(base)[idx]; }
    static __device__ __forceinline__ void store_elem(void *base, long long idx, uint32_t bits) { reinterpret_cast<uint16_t *>(base)[idx] = static_cast<uint16_t>(bits); }
    static __device__ __forceinline__ float to_float(uint32_t bits) { return __uint_as_float(bits << 16); }
    // round to nearest, ties to even; a NaN stays a quiet NaN
    static __device__ __forceinline__ uint32_t from_float(float f)
    {
        uint32_t u = __float_as_uint(f);
        if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x0040u;
        u += 0x7FFFu + ((u >> 16) & 1u);
        return u >> 16;
    }
    // Two values per conversion instruction (round to nearest even, as from_float); the
    // instruction turns every NaN into one canonical pattern, so the rare pair with a NaN
    // is redone by from_float, which keeps sign and payload.
    static __device__ __forceinline__ uint32_t pair_from_floats(float lo, float hi)
    {
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        if (lo != lo || hi != hi) r = from_float(lo) | (from_float(hi) << 16);
        return r;
    }
    static __device__ __forceinline__ vec pack_floats(float a, float b, float c, float d)
    {
        return make_uint2(pair_from_floats(a, b), pair_from_floats(c, d));
    }
};

struct NoStack {   // placeholder for "no second stack"
    using vec = uint32_t;
    static constexpr int kBytes = 0;
    static constexpr int kCode = kDtypeNone;
};

// ---- addressing ----------------------------------------------------------------------
// element index of (model n, row element e)
template <int LAYOUT>
__device__ __forceinline__ long long elem_index(const PopView &pop, int n, long long e)
{
    return LAYOUT == kLayoutNP ? static_cast<long long>(n) * pop.padded_P + e
                               : e * static_cast<long long>(pop.N) + n;
}

// Byte address of the j-th vector of group g.  [N][P]: vector j is model j's group.
// [P][N]: the group's 4N elements are contiguous and vector j is elements 4j..4j+3.
template <class T, int LAYOUT>
__device__ __forceinline__ char *group_vec_ptr(void *base, const PopView &pop, uint64_t g, int j)
{
    const long long e = LAYOUT == kLayoutNP ? static_cast<long long>(j) * pop.padded_P + 4ll * static_cast<long long>(g)
                                            : 4ll * static_cast<long long>(g) * pop.N + 4ll * j;
    return static_cast<char *>(base) + e * T::kBytes;
}

// raw bits of (model n, coordinate c of the group) out of the group's N vectors
template <class T, int LAYOUT, int CAP>
__device__ __forceinline__ uint32_t group_value(const typename T::vec (&v)[CAP], int n_models, int n, int c)
{
    if (LAYOUT == kLayoutNP) return T::get(v[n], c);
    const int f = c * n_models + n;
    return T::get(v[f >> 2], f & 3);
}

// ---- statistics -----------------------------------------------------------------------
// Called by every thread of the block at the end of a shuffle kernel.  Warp sums go to
// shared memory and a block that selected anything adds its sums to slot (blockIdx mod
// kStatSlots).  flush_stats_kernel, launched right after the shuffle, moves the slots'
// totals into the caller's counters and zeroes the slots.
__device__ __forceinline__ void publish_block_stats(unsigned long long *stats, StatSlot *slots, uint32_t selected, uint32_t moved)
{
    if (!stats) return;
    if (!__syncthreads_or(selected != 0)) return;   // most blocks have nothing to report at small p
    __shared__ uint32_t block_sum[2];
    if (threadIdx.x == 0) block_sum[0] = block_sum[1] = 0;
    __syncthreads();
    selected = __reduce_add_sync(0xFFFFFFFFu, selected);
    moved = __reduce_add_sync(0xFFFFFFFFu, moved);
    if ((threadIdx.x & 31) == 0 && selected) {
        atomicAdd(&block_sum[0], selected);
        atomicAdd(&block_sum[1], moved);
    }
    __syncthreads();
    if (threadIdx.x != 0 || block_sum[0] == 0) return;
    unsigned long long *dst = slots ? &slots[blockIdx.x % kStatSlots].selected : stats;   // {selected, moved} are adjacent in both
    atomicAdd(dst, static_cast<unsigned long long>(block_sum[0]));
    atomicAdd(dst + 1, static_cast<unsigned long long>(block_sum[1]));
}

// ---- which segment does group g belong to ---------------------------------------------
struct GroupInfo {
    uint32_t tensor_id;
    uint32_t cgroup;      // index of the group within its tensor (coordinate / 4)
    int valid;            // coordinates of this group that exist (0..4)
    uint64_t thr;
    uint32_t seg;         // index of the group's segment in the table
};

// Describes group g given its segment's table entry (two 16-byte halves).
__device__ __forceinline__ GroupInfo group_info(uint4 lo, uint4 hi, uint32_t g, uint32_t seg, uint32_t *status);

__device__ __forceinline__ GroupInfo find_group(const PopView &pop, uint32_t g, uint32_t *status)
{
    uint32_t s = __ldg(pop.tile_first + (g >> kTileShift));
    const uint32_t last = static_cast<uint32_t>(pop.n_seg) - 1u;
    while (s < last && g >= __ldg(&pop.seg[s].group_end)) ++s;
    const uint4 lo = __ldg(reinterpret_cast<const uint4 *>(pop.seg + s));       // begin, end, tensor, cgroup_begin
    const uint4 hi = __ldg(reinterpret_cast<const uint4 *>(pop.seg + s) + 1);   // numel, -, thr
    return group_info(lo, hi, g, s, status);
}

// As find_group, for a caller that visits groups in increasing order: `cursor` is the
// segment of the previous group (or any segment not after g's) and is advanced; `seg`
// may be a copy of the table in shared memory.
__device__ __forceinline__ GroupInfo find_group_forward(const SegEntry *seg, int n_seg, uint32_t &cursor, uint32_t g,
                                                        uint32_t *status)
{
    const uint32_t last = static_cast<uint32_t>(n_seg) - 1u;
    uint32_t s = cursor;
    while (s < last && g >= seg[s].group_end) ++s;
    cursor = s;
    const uint4 lo = reinterpret_cast<const uint4 *>(seg + s)[0];
    const uint4 hi = reinterpret_cast<const uint4 *>(seg + s)[1];
    return group_info(lo, hi, g, s, status);
}

__device__ __forceinline__ GroupInfo group_info(uint4 lo, uint4 hi, uint32_t g, uint32_t seg, uint32_t *status)
{
    GroupInfo gi;
    gi.seg = seg;
    if (g < lo.x || g >= lo.y) {   // table inconsistent with the row: report, touch nothing
        if (status) atomicOr(status, 1u);
        gi.tensor_id = 0; gi.cgroup = 0; gi.valid = 0; gi.thr = 0;
        return gi;
    }
    const uint32_t local = g - lo.x;
    const long long left = static_cast<long long>(hi.x) - 4ll * local;
    gi.tensor_id = lo.z;
    gi.cgroup = lo.w + local;
    gi.valid = left >= 4 ? 4 : (left > 0 ? static_cast<int>(left) : 0);
    gi.thr = static_cast<uint64_t>(hi.z) | (static_cast<uint64_t>(hi.w) << 32);
    return gi;
}

}  // namespace wash
