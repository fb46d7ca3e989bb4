// The permutation pi_i of a selected coordinate: Fisher-Yates over the models, position
// k = N-1 .. 1 swapped with j = floor(word * (k+1) / 2^32), the words taken in order from the
// coordinate's Philox blocks (block b = words 4b .. 4b+3).  Three carriers of the same
// permutation: nibbles of a 32-bit register (N <= 8), nibbles of a 64-bit register (N <= 16),
// a column of bytes in shared memory (any N).
#pragma once
#include "wash_device.cuh"

namespace wash {

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// pi(n) in nibble n of the result, N <= 8: every shift is a 32-bit one
__device__ __forceinline__ uint32_t draw_permutation_packed32(int n_models, uint32_t i, uint32_t tensor, uint32_t step_lo,
                                                              uint32_t step_hi8, const PhiloxKeys &keys)
{
    uint32_t perm = 0x76543210u;
    Philox4 w{0, 0, 0, 0};
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
        if ((m & 3) == 0) w = philox4x32_10(i, tensor, step_lo, step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), keys);
        const uint32_t r = w.x;
        w.x = w.y; w.y = w.z; w.z = w.w;
        const uint32_t sk = 4u * k, sj = 4u * __umulhi(r, static_cast<uint32_t>(k + 1));
        const uint32_t diff = ((perm >> sk) ^ (perm >> sj)) & 15u;   // swap nibbles k and j
        perm ^= (diff << sk) | (diff << sj);
    }
    return perm;
}

// pi(n) in nibble n of the result, N <= 16
__device__ __forceinline__ uint64_t draw_permutation_packed(int n_models, uint32_t i, uint32_t tensor, uint32_t step_lo,
                                                            uint32_t step_hi8, const PhiloxKeys &keys)
{
    if (n_models <= 8) return 0xFEDCBA9800000000ull | draw_permutation_packed32(n_models, i, tensor, step_lo, step_hi8, keys);
    uint64_t perm = 0xFEDCBA9876543210ull;
    Philox4 w{0, 0, 0, 0};
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
        if ((m & 3) == 0) w = philox4x32_10(i, tensor, step_lo, step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), keys);
        const uint32_t r = w.x;
        w.x = w.y; w.y = w.z; w.z = w.w;
        const uint32_t sk = 4u * k, sj = 4u * __umulhi(r, static_cast<uint32_t>(k + 1));
        const uint64_t diff = ((perm >> sk) ^ (perm >> sj)) & 15ull;   // swap nibbles k and j
        perm ^= (diff << sk) | (diff << sj);
    }
    return perm;
}

// pi(n) in s_perm[n * stride], any N
static __device__ __noinline__ void draw_permutation_u8(uint8_t *s_perm, int stride, int n_models, uint32_t i,
                                                        uint32_t tensor, uint32_t step_lo, uint32_t step_hi8,
                                                        const PhiloxKeys &keys)
{
    for (int n = 0; n < n_models; ++n) s_perm[n * stride] = static_cast<uint8_t>(n);
    Philox4 w{0, 0, 0, 0};
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
        if ((m & 3) == 0) w = philox4x32_10(i, tensor, step_lo, step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), keys);
        const uint32_t r = w.x;
        w.x = w.y; w.y = w.z; w.z = w.w;
        const uint32_t j = __umulhi(r, static_cast<uint32_t>(k + 1));
        const uint8_t pk = s_perm[k * stride], pj = s_perm[j * stride];
        s_perm[k * stride] = pj;
        s_perm[j * stride] = pk;
    }
}

}  // namespace wash
