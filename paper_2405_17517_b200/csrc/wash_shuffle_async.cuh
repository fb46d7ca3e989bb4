// Streaming shuffle with the stack staged through shared memory by per-thread
// asynchronous copies (cp.async, 16 or 8 bytes each).
//
// The register-resident kernel needs 4N (or 8N) registers per thread just to hold the
// loads in flight, which caps it at ~24 warps and ~120 KB in flight per SM.  Here a thread
// sends its group's N (or 2N) vectors straight from global to shared memory, draws the
// Philox mask while they travel, and only looks at them if one of its coordinates was
// selected.  Registers stay near 32, so the bytes in flight are bounded by shared memory
// (~200 KB per SM) instead.  Unlike bulk copies, cp.async goes through the ordinary
// load path and has no per-copy serialisation.  N is a run-time value.
//
// One group per thread, one trip per thread (the block scheduler refills the SM as
// blocks retire).  Block image in shared memory:
//   [N][P]: vector j of thread t at (j*T + t) * vec      (T = threads per block); fp32 vectors
//           are copied by their own thread, bf16 vectors in 16-byte pairs by the two lanes that own them
//   [P][N]: the block's T*4N elements are contiguous in global memory and are copied
//           vector by vector, vector k*T + t by thread t; a group's 4N elements stay together
//           and, when N is even and the launch expects to serve many coordinates, are followed
//           by one vector of padding, so that a group spans an odd number of vectors and the
//           lanes of a warp (one group each) fall into different shared-memory banks (at small
//           p the image is hardly read and the padding would only cost bytes in flight):
//           thread t's coordinate c of model n is element t*pn_group_elems + c*N + n.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"
#include "wash_permutation.cuh"

namespace wash {

constexpr uint32_t kDenseMinSelected = 64;   // selected coordinates of a warp's 128 from which every lane serves its own group

template <int BYTES>
__device__ __forceinline__ void cp_async(uint32_t dst_smem, const void *src)
{
    if (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.wait_all;" ::: "memory");
}

// elements a group takes in the [P][N] image: its 4N values plus the launch's padding (0 or one vector)
__device__ __forceinline__ uint32_t pn_group_elems(int n_models, uint32_t pad)
{
    return 4u * static_cast<uint32_t>(n_models) + pad;
}

// Starts the copies of one stack for this thread's block position; returns nothing.
template <class T, int LAYOUT>
__device__ __forceinline__ void async_fetch(uint32_t image, void *base, const PopView &pop, uint64_t g_block,
                                            uint32_t groups_in_block, int n_models, uint32_t pn_pad)
{
    constexpr int kVec = T::kBytes * 4;
    const uint32_t t = threadIdx.x, T_ = blockDim.x;
    if (LAYOUT == kLayoutNP && kVec == 8) {
        // bf16: two neighbouring groups of a row are 16 contiguous bytes in global memory and in the
        // image.  The two lanes that own them share the work: lane 2k takes the even rows of the
        // pair's piece, lane 2k+1 the odd rows, each copy 16 bytes (the number of groups in a block
        // is even).  A warp's groups are thus copied by that warp's lanes alone.
        const uint32_t piece = t >> 1;
        if (2u * piece < groups_in_block) {
            const size_t row_bytes = static_cast<size_t>(pop.padded_P) * T::kBytes;
            const char *src = group_vec_ptr<T, LAYOUT>(base, pop, g_block, 0) + (t & 1u) * row_bytes + piece * 16;
            uint32_t dst = image + (t & 1u) * T_ * kVec + piece * 16;
            for (uint32_t j = t & 1u; j < static_cast<uint32_t>(n_models); j += 2, src += 2 * row_bytes, dst += 2 * T_ * kVec) cp_async<16>(dst, src);
        }
    } else if (LAYOUT == kLayoutNP) {
        if (t < groups_in_block) {
            // model j's vector of this thread's group: one row further in global memory,
            // one row of T vectors further in the image
            const char *src = group_vec_ptr<T, LAYOUT>(base, pop, g_block + t, 0);
            const size_t row_bytes = static_cast<size_t>(pop.padded_P) * T::kBytes;
            uint32_t dst = image + t * kVec;
#pragma unroll 4
            for (int j = 0; j < n_models; ++j, src += row_bytes, dst += T_ * kVec) cp_async<kVec>(dst, src);
        }
    } else {
        const uint32_t vecs = groups_in_block * n_models, N_ = static_cast<uint32_t>(n_models);
        if (pn_pad == 0) {   // the image is the block's bytes as they lie
            const char *src = static_cast<const char *>(base) + 4ll * static_cast<long long>(g_block) * n_models * T::kBytes;
            for (uint32_t k = t; k < vecs; k += T_) cp_async<kVec>(image + k * kVec, src + static_cast<size_t>(k) * kVec);
            return;
        }
        // vector k is vector j = k % N of group k / N; the pair is advanced without dividing again
        const uint32_t stride = pn_group_elems(n_models, pn_pad) / 4u, dq = T_ / N_, dr = T_ - dq * N_;
        const char *src = static_cast<const char *>(base) + 4ll * static_cast<long long>(g_block) * n_models * T::kBytes;
        uint32_t group = t / N_, j = t - group * N_;
        for (uint32_t k = t; k < vecs; k += T_) {
            cp_async<kVec>(image + (group * stride + j) * kVec, src + static_cast<size_t>(k) * kVec);
            group += dq;
            j += dr;
            if (j >= N_) { j -= N_; ++group; }
        }
    }
}

// raw bits of (model n, coordinate c) of the group of block thread t, out of the block image
template <class T, int LAYOUT>
__device__ __forceinline__ uint32_t image_value(const unsigned char *image, int n_models, uint32_t pn_pad, uint32_t t, int n, int c)
{
    const uint32_t T_ = blockDim.x;
    const uint32_t elem = LAYOUT == kLayoutNP ? (static_cast<uint32_t>(n) * T_ + t) * 4u + c
                                              : t * pn_group_elems(n_models, pn_pad) + static_cast<uint32_t>(c * n_models + n);
    if (T::kBytes == 4) return reinterpret_cast<const uint32_t *>(image)[elem];
    return reinterpret_cast<const uint16_t *>(image)[elem];
}

// Dense selection: every lane serves its own group.  It draws the permutations of its selected
// coordinates (identity for the others) and writes the group back as whole vectors -- model n's
// vector takes coordinate c from model pi_c(n) -- instead of one 4-byte store per moved value:
// no list, no dealing, a quarter of the store instructions, and full 16-byte pieces of a sector.
// An unselected coordinate of such a group is rewritten with the bits it already has.  PERM is
// uint32_t (N <= 8) or uint64_t (N <= 16); the caller has checked that the group is whole.
// The draw needs no data, the write needs the image: two halves, so that a kernel can draw while
// its copies are still in flight.
template <class PERM>
__device__ __forceinline__ void dense_draw(const ShuffleArgs &a, uint32_t sel, const GroupInfo &gi, PERM (&perm)[4],
                                           uint32_t &selected, uint32_t &moved)
{
    constexpr PERM kIdentity = static_cast<PERM>(0xFEDCBA9876543210ull), kOnes = static_cast<PERM>(0x1111111111111111ull);
    const int n_models = a.pop.N;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        perm[c] = kIdentity;
        if ((sel >> c) & 1u) {
            if (sizeof(PERM) == 4) perm[c] = static_cast<PERM>(draw_permutation_packed32(n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.keys));
            else perm[c] = static_cast<PERM>(draw_permutation_packed(n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.keys));
            // values that leave their model: the nibbles of pi that differ from the identity's
            PERM x = perm[c] ^ kIdentity;
            x = (x | (x >> 1) | (x >> 2) | (x >> 3)) & kOnes;
            moved += sizeof(PERM) == 4 ? __popc(static_cast<uint32_t>(x)) : __popcll(static_cast<uint64_t>(x));
            ++selected;
        }
    }
}

template <class TA, class TB, int LAYOUT, class PERM>
__device__ __forceinline__ void dense_write(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                            uint64_t g_block, PERM (&perm)[4])
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x, t = threadIdx.x;
    auto value_a = [&](uint32_t from) -> uint32_t {
        return TA::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_a)[from] : reinterpret_cast<const uint16_t *>(image_a)[from];
    };
    auto value_b = [&](uint32_t from) -> uint32_t {
        return TB::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_b)[from] : reinterpret_cast<const uint16_t *>(image_b)[from];
    };
    if (LAYOUT == kLayoutNP) {
        // model n's vector of the group: one row further in the stack per n
        char *out_a = group_vec_ptr<TA, LAYOUT>(a.a, a.pop, g_block + t, 0);
        char *out_b = kHasB ? group_vec_ptr<TB, LAYOUT>(a.b, a.pop, g_block + t, 0) : nullptr;
        const size_t row_a = static_cast<size_t>(a.pop.padded_P) * TA::kBytes, row_b = static_cast<size_t>(a.pop.padded_P) * TB::kBytes;
        const uint32_t img_step = T_ * 4u, img0 = t * 4u;
        for (int n = 0; n < n_models; ++n, out_a += row_a, out_b += row_b) {
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t from = (static_cast<uint32_t>(perm[c]) & 15u) * img_step + img0 + c;
                perm[c] >>= 4;
                wa[c] = value_a(from);
                if constexpr (kHasB) wb[c] = value_b(from);
            }
            TA::store_group(out_a, TA::pack(wa[0], wa[1], wa[2], wa[3]));
            if constexpr (kHasB) TB::store_group(out_b, TB::pack(wb[0], wb[1], wb[2], wb[3]));
        }
    } else {
        // the group's 4N elements are contiguous: element c*N + n is (coordinate c, model n)
        char *out_a = group_vec_ptr<TA, LAYOUT>(a.a, a.pop, g_block + t, 0);
        char *out_b = kHasB ? group_vec_ptr<TB, LAYOUT>(a.b, a.pop, g_block + t, 0) : nullptr;
        const uint32_t img0 = t * pn_group_elems(n_models, a.pn_pad);
        PERM rest = perm[0];
        uint32_t base = img0;   // image element of (coordinate c, model 0)
        int n = 0, c = 0;
        for (int j = 0; j < n_models; ++j) {
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t from = base + (static_cast<uint32_t>(rest) & 15u);
                rest >>= 4;
                wa[q] = value_a(from);
                if constexpr (kHasB) wb[q] = value_b(from);
                if (++n == n_models) {
                    n = 0;
                    ++c;
                    base += static_cast<uint32_t>(n_models);
                    rest = c == 1 ? perm[1] : (c == 2 ? perm[2] : perm[3]);
                }
            }
            TA::store_group(out_a + static_cast<size_t>(j) * (TA::kBytes * 4), TA::pack(wa[0], wa[1], wa[2], wa[3]));
            if constexpr (kHasB) TB::store_group(out_b + static_cast<size_t>(j) * (TB::kBytes * 4), TB::pack(wb[0], wb[1], wb[2], wb[3]));
        }
    }
}

// The same for N > 16, where a permutation does not fit a register: the four coordinates'
// permutations are four columns of bytes in shared memory (column c of the thread at
// s_perm + c*N*T, entry n at [n*T]) and their Fisher-Yates chains run side by side, so that the
// four Philox draws of a step overlap and a swap's shared-memory round trip hides behind the
// other three chains.
__device__ __forceinline__ void dense_bytes_draw(const ShuffleArgs &a, uint8_t *s_perm, uint32_t sel, uint32_t cgroup, uint32_t tensor_id)
{
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    const uint32_t col = static_cast<uint32_t>(n_models) * T_;   // bytes from one coordinate's column to the next
    for (int n = 0; n < n_models; ++n) {
#pragma unroll
        for (int c = 0; c < 4; ++c) s_perm[c * col + n * T_] = static_cast<uint8_t>(n);
    }
    Philox4 w[4];
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (!((sel >> c) & 1u)) continue;
            if ((m & 3) == 0) w[c] = philox4x32_10(4u * cgroup + c, tensor_id, a.step_lo, a.step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), a.keys);
            const uint32_t r = w[c].x;
            w[c].x = w[c].y; w[c].y = w[c].z; w[c].z = w[c].w;
            const uint32_t j = __umulhi(r, static_cast<uint32_t>(k + 1));
            uint8_t *column = s_perm + c * col;
            const uint8_t pk = column[k * T_], pj = column[j * T_];
            column[k * T_] = pj;
            column[j * T_] = pk;
        }
    }
}

// (an unselected coordinate adds nothing to the moved-values count: its column is the identity)
// Returns the number of values that moved.
template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ uint32_t dense_bytes_write(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                                          const uint8_t *s_perm, uint64_t g_block)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    uint32_t moved = 0;
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x, t = threadIdx.x;
    const uint32_t col = static_cast<uint32_t>(n_models) * T_;
    auto value_a = [&](uint32_t from) -> uint32_t {
        return TA::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_a)[from] : reinterpret_cast<const uint16_t *>(image_a)[from];
    };
    auto value_b = [&](uint32_t from) -> uint32_t {
        return TB::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_b)[from] : reinterpret_cast<const uint16_t *>(image_b)[from];
    };
    char *out_a = group_vec_ptr<TA, LAYOUT>(a.a, a.pop, g_block + t, 0);
    char *out_b = kHasB ? group_vec_ptr<TB, LAYOUT>(a.b, a.pop, g_block + t, 0) : nullptr;
    if (LAYOUT == kLayoutNP) {
        const size_t row_a = static_cast<size_t>(a.pop.padded_P) * TA::kBytes, row_b = static_cast<size_t>(a.pop.padded_P) * TB::kBytes;
        const uint32_t img_step = T_ * 4u, img0 = t * 4u;
        for (int n = 0; n < n_models; ++n, out_a += row_a, out_b += row_b) {
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t src = s_perm[c * col + n * T_];
                moved += src != static_cast<uint32_t>(n) ? 1u : 0u;
                const uint32_t from = src * img_step + img0 + c;
                wa[c] = value_a(from);
                if constexpr (kHasB) wb[c] = value_b(from);
            }
            TA::store_group(out_a, TA::pack(wa[0], wa[1], wa[2], wa[3]));
            if constexpr (kHasB) TB::store_group(out_b, TB::pack(wb[0], wb[1], wb[2], wb[3]));
        }
    } else {
        // the group's 4N elements are contiguous: element c*N + n is (coordinate c, model n)
        const uint32_t img0 = t * pn_group_elems(n_models, a.pn_pad);
        int n = 0, c = 0;
        for (int j = 0; j < n_models; ++j) {
            uint32_t wa[4], wb[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t src = s_perm[c * col + n * T_];
                moved += src != static_cast<uint32_t>(n) ? 1u : 0u;
                const uint32_t from = img0 + static_cast<uint32_t>(c * n_models) + src;
                wa[q] = value_a(from);
                if constexpr (kHasB) wb[q] = value_b(from);
                if (++n == n_models) { n = 0; ++c; }
            }
            TA::store_group(out_a + static_cast<size_t>(j) * (TA::kBytes * 4), TA::pack(wa[0], wa[1], wa[2], wa[3]));
            if constexpr (kHasB) TB::store_group(out_b + static_cast<size_t>(j) * (TB::kBytes * 4), TB::pack(wb[0], wb[1], wb[2], wb[3]));
        }
    }
    return moved;
}

// The moves of one selected coordinate (coordinate c of the group of block thread t_owner): model n
// takes the value of model pi(n), nibble n of `perm` (N <= 16) or byte n of the column s_perm.
template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ void move_coordinate(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                                const uint8_t *s_perm, uint64_t perm, uint32_t t_owner, uint32_t c, uint64_t g_block,
                                                uint32_t &moved)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    const long long e = 4ll * static_cast<long long>(g_block + t_owner) + c;
    // model n's value of this coordinate sits at out0 + n*out_step in the stack and at
    // element img0 + n*img_step of the image: no multiplication left inside the loop
    const long long out_step = LAYOUT == kLayoutNP ? a.pop.padded_P : 1;
    const long long out0 = LAYOUT == kLayoutNP ? e : e * n_models;
    const uint32_t img_step = LAYOUT == kLayoutNP ? T_ * 4u : 1u;
    const uint32_t img0 = LAYOUT == kLayoutNP ? t_owner * 4u + c : t_owner * pn_group_elems(n_models, a.pn_pad) + c * n_models;
    long long out = out0;
    uint64_t rest = perm;   // nibble n on top of the low end when model n's turn comes
    for (int n = 0; n < n_models; ++n, out += out_step, rest >>= 4) {
        const uint32_t src = n_models <= 16 ? static_cast<uint32_t>(rest) & 15u : static_cast<uint32_t>(s_perm[n * T_]);
        if (src == static_cast<uint32_t>(n)) continue;
        const uint32_t from = img0 + src * img_step;
        TA::store_elem(a.a, out, TA::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_a)[from]
                                                 : reinterpret_cast<const uint16_t *>(image_a)[from]);
        if constexpr (kHasB)
            TB::store_elem(a.b, out, TB::kBytes == 4 ? reinterpret_cast<const uint32_t *>(image_b)[from]
                                                     : reinterpret_cast<const uint16_t *>(image_b)[from]);
        ++moved;
    }
}

// Serving one tile of T groups (one group per thread), in two halves.  `plan_tile` needs no data:
// it decides how the warp serves the tile and draws permutations; `apply_tile` moves the values
// once the image has landed.  A kernel may run the first while its copies are still in flight.
//   dealt  the warp's selected coordinates are listed in shared memory and dealt out to the lanes
//          32 at a time: with a few selected coordinates per warp (p around 0.01-0.1) one round
//          serves them all, instead of one divergent pass per coordinate slot; the plan draws the
//          first round's permutations, later rounds draw theirs when they are served;
//   dense  half of the warp's coordinates or more selected (and every such group whole): dealing
//          would take two rounds or more, in each of which a lane draws one permutation and stores
//          4-byte values; every lane serving its own group costs less from there on.
// Both are called by all threads of the block.
struct TilePlan {
    uint32_t mode;      // kServeNothing / kServeDealt / kServeDense: the same on every lane of a warp
    uint32_t total;     // dealt: selected coordinates of the warp
    uint32_t entry;     // dealt: the lane's coordinate of the first round, owner lane * 4 + coordinate slot
    uint64_t perm[4];   // dense: the permutations of the lane's four coordinates; dealt: [0] is the entry's (N <= 16)
};
constexpr uint32_t kServeNothing = 0, kServeDealt = 1, kServeDense = 2;

__device__ __forceinline__ void plan_tile(const ShuffleArgs &a, uint8_t *s_list, uint8_t *s_perm, uint32_t sel, const GroupInfo &gi,
                                          TilePlan &pl, uint32_t &selected, uint32_t &moved)
{
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    const uint32_t lane = threadIdx.x & 31u;
    pl.mode = kServeNothing;
    if (!__any_sync(0xFFFFFFFFu, sel != 0)) return;   // most warps have nothing selected at small p
    const uint32_t mine = __popc(sel);
    const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (total >= kDenseMinSelected && __all_sync(0xFFFFFFFFu, sel == 0 || gi.valid == 4)) {
        pl.mode = kServeDense;
        if (sel) {
            if (n_models <= 16) dense_draw<uint64_t>(a, sel, gi, pl.perm, selected, moved);
            else {
                dense_bytes_draw(a, s_perm, sel, gi.cgroup, gi.tensor_id);
                selected += __popc(sel);
            }
        }
        return;
    }
    pl.mode = kServeDealt;
    pl.total = total;
    uint32_t upto = mine;   // inclusive prefix sum over the lanes
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, upto, d);
        if (lane >= static_cast<uint32_t>(d)) upto += v;
    }
    uint8_t *list = s_list + (threadIdx.x >> 5) * 128;   // entry = owner lane * 4 + coordinate slot
    uint32_t pos = upto - mine;
#pragma unroll
    for (int c = 0; c < 4; ++c)
        if ((sel >> c) & 1u) list[pos++] = static_cast<uint8_t>(lane * 4 + c);
    __syncwarp();
    const bool active = lane < total;
    pl.entry = active ? list[lane] : 0u;
    const uint32_t owner = pl.entry >> 2, c = pl.entry & 3u;
    const uint32_t cgroup = __shfl_sync(0xFFFFFFFFu, gi.cgroup, owner);
    const uint32_t tensor = __shfl_sync(0xFFFFFFFFu, gi.tensor_id, owner);
    if (active) {
        if (n_models <= 16) pl.perm[0] = draw_permutation_packed(n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        else draw_permutation_u8(s_perm, T_, n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        ++selected;
    }
}

template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ void apply_tile(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                           uint8_t *s_list, uint8_t *s_perm, uint64_t g_block, uint32_t sel, const GroupInfo &gi,
                                           TilePlan &pl, uint32_t &selected, uint32_t &moved)
{
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    const uint32_t lane = threadIdx.x & 31u, warp_base = threadIdx.x & ~31u;
    if (pl.mode == kServeNothing) return;
    if (pl.mode == kServeDense) {
        if (sel) {
            if (n_models <= 16) dense_write<TA, TB, LAYOUT, uint64_t>(a, image_a, image_b, g_block, pl.perm);
            else moved += dense_bytes_write<TA, TB, LAYOUT>(a, image_a, image_b, s_perm, g_block);
        }
        return;
    }
    if (lane < pl.total) move_coordinate<TA, TB, LAYOUT>(a, image_a, image_b, s_perm, pl.perm[0], warp_base + (pl.entry >> 2), pl.entry & 3u, g_block, moved);
    const uint8_t *list = s_list + (threadIdx.x >> 5) * 128;
    for (uint32_t first = 32; first < pl.total; first += 32) {   // further rounds: draw and move
        const bool active = first + lane < pl.total;
        const uint32_t entry = active ? list[first + lane] : 0u;
        const uint32_t owner = entry >> 2, c = entry & 3u;
        const uint32_t cgroup = __shfl_sync(0xFFFFFFFFu, gi.cgroup, owner);
        const uint32_t tensor = __shfl_sync(0xFFFFFFFFu, gi.tensor_id, owner);
        if (!active) continue;
        uint64_t perm = 0;
        if (n_models <= 16) perm = draw_permutation_packed(n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        else draw_permutation_u8(s_perm, T_, n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        move_coordinate<TA, TB, LAYOUT>(a, image_a, image_b, s_perm, perm, warp_base + owner, c, g_block, moved);
        ++selected;
    }
    __syncwarp();   // the warp's list is rewritten by the next tile
}

// ---- the lean flavour's serving: everything after the wait, in one piece --------------------
// (The early flavour splits the same work in two halves around the wait, see plan_tile.  The lean
// one is compiled for 48 registers so that as many blocks stay resident as the shared memory
// allows; it keeps a permutation in a 32-bit register where it can and serves N > 16 by dealing.)
template <class TA, class TB, int LAYOUT, class PERM>
__device__ __forceinline__ void serve_group_dense(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                                  uint64_t g_block, uint32_t sel, const GroupInfo &gi, uint32_t &selected, uint32_t &moved)
{
    PERM perm[4];
    dense_draw<PERM>(a, sel, gi, perm, selected, moved);
    dense_write<TA, TB, LAYOUT, PERM>(a, image_a, image_b, g_block, perm);
}

// One selected coordinate served by the whole warp: the permutation is drawn so that lane n ends up
// with pi(n), and lane n moves model n's value -- one load and one store per lane instead of N of
// each on a single lane.  N <= 32.  Called by all lanes with the same arguments.
//   N <= 8: every lane draws the packed permutation (one or two Philox blocks, the same instructions
//           on all lanes) and takes its nibble;
//   N > 8:  lane b draws block b of the coordinate's permutation stream (up to eight blocks side by
//           side instead of one after the other); the Fisher-Yates steps run on a permutation held
//           one entry per lane: step k hands lane k's and lane j's entries to each other.
template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ void serve_coordinate_by_warp(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                                         uint64_t g_block, uint32_t t_owner, uint32_t c, uint32_t cgroup, uint32_t tensor,
                                                         uint32_t &selected, uint32_t &moved)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int n_models = a.pop.N;
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t src;
    if (n_models <= 8) {
        const uint32_t perm = draw_permutation_packed32(n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        src = (perm >> (4u * (lane & 7u))) & 15u;
    } else {
        const Philox4 w = philox4x32_10(4u * cgroup + c, tensor, a.step_lo, a.step_hi8 | (1u + lane), a.keys);
        src = lane;
        int k = n_models - 1;
        for (uint32_t b = 0; k >= 1; ++b) {
            const uint32_t r[4] = {__shfl_sync(0xFFFFFFFFu, w.x, b), __shfl_sync(0xFFFFFFFFu, w.y, b),
                                   __shfl_sync(0xFFFFFFFFu, w.z, b), __shfl_sync(0xFFFFFFFFu, w.w, b)};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (k < 1) break;
                const uint32_t j = __umulhi(r[q], static_cast<uint32_t>(k + 1));
                const uint32_t at_k = __shfl_sync(0xFFFFFFFFu, src, k), at_j = __shfl_sync(0xFFFFFFFFu, src, j);
                src = lane == static_cast<uint32_t>(k) ? at_j : (lane == j ? at_k : src);
                --k;
            }
        }
    }
    if (lane == 0) ++selected;
    if (lane >= static_cast<uint32_t>(n_models) || src == lane) return;
    const long long e = 4ll * static_cast<long long>(g_block + t_owner) + c;
    const long long out = elem_index<LAYOUT>(a.pop, static_cast<int>(lane), e);
    TA::store_elem(a.a, out, image_value<TA, LAYOUT>(image_a, n_models, a.pn_pad, t_owner, static_cast<int>(src), static_cast<int>(c)));
    if constexpr (kHasB) TB::store_elem(a.b, out, image_value<TB, LAYOUT>(image_b, n_models, a.pn_pad, t_owner, static_cast<int>(src), static_cast<int>(c)));
    ++moved;
}

// A warp tile with very few selected coordinates (the usual case from p = 1e-3 to 1e-2): no list and
// no dealing, the warp serves them one after the other.  `few`: 1 for N <= 16 (two to four
// coordinates served this way measured 1-30 % slower than dealing them), more for larger
// populations, where a dealt coordinate costs a lane up to eight Philox blocks in a row, a
// permutation kept as bytes in shared memory and N loads and stores.
constexpr uint32_t kFewWide = 3;   // N = 32, 2^25 coordinates, p = 0.01: 0.877 ms with 1, 0.818 with 3, 0.820 with 5; p = 0.03: 1.19, 1.17, 1.22
template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ void serve_few(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                          uint64_t g_block, uint32_t sel, const GroupInfo &gi, uint32_t &selected, uint32_t &moved)
{
    const uint32_t warp_base = threadIdx.x & ~31u;
    for (uint32_t owners = __ballot_sync(0xFFFFFFFFu, sel != 0); owners; owners &= owners - 1u) {
        const uint32_t owner = __ffs(owners) - 1;
        const uint32_t cgroup = __shfl_sync(0xFFFFFFFFu, gi.cgroup, owner);
        const uint32_t tensor = __shfl_sync(0xFFFFFFFFu, gi.tensor_id, owner);
        for (uint32_t bits = __shfl_sync(0xFFFFFFFFu, sel, owner); bits; bits &= bits - 1u)
            serve_coordinate_by_warp<TA, TB, LAYOUT>(a, image_a, image_b, g_block, warp_base + owner, __ffs(bits) - 1, cgroup, tensor, selected, moved);
    }
}

template <class TA, class TB, int LAYOUT>
__device__ __forceinline__ void serve_tile(const ShuffleArgs &a, const unsigned char *image_a, const unsigned char *image_b,
                                           uint8_t *s_list, uint8_t *s_perm, uint64_t g_block,
                                           uint32_t sel, const GroupInfo &gi, uint32_t &selected, uint32_t &moved)
{
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    const uint32_t lane = threadIdx.x & 31u, warp_base = threadIdx.x & ~31u;
    if (!__any_sync(0xFFFFFFFFu, sel != 0)) return;   // most warps have nothing selected at small p
    const uint32_t mine = __popc(sel);
    const uint32_t total = __reduce_add_sync(0xFFFFFFFFu, mine);
    if (n_models <= 32 && total <= (n_models <= 16 ? 1u : kFewWide)) {
        serve_few<TA, TB, LAYOUT>(a, image_a, image_b, g_block, sel, gi, selected, moved);
        return;
    }
    if (n_models <= 16 && total >= kDenseMinSelected && __all_sync(0xFFFFFFFFu, sel == 0 || gi.valid == 4)) {
        if (sel) {
            if (n_models <= 8) serve_group_dense<TA, TB, LAYOUT, uint32_t>(a, image_a, image_b, g_block, sel, gi, selected, moved);
            else serve_group_dense<TA, TB, LAYOUT, uint64_t>(a, image_a, image_b, g_block, sel, gi, selected, moved);
        }
        return;
    }
    uint32_t upto = mine;   // inclusive prefix sum over the lanes
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, upto, d);
        if (lane >= static_cast<uint32_t>(d)) upto += v;
    }
    uint8_t *list = s_list + (threadIdx.x >> 5) * 128;   // entry = owner lane * 4 + coordinate slot
    uint32_t pos = upto - mine;
#pragma unroll
    for (int c = 0; c < 4; ++c)
        if ((sel >> c) & 1u) list[pos++] = static_cast<uint8_t>(lane * 4 + c);
    __syncwarp();
    for (uint32_t first = 0; first < total; first += 32) {
        const bool active = first + lane < total;
        const uint32_t entry = active ? list[first + lane] : 0u;
        const uint32_t owner = entry >> 2, c = entry & 3u;
        const uint32_t cgroup = __shfl_sync(0xFFFFFFFFu, gi.cgroup, owner);
        const uint32_t tensor = __shfl_sync(0xFFFFFFFFu, gi.tensor_id, owner);
        if (!active) continue;
        uint64_t perm = 0;
        if (n_models <= 16) perm = draw_permutation_packed(n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        else draw_permutation_u8(s_perm, T_, n_models, 4u * cgroup + c, tensor, a.step_lo, a.step_hi8, a.keys);
        move_coordinate<TA, TB, LAYOUT>(a, image_a, image_b, s_perm, perm, warp_base + owner, c, g_block, moved);
        ++selected;
    }
    __syncwarp();   // the warp's list is rewritten by the next tile
}

// the four values of model n in the group of block thread t, widened to binary32
template <class T, int LAYOUT>
__device__ __forceinline__ void image_group(const unsigned char *image, int n_models, uint32_t pn_pad, uint32_t t, int n, float (&x)[4])
{
    if (LAYOUT == kLayoutNP) {
        const typename T::vec v = reinterpret_cast<const typename T::vec *>(image)[static_cast<uint32_t>(n) * blockDim.x + t];
#pragma unroll
        for (int c = 0; c < 4; ++c) x[c] = T::to_float(T::get(v, c));
    } else {
#pragma unroll
        for (int c = 0; c < 4; ++c) x[c] = T::to_float(image_value<T, LAYOUT>(image, n_models, pn_pad, t, n, c));
    }
}

// Distance to the consensus (Eq. 2 / Eq. 5; Fig. 2 plots its square root averaged over models)
// of one tile, from the image the copies have already brought into shared memory: for the four
// coordinates of a lane's group the binary64 mean over the models, then per model the sum of the
// squared deviations, summed over the warp by a butterfly and added to one of kSqSlots partial
// copies of the [range][model] table.  The exchange preserves the quantity (Eq. 5), so the values
// before it serve.  Called by all threads of the block; `exists`: the thread has a group in this
// tile.  WHOLE: every lane of the warp has a whole group of one and the same range (the usual
// case, decided by the caller with one vote), so nothing is predicated per coordinate.
template <class T, int LAYOUT, bool WHOLE>
__device__ __forceinline__ void consensus_warp(const ShuffleArgs &a, const unsigned char *image, int valid, uint32_t r1,
                                               uint32_t r_lo, uint32_t r_hi)
{
    const int n_models = a.pop.N;
    const uint32_t lane = threadIdx.x & 31u;
    double mean[4] = {0.0, 0.0, 0.0, 0.0};
    if (WHOLE || r1) {
        float x[4];
        for (int n = 0; n < n_models; ++n) {
            image_group<T, LAYOUT>(image, n_models, a.pn_pad, threadIdx.x, n, x);
#pragma unroll
            for (int c = 0; c < 4; ++c) mean[c] += static_cast<double>(x[c]);
        }
        const double count = static_cast<double>(n_models);
#pragma unroll
        for (int c = 0; c < 4; ++c) {   // sum / N: the reciprocal's product, corrected by its remainder
            const double q = mean[c] * a.sq.inv_n;
            mean[c] = fma(fma(-q, count, mean[c]), a.sq.inv_n, q);
        }
    }
    const uint32_t slot = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) % kSqSlots;
    for (uint32_t r = r_lo; r <= r_hi; ++r) {   // one trip unless the warp's groups lie in several ranges
        double *table = a.sq.slots + (static_cast<size_t>(slot) * a.sq.n_ranges + (r - 1)) * n_models;
        double keep = 0.0;   // lane l keeps the warp's sum of model l (mod 32)
        for (int n = 0; n < n_models; ++n) {
            double s = 0.0;
            if (WHOLE || r1 == r) {
                float x[4];
                image_group<T, LAYOUT>(image, n_models, a.pn_pad, threadIdx.x, n, x);
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (WHOLE || c < valid) {   // padding beyond the tensor's end holds no coordinate
                        const double d = static_cast<double>(x[c]) - mean[c];
                        s = fma(d, d, s);
                    }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
            if (static_cast<uint32_t>(n & 31) == lane) keep = s;
            if ((n & 31) == 31 || n == n_models - 1) {
                const int n_lane = (n & ~31) + static_cast<int>(lane);
                if (n_lane <= n && keep != 0.0) atomicAdd(table + n_lane, keep);
                keep = 0.0;
            }
        }
    }
}

template <class T, int LAYOUT>
__device__ __forceinline__ void consensus_tile(const ShuffleArgs &a, const unsigned char *image, const GroupInfo &gi, bool exists)
{
    // this lane's range, counted from 1 (0: its group lies in none, or does not exist)
    uint32_t r1 = 0;
    if (exists && gi.valid > 0 && gi.seg >= a.sq.seg_bound[0] && gi.seg < a.sq.seg_bound[a.sq.n_ranges]) {
        r1 = 1;
        for (int k = 1; k < a.sq.n_ranges; ++k) r1 += gi.seg >= a.sq.seg_bound[k] ? 1u : 0u;
    }
    const uint32_t r_hi = __reduce_max_sync(0xFFFFFFFFu, r1);
    if (r_hi == 0) return;
    const uint32_t r_lo = __reduce_min_sync(0xFFFFFFFFu, r1 ? r1 : 0xFFFFFFFFu);
    if (__all_sync(0xFFFFFFFFu, r1 == r_hi && gi.valid == 4)) consensus_warp<T, LAYOUT, true>(a, image, 4, r1, r_hi, r_hi);
    else consensus_warp<T, LAYOUT, false>(a, image, exists ? gi.valid : 0, r1, r_lo, r_hi);
}

#ifndef WASH_SERVING_ONLY   // a translation unit that only wants the copy and serving helpers above
// G = tiles per block (one group per thread and tile).  Small populations move few bytes per
// group (N * 16 for fp32), so a thread takes G = 2 groups, T apart, to keep more bytes in
// flight per SM; the two Philox draws overlap as well.
// EARLY: the tile's serving is planned (permutations drawn) before the wait for the copies, so that
// the integer work of a launch that selects much hides behind the copies' flight instead of holding
// the block's shared memory after them; it keeps a plan in registers across the wait, which the
// lean flavour (48 registers, as many resident blocks as the shared memory allows) cannot afford.
template <class TA, class TB, int LAYOUT, int G, bool STAT, bool EARLY>
__global__ void __launch_bounds__(256, EARLY ? 3 : 5) shuffle_async_kernel(const __grid_constant__ ShuffleArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    // G pairs of images of the two stacks, then the warps' lists, then the permutation columns
    const size_t group_elems = LAYOUT == kLayoutPN ? pn_group_elems(n_models, a.pn_pad) : 4u * static_cast<size_t>(n_models);
    const size_t a_bytes = group_elems * T_ * TA::kBytes;
    const size_t b_bytes = kHasB ? group_elems * T_ * TB::kBytes : 0;
    uint8_t *s_list = smem_raw + G * (a_bytes + b_bytes);   // 128 bytes per warp and tile
    uint8_t *s_perm = s_list + G * 4 * T_ + threadIdx.x;    // four columns [c][n][T] of bytes, used when N > 16

    const uint64_t g_first = a.group_lo + static_cast<uint64_t>(blockIdx.x) * (T_ * G);
    uint32_t in_tile[G];   // groups of tile i that exist
#pragma unroll
    for (int i = 0; i < G; ++i) {
        const uint64_t g_block = g_first + static_cast<uint64_t>(i) * T_;
        in_tile[i] = g_block < a.group_hi ? static_cast<uint32_t>(min(static_cast<uint64_t>(T_), a.group_hi - g_block)) : 0u;
        if (in_tile[i] == 0) continue;
        unsigned char *image_a = smem_raw + i * (a_bytes + b_bytes);
        async_fetch<TA, LAYOUT>(smem_addr(image_a), a.a, a.pop, g_block, in_tile[i], n_models, a.pn_pad);
        if constexpr (kHasB) async_fetch<TB, LAYOUT>(smem_addr(image_a + a_bytes), a.b, a.pop, g_block, in_tile[i], n_models, a.pn_pad);
    }

    uint32_t selected = 0, moved = 0;
    uint32_t sel[G];
    GroupInfo gi[G];
#pragma unroll
    for (int i = 0; i < G; ++i) {
        sel[i] = 0;
        gi[i] = GroupInfo{0, 0, 0, 0};
        if (threadIdx.x < in_tile[i]) {
            gi[i] = find_group(a.pop, static_cast<uint32_t>(g_first + static_cast<uint64_t>(i) * T_ + threadIdx.x), a.status);
            if (gi[i].thr != 0 && gi[i].valid != 0) {
                // word < thr with thr in [0, 2^32]: a 32-bit compare; a threshold of 2^32 selects
                // whatever the word is, so the block is not drawn at all
                uint32_t m = 0xFu;
                if ((gi[i].thr >> 32) == 0) {
                    const Philox4 w = philox4x32_10(gi[i].cgroup, gi[i].tensor_id, a.step_lo, a.step_hi8, a.keys);
                    const uint32_t thr_lo = static_cast<uint32_t>(gi[i].thr);
                    m = (w.x < thr_lo ? 1u : 0u) | (w.y < thr_lo ? 2u : 0u) | (w.z < thr_lo ? 4u : 0u) | (w.w < thr_lo ? 8u : 0u);
                }
                sel[i] = m & ((1u << gi[i].valid) - 1u);   // coordinates beyond the tensor's end do not exist
            }
        }
    }
    // Every thread waits for its own copies (none may be in flight when the block ends).
    // A selected coordinate is served by whichever lane of the warp gets it, so the warp
    // must see each other's copies; in the [P][N] image a group's values were copied by
    // threads of other warps, so there a block-wide barrier is needed instead.
    constexpr bool kSharedCopies = LAYOUT == kLayoutPN;   // a group's bytes were copied by threads of other warps
    if constexpr (EARLY) {
        TilePlan plan[G];
#pragma unroll
        for (int i = 0; i < G; ++i) plan_tile(a, s_list + i * 4 * T_, s_perm, sel[i], gi[i], plan[i], selected, moved);
        cp_async_wait_all();
        if (kSharedCopies) __syncthreads();
        else __syncwarp();
#pragma unroll
        for (int i = 0; i < G; ++i) {
            const unsigned char *image_a = smem_raw + i * (a_bytes + b_bytes);
            apply_tile<TA, TB, LAYOUT>(a, image_a, image_a + a_bytes, s_list + i * 4 * T_, s_perm,
                                       g_first + static_cast<uint64_t>(i) * T_, sel[i], gi[i], plan[i], selected, moved);
        }
    } else {
        cp_async_wait_all();
        if (kSharedCopies) __syncthreads();
        else __syncwarp();
        if constexpr (STAT) {
#pragma unroll
            for (int i = 0; i < G; ++i)
                consensus_tile<TA, LAYOUT>(a, smem_raw + i * (a_bytes + b_bytes), gi[i], threadIdx.x < in_tile[i]);
        }
#pragma unroll
        for (int i = 0; i < G; ++i) {
            const unsigned char *image_a = smem_raw + i * (a_bytes + b_bytes);
            serve_tile<TA, TB, LAYOUT>(a, image_a, image_a + a_bytes, s_list, s_perm,
                                       g_first + static_cast<uint64_t>(i) * T_, sel[i], gi[i], selected, moved);
        }
    }
    publish_block_stats(a.stats, a.stat_slots, selected, moved);
}

template <class TA, class TB, int G>
cudaError_t launch_shuffle_async_tiles(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    // a group's values in both images (with the launch's padding per group and stack in [P][N])
    const size_t group_elems = 4 * static_cast<size_t>(args.pop.N) + (args.pop.layout == kLayoutPN ? args.pn_pad : 0);
    const size_t image = group_elems * (TA::kBytes + (kHasB ? TB::kBytes : 0));
    // images, the permutation columns of bytes (N > 16: one, four in the early flavour), the warps' lists
    const size_t per_thread = image * G + (args.pop.N > 16 ? (args.early ? 4 : 1) * args.pop.N : 0) + 4 * G;
    // block size: as many threads as keep a block's image near 44 KiB, so that five blocks
    // (about 200 KiB in flight) share an SM
    int threads = shape.threads > 0 ? shape.threads : 64;   // measured: 64 beats 128 and 256 (a block holds its shared memory until its slowest thread is done)
    if (threads > 256) threads = 256;
    if (shape.threads <= 0)
        while (threads > 32 && per_thread * threads > 44 * 1024) threads >>= 1;
    const size_t smem = (per_thread * threads + 15) & ~static_cast<size_t>(15);
    const bool np = args.pop.layout == kLayoutNP;
    constexpr bool kEarlyBuilt = G == 1;   // the early flavour exists for one group per thread (what large populations get)
    auto kernel = np ? shuffle_async_kernel<TA, TB, kLayoutNP, G, false, false> : shuffle_async_kernel<TA, TB, kLayoutPN, G, false, false>;
    if (args.sq.slots) kernel = np ? shuffle_async_kernel<TA, TB, kLayoutNP, G, true, false> : shuffle_async_kernel<TA, TB, kLayoutPN, G, true, false>;
    else if (args.early && kEarlyBuilt) kernel = np ? shuffle_async_kernel<TA, TB, kLayoutNP, 1, false, true> : shuffle_async_kernel<TA, TB, kLayoutPN, 1, false, true>;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), threads, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    const uint64_t per_block = static_cast<uint64_t>(threads) * G;
    const uint64_t grid = (static_cast<uint64_t>(args.group_hi - args.group_lo) + per_block - 1) / per_block;
    if (grid == 0) return cudaSuccess;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    kernel<<<static_cast<unsigned>(grid), threads, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

template <class TA, class TB>
cudaError_t launch_shuffle_async_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    // bytes a thread has in flight for one group: up to 64 (N = 2 .. 4 in fp32, one stack) it
    // takes two groups (measured on 2^27 coordinates, p = 1e-3: N = 4 0.84 -> 0.95 of the copy
    // bandwidth, N = 2 0.48 -> 0.56; four groups were slower than two for every N).
    // blocks_per_sm of wash_set_launch, when 1 or 2, overrides.
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const size_t per_group = static_cast<size_t>(args.pop.N) * (TA::kBytes * 4 + (kHasB ? TB::kBytes * 4 : 0));
    int tiles = per_group <= 64 ? 2 : 1;
    if (shape.blocks_per_sm == 1 || shape.blocks_per_sm == 2) tiles = shape.blocks_per_sm;
    if (tiles == 2) return launch_shuffle_async_tiles<TA, TB, 2>(args, shape, stream);
    return launch_shuffle_async_tiles<TA, TB, 1>(args, shape, stream);
}

inline cudaError_t launch_shuffle_async(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                        cudaStream_t stream, bool *supported)
{
    *supported = true;
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeNone) return launch_shuffle_async_typed<F32, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeNone) return launch_shuffle_async_typed<BF16, NoStack>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeF32) return launch_shuffle_async_typed<F32, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeF32) return launch_shuffle_async_typed<BF16, F32>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeBF16) return launch_shuffle_async_typed<BF16, BF16>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeBF16) return launch_shuffle_async_typed<F32, BF16>(args, shape, stream);
    *supported = false;
    return cudaSuccess;
}

#endif  // WASH_SERVING_ONLY

}  // namespace wash
