// The shuffling step (Eq. 3; Algorithm 1, "Shuffling step") as one grid-stride kernel.
//
// A thread owns one group of 4 neighbouring coordinates and, for them, all N models'
// values of one or two stacks.  Per group: one Philox block gives the 4 Bernoulli
// words; a selected coordinate draws its permutation (Fisher-Yates on further Philox
// words), and the N values move as new[n] = old[pi(n)].  Unselected coordinates are
// never written.
//
//   STREAM = true   every group's values are first loaded (coalesced 16-byte loads for
//                   fp32, 8-byte for bf16) and the exchange takes them from registers:
//                   one pass over the whole stack.
//   STREAM = false  the mask is drawn first and memory is touched only for selected
//                   coordinates (N is a run-time value here).
//
// No two threads touch the same coordinate, so the in-place exchange needs no
// synchronisation between threads.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"

namespace wash {

// pi for coordinate i of tensor `tensor`, left in the calling thread's column of
// shared memory: s_perm[n * ts], n = 0..N-1.  Fisher-Yates from the top index down,
// word m of the coordinate's permutation stream decides the swap of position N-1-m;
// j = floor(word * (k+1) / 2^32).
static __device__ __noinline__ void draw_permutation(uint32_t *s_perm, int ts, int n_models, uint32_t i,
                                              uint32_t tensor, uint32_t step_lo, uint32_t step_hi8,
                                              const PhiloxKeys &keys)
{
    for (int n = 0; n < n_models; ++n) s_perm[n * ts] = n;
    Philox4 w{0, 0, 0, 0};
    for (int k = n_models - 1, m = 0; k >= 1; --k, ++m) {
        if ((m & 3) == 0) w = philox4x32_10(i, tensor, step_lo, step_hi8 | (1u + (static_cast<uint32_t>(m) >> 2)), keys);
        const uint32_t r = w.x;
        w.x = w.y; w.y = w.z; w.z = w.w;
        const uint32_t j = __umulhi(r, static_cast<uint32_t>(k + 1));
        const uint32_t pk = s_perm[k * ts], pj = s_perm[j * ts];
        s_perm[k * ts] = pj;
        s_perm[j * ts] = pk;
    }
}

template <int N, class TA, class TB, int LAYOUT, bool STREAM>
__global__ void __launch_bounds__(256) shuffle_kernel(const __grid_constant__ ShuffleArgs a)
{
    extern __shared__ uint32_t smem[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    constexpr int kRegs = N > 0 ? N : 1;
    static_assert(!STREAM || N > 0, "the streaming kernel needs a compile-time N");
    const int ts = blockDim.x;
    const int n_models = N > 0 ? N : a.pop.N;
    uint32_t *s_perm = smem + threadIdx.x;                      // [n][ts]
    uint32_t *s_val = smem + n_models * ts + threadIdx.x;       // [n][ts]
    uint32_t selected = 0, moved = 0;
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t g = a.group_lo + static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; g < a.group_hi; g += stride) {
        typename TA::vec va[kRegs];
        typename TB::vec vb[kRegs];
        if constexpr (STREAM) {
#pragma unroll
            for (int j = 0; j < N; ++j) va[j] = TA::load_group(group_vec_ptr<TA, LAYOUT>(a.a, a.pop, g, j));
            if constexpr (kHasB) {
#pragma unroll
                for (int j = 0; j < N; ++j) vb[j] = TB::load_group(group_vec_ptr<TB, LAYOUT>(a.b, a.pop, g, j));
            }
        }
        const GroupInfo gi = find_group(a.pop, static_cast<uint32_t>(g), a.status);
        if (gi.thr == 0 || gi.valid == 0) continue;
        const Philox4 w = philox4x32_10(gi.cgroup, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
        uint32_t sel = 0;
        sel |= (static_cast<uint64_t>(w.x) < gi.thr && gi.valid > 0) ? 1u : 0u;
        sel |= (static_cast<uint64_t>(w.y) < gi.thr && gi.valid > 1) ? 2u : 0u;
        sel |= (static_cast<uint64_t>(w.z) < gi.thr && gi.valid > 2) ? 4u : 0u;
        sel |= (static_cast<uint64_t>(w.w) < gi.thr && gi.valid > 3) ? 8u : 0u;
        if (sel == 0) continue;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (!((sel >> c) & 1u)) continue;
            draw_permutation(s_perm, ts, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.keys);
            const long long e = 4ll * static_cast<long long>(g) + c;
            // first stack
            if constexpr (STREAM) {
#pragma unroll
                for (int n = 0; n < N; ++n) s_val[n * ts] = group_value<TA, LAYOUT, kRegs>(va, N, n, c);
            } else {
                for (int n = 0; n < n_models; ++n) s_val[n * ts] = TA::load_elem(a.a, elem_index<LAYOUT>(a.pop, n, e));
            }
            for (int n = 0; n < n_models; ++n) {
                const uint32_t src = s_perm[n * ts];
                if (src != static_cast<uint32_t>(n)) {
                    TA::store_elem(a.a, elem_index<LAYOUT>(a.pop, n, e), s_val[src * ts]);
                    ++moved;
                }
            }
            // second stack: same permutation
            if constexpr (kHasB) {
                if constexpr (STREAM) {
#pragma unroll
                    for (int n = 0; n < N; ++n) s_val[n * ts] = group_value<TB, LAYOUT, kRegs>(vb, N, n, c);
                } else {
                    for (int n = 0; n < n_models; ++n) s_val[n * ts] = TB::load_elem(a.b, elem_index<LAYOUT>(a.pop, n, e));
                }
                for (int n = 0; n < n_models; ++n) {
                    const uint32_t src = s_perm[n * ts];
                    if (src != static_cast<uint32_t>(n)) TB::store_elem(a.b, elem_index<LAYOUT>(a.pop, n, e), s_val[src * ts]);
                }
            }
            ++selected;
        }
    }
    publish_block_stats(a.stats, a.stat_slots, selected, moved);
}

template <int N, class TA, class TB, bool STREAM>
cudaError_t launch_shuffle_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    const size_t smem_per_thread = 2u * sizeof(uint32_t) * static_cast<size_t>(N > 0 ? N : args.pop.N);
    // 128-thread blocks in a persistent grid: with 80-200 registers per thread this keeps
    // the most warps resident and measured fastest on the ResNet-50 populations
    const GridDefault dflt{128, true};
    if (args.pop.layout == kLayoutNP)
        return launch_grid_stride(shuffle_kernel<N, TA, TB, kLayoutNP, STREAM>, args, args.group_hi - args.group_lo, smem_per_thread, shape, stream, dflt);
    return launch_grid_stride(shuffle_kernel<N, TA, TB, kLayoutPN, STREAM>, args, args.group_hi - args.group_lo, smem_per_thread, shape, stream, dflt);
}

// dtype dispatch: parameters fp32 or bf16; second stack absent, fp32 or bf16
template <int N, bool STREAM>
cudaError_t launch_shuffle_n(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                             cudaStream_t stream, bool *supported)
{
    *supported = true;
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeNone) return launch_shuffle_typed<N, F32, NoStack, STREAM>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeNone) return launch_shuffle_typed<N, BF16, NoStack, STREAM>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeF32) return launch_shuffle_typed<N, F32, F32, STREAM>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeF32) return launch_shuffle_typed<N, BF16, F32, STREAM>(args, shape, stream);
    if (a_dtype == kDtypeBF16 && b_dtype == kDtypeBF16) return launch_shuffle_typed<N, BF16, BF16, STREAM>(args, shape, stream);
    if (a_dtype == kDtypeF32 && b_dtype == kDtypeBF16) return launch_shuffle_typed<N, F32, BF16, STREAM>(args, shape, stream);
    *supported = false;
    return cudaSuccess;
}

}  // namespace wash
