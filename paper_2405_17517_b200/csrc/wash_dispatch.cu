// Chooses the kernel instantiation for a population size.
#include <atomic>
#include "wash_internal.h"
#include "wash_device.cuh"
#include "wash_nlist.h"

namespace wash {

#define WASH_DECL(n) cudaError_t launch_reduce_n##n(const ReduceArgs &, int, int, int, const LaunchShape &, cudaStream_t, bool *);
WASH_N_LIST(WASH_DECL)
#undef WASH_DECL
cudaError_t launch_shuffle_sparse(const ShuffleArgs &, int, int, const LaunchShape &, cudaStream_t, bool *);
cudaError_t launch_shuffle_stream(const ShuffleArgs &, int, int, const LaunchShape &, cudaStream_t, bool *);
cudaError_t launch_shuffle_stream_loop(const ShuffleArgs &, int, int, const LaunchShape &, cudaStream_t, bool *);
cudaError_t launch_reduce_n0(const ReduceArgs &, int, int, int, const LaunchShape &, cudaStream_t, bool *);

static std::atomic<uint64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
uint64_t launch_count() { return g_launches.load(std::memory_order_relaxed); }

// Sums the partial statistics into the caller's counters and zeroes them again.
// (Warp shuffles, then eight partial sums: 64-bit atomics on one shared-memory word are
// compare-and-swap loops and cost this one-block kernel 20 us when 256 threads contended.)
__global__ void __launch_bounds__(kStatSlots) flush_stats_kernel(StatSlot *slots, unsigned long long *stats)
{
    __shared__ unsigned long long part[2][kStatSlots / 32];
    unsigned long long sel = slots[threadIdx.x].selected, mov = slots[threadIdx.x].moved;
    if (sel) {
        slots[threadIdx.x].selected = 0;
        slots[threadIdx.x].moved = 0;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sel += __shfl_down_sync(0xFFFFFFFFu, sel, d);
        mov += __shfl_down_sync(0xFFFFFFFFu, mov, d);
    }
    if ((threadIdx.x & 31) == 0) {
        part[0][threadIdx.x >> 5] = sel;
        part[1][threadIdx.x >> 5] = mov;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0, m = 0;
#pragma unroll
        for (int w = 0; w < kStatSlots / 32; ++w) {
            s += part[0][w];
            m += part[1][w];
        }
        if (s) {
            atomicAdd(stats, s);
            atomicAdd(stats + 1, m);
        }
    }
}

// Adds the kSqSlots partial copies of the [range][model] table of squared distances into the
// caller's array and leaves the slots zeroed for the next launch.
__global__ void __launch_bounds__(256) sq_flush_kernel(double *slots, int count, double *out)
{
    for (int j = threadIdx.x; j < count; j += blockDim.x) {
        double s = 0.0;
        for (int k = 0; k < kSqSlots; ++k) {
            s += slots[k * count + j];
            slots[k * count + j] = 0.0;
        }
        out[j] += s;
    }
}

cudaError_t launch_sq_flush(const SqArgs &sq, int N, double *out, cudaStream_t stream)
{
    sq_flush_kernel<<<1, 256, 0, stream>>>(sq.slots, sq.n_ranges * N, out);
    count_launch();
    return cudaGetLastError();
}

// Nothing but the mask's Philox blocks: four blocks per thread (four independent chains, as in the
// kernels that draw masks without touching memory), folded by XOR.  With one block per thread the
// same kernel measures a quarter less (3.17 against 4.2e11 blocks/s): the chains' latency shows.
__global__ void __launch_bounds__(256) philox_probe_kernel(unsigned long long n_blocks, const __grid_constant__ PhiloxKeys keys, uint32_t *checksum)
{
    const unsigned long long i = (static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x) * 4ull;
    uint32_t fold = 0;
    if (i + 3 < n_blocks) {   // the four chains under one condition, so that they interleave
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const Philox4 w = philox4x32_10(static_cast<uint32_t>(i + q), 0u, 0u, static_cast<uint32_t>((i + q) >> 32) << 8, keys);
            fold ^= w.x ^ w.y ^ w.z ^ w.w;
        }
    } else {
        for (int q = 0; q < 4 && i + q < n_blocks; ++q) {
            const Philox4 w = philox4x32_10(static_cast<uint32_t>(i + q), 0u, 0u, static_cast<uint32_t>((i + q) >> 32) << 8, keys);
            fold ^= w.x ^ w.y ^ w.z ^ w.w;
        }
    }
    fold = __reduce_xor_sync(0xFFFFFFFFu, fold);
    if (checksum && (threadIdx.x & 31) == 0 && fold == 0x9E3779B9u) atomicAdd(checksum, 1u);   // keeps the work alive; rarely true
}

cudaError_t launch_philox_probe(unsigned long long n_blocks, uint64_t seed, uint32_t *checksum, cudaStream_t stream)
{
    if (n_blocks == 0) return cudaSuccess;
    const unsigned long long grid = ((n_blocks + 3) / 4 + 255) / 256;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    philox_probe_kernel<<<static_cast<unsigned>(grid), 256, 0, stream>>>(n_blocks, philox_keys(seed), checksum);
    count_launch();
    return cudaGetLastError();
}

static cudaError_t launch_shuffle_kernel(const ShuffleArgs &args, int a_dtype, int b_dtype, int mode,
                                         const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    if (mode == kModeSparse) return launch_shuffle_sparse(args, a_dtype, b_dtype, shape, stream, supported);
    // Two streaming kernels.  A group of all models (both stacks) of at most kLoopMaxGroupBytes goes to the
    // resident-warp kernel, whose instruction count per group is a fraction of the one-trip kernel's, unless
    // most coordinates are expected to be served (there the one-trip kernel measured 6 % faster); larger
    // groups, the consensus statistic and the early flavour stay with the one-trip kernel.
    // blocks_per_sm of wash_set_launch: -4 forces the resident-warp kernel, -5 the one-trip kernel.
    const size_t elem_a = a_dtype == kDtypeF32 ? 4 : a_dtype == kDtypeBF16 ? 2 : 0, elem_b = b_dtype == kDtypeF32 ? 4 : b_dtype == kDtypeBF16 ? 2 : 0;
    const size_t per_group = static_cast<size_t>(args.pop.N) * 4 * (elem_a + elem_b);
    bool loop = per_group <= kLoopMaxGroupBytes && args.expected_share <= kLoopMaxShare;
    // 64-byte groups (fp32 N = 4, two fp32 stacks of N = 2, bf16 N = 8): only where serving weighs most
    if (per_group > kLoopMaxGroupBytes && per_group <= kLoopWideGroupBytes) loop = args.expected_share >= kLoopWideShareLo && args.expected_share <= kLoopWideShareHi;
    if (shape.blocks_per_sm == -4) loop = true;
    if (shape.blocks_per_sm == -5 || args.sq.slots || args.early) loop = false;
    if (loop) return launch_shuffle_stream_loop(args, a_dtype, b_dtype, shape, stream, supported);
    return launch_shuffle_stream(args, a_dtype, b_dtype, shape, stream, supported);
}

cudaError_t launch_shuffle(const ShuffleArgs &args, int a_dtype, int b_dtype, int mode,
                           const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    cudaError_t err = launch_shuffle_kernel(args, a_dtype, b_dtype, mode, shape, stream, supported);
    if (err != cudaSuccess || !*supported || !args.stats || !args.stat_slots) return err;
    flush_stats_kernel<<<1, kStatSlots, 0, stream>>>(args.stat_slots, args.stats);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_reduce(const ReduceArgs &args, int op, int dtype, int out_dtype,
                          const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    switch (args.pop.N) {
#define WASH_CASE(n) case n: return launch_reduce_n##n(args, op, dtype, out_dtype, shape, stream, supported);
        WASH_N_LIST(WASH_CASE)
#undef WASH_CASE
    default:
        return launch_reduce_n0(args, op, dtype, out_dtype, shape, stream, supported);
    }
}

}  // namespace wash
