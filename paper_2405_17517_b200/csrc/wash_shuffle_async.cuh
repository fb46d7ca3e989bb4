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
//   [N][P]: vector j of thread t at (j*T + t) * vec      (T = threads per block)
//   [P][N]: the block's T*4N elements are contiguous in global memory and are copied
//           as they lie, vector k*T + t by thread t; thread t's coordinate c of model n
//           is element (4t + c)*N + n of that image.
#pragma once
#include "wash_device.cuh"
#include "wash_launch.cuh"
#include "wash_shuffle_tma.cuh"   // draw_permutation_u8

namespace wash {

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

// Starts the copies of one stack for this thread's block position; returns nothing.
template <class T, int LAYOUT>
__device__ __forceinline__ void async_fetch(uint32_t image, void *base, const PopView &pop, uint64_t g_block,
                                            uint32_t groups_in_block, int n_models)
{
    constexpr int kVec = T::kBytes * 4;
    const uint32_t t = threadIdx.x, T_ = blockDim.x;
    if (LAYOUT == kLayoutNP) {
        if (t < groups_in_block) {
            // model j's vector of this thread's group: one row further in global memory,
            // one row of T vectors further in the image
            const char *src = group_vec_ptr<T, LAYOUT>(base, pop, g_block + t, 0);
            const size_t row_bytes = static_cast<size_t>(pop.padded_P) * T::kBytes;
            uint32_t dst = image + t * kVec;
            for (int j = 0; j < n_models; ++j, src += row_bytes, dst += T_ * kVec) cp_async<kVec>(dst, src);
        }
    } else {
        const uint32_t vecs = groups_in_block * n_models;
        const char *src = static_cast<const char *>(base) + 4ll * static_cast<long long>(g_block) * n_models * T::kBytes;
        for (uint32_t k = t; k < vecs; k += T_) cp_async<kVec>(image + k * kVec, src + static_cast<size_t>(k) * kVec);
    }
}

// raw bits of (model n, coordinate c) of this thread's group, out of the block image
template <class T, int LAYOUT>
__device__ __forceinline__ uint32_t image_value(const unsigned char *image, int n_models, int n, int c)
{
    const uint32_t t = threadIdx.x, T_ = blockDim.x;
    const uint32_t elem = LAYOUT == kLayoutNP ? (static_cast<uint32_t>(n) * T_ + t) * 4u + c
                                              : (4u * t + c) * n_models + n;
    if (T::kBytes == 4) return reinterpret_cast<const uint32_t *>(image)[elem];
    return reinterpret_cast<const uint16_t *>(image)[elem];
}

template <class TA, class TB, int LAYOUT>
__global__ void __launch_bounds__(256, 5) shuffle_async_kernel(const __grid_constant__ ShuffleArgs a)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const int n_models = a.pop.N;
    const uint32_t T_ = blockDim.x;
    unsigned char *image_a = smem_raw;
    unsigned char *image_b = image_a + static_cast<size_t>(n_models) * T_ * TA::kBytes * 4;
    uint8_t *s_perm = image_b + (kHasB ? static_cast<size_t>(n_models) * T_ * TB::kBytes * 4 : 0) + threadIdx.x;   // column [n][T]

    const uint64_t g_block = static_cast<uint64_t>(blockIdx.x) * T_;
    const uint32_t groups_in_block = static_cast<uint32_t>(min(static_cast<uint64_t>(T_), a.pop.n_groups - g_block));
    async_fetch<TA, LAYOUT>(smem_addr(image_a), a.a, a.pop, g_block, groups_in_block, n_models);
    if constexpr (kHasB) async_fetch<TB, LAYOUT>(smem_addr(image_b), a.b, a.pop, g_block, groups_in_block, n_models);

    uint32_t selected = 0, moved = 0, sel = 0;
    GroupInfo gi{0, 0, 0, 0};
    const uint64_t g = g_block + threadIdx.x;
    if (threadIdx.x < groups_in_block) {
        gi = find_group(a.pop, static_cast<uint32_t>(g), a.status);
        if (gi.thr != 0 && gi.valid != 0) {
            const Philox4 w = philox4x32_10(gi.cgroup, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
            sel |= (static_cast<uint64_t>(w.x) < gi.thr && gi.valid > 0) ? 1u : 0u;
            sel |= (static_cast<uint64_t>(w.y) < gi.thr && gi.valid > 1) ? 2u : 0u;
            sel |= (static_cast<uint64_t>(w.z) < gi.thr && gi.valid > 2) ? 4u : 0u;
            sel |= (static_cast<uint64_t>(w.w) < gi.thr && gi.valid > 3) ? 8u : 0u;
        }
    }
    // Every thread waits for its own copies (none may be in flight when the block ends).
    // In the [P][N] image a thread's values were copied by other threads, so a block with
    // a selected coordinate also needs a block-wide barrier before it reads the image.
    cp_async_wait_all();
    const bool block_has_work = LAYOUT == kLayoutPN ? (__syncthreads_or(sel != 0) != 0) : (sel != 0);
    if (block_has_work && sel != 0) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
            if (!((sel >> c) & 1u)) continue;
            draw_permutation_u8(s_perm, T_, n_models, 4u * gi.cgroup + c, gi.tensor_id, a.step_lo, a.step_hi8, a.key0, a.key1);
            const long long e = 4ll * static_cast<long long>(g) + c;
            for (int n = 0; n < n_models; ++n) {
                const int src = s_perm[n * T_];
                if (src == n) continue;
                TA::store_elem(a.a, elem_index<LAYOUT>(a.pop, n, e), image_value<TA, LAYOUT>(image_a, n_models, src, c));
                if constexpr (kHasB)
                    TB::store_elem(a.b, elem_index<LAYOUT>(a.pop, n, e), image_value<TB, LAYOUT>(image_b, n_models, src, c));
                ++moved;
            }
            ++selected;
        }
    }
    publish_block_stats(a.stats, a.stat_slots, selected, moved);
}

template <class TA, class TB>
cudaError_t launch_shuffle_async_typed(const ShuffleArgs &args, const LaunchShape &shape, cudaStream_t stream)
{
    constexpr bool kHasB = TB::kCode != kDtypeNone;
    const size_t per_thread = static_cast<size_t>(args.pop.N) * (TA::kBytes * 4 + (kHasB ? TB::kBytes * 4 : 0) + 1);
    // block size: as many threads as keep a block's image near 44 KiB, so that five blocks
    // (about 200 KiB in flight) share an SM
    int threads = shape.threads > 0 ? shape.threads : 64;   // measured: 64 beats 128 and 256 (a block holds its shared memory until its slowest thread is done)
    if (threads > 256) threads = 256;
    if (shape.threads <= 0)
        while (threads > 32 && per_thread * threads > 44 * 1024) threads >>= 1;
    const size_t smem = (per_thread * threads + 15) & ~static_cast<size_t>(15);
    auto kernel = args.pop.layout == kLayoutNP ? shuffle_async_kernel<TA, TB, kLayoutNP> : shuffle_async_kernel<TA, TB, kLayoutPN>;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), threads, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    const uint64_t grid = (static_cast<uint64_t>(args.pop.n_groups) + threads - 1) / threads;
    if (grid == 0) return cudaSuccess;
    if (grid > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
    kernel<<<static_cast<unsigned>(grid), threads, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
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

}  // namespace wash
