// Grid sizing for the grid-stride kernels: either one work item per thread (the block
// scheduler balances the SMs) or a persistent grid of SM count x resident blocks per SM.
// Each kernel family states the default that measured faster for it; wash_set_launch
// overrides (blocks_per_sm > 0: persistent with at most that many blocks per SM,
// < 0: one item per thread).
#pragma once
#include <cstdint>
#include <map>
#include <mutex>
#include <tuple>
#include <cuda_runtime.h>
#include "wash_internal.h"

namespace wash {

struct KernelFit {
    int occupancy;   // resident blocks per SM at (threads, smem)
};

inline cudaError_t kernel_fit(const void *kernel, int threads, size_t smem, KernelFit *fit)
{
    static std::mutex mu;
    static std::map<std::tuple<const void *, int, size_t, int>, KernelFit> cache;
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    const auto key = std::make_tuple(kernel, threads, smem, dev);
    {
        std::lock_guard<std::mutex> lock(mu);
        auto it = cache.find(key);
        if (it != cache.end()) { *fit = it->second; return cudaSuccess; }
    }
    if (smem > 32 * 1024) {   // static shared memory counts against the default 48 KiB too
        // raise the kernel's limit to the device's opt-in maximum (never lower it: other
        // launch shapes of the same kernel may already rely on a larger value)
        int optin = 0;
        err = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        if (err != cudaSuccess) return err;
        optin -= 1024;   // room for the kernels' few bytes of static shared memory
        if (optin < 0 || smem > static_cast<size_t>(optin)) return cudaErrorInvalidConfiguration;
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
        if (err != cudaSuccess) return err;
    }
    int occ = 0;
    err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, threads, smem);
    if (err != cudaSuccess) return err;
    KernelFit f{occ};
    {
        std::lock_guard<std::mutex> lock(mu);
        cache[key] = f;
    }
    *fit = f;
    return cudaSuccess;
}

// Launch `kernel(args)` over n_items work items, one item per thread per loop trip.
// smem_per_thread bytes of dynamic shared memory are given to every thread.
struct GridDefault {
    int threads;        // block size when the caller gave none
    bool persistent;    // grid style when the caller gave none
};

template <typename Args>
cudaError_t launch_grid_stride(void (*kernel)(Args), const Args &args, uint64_t n_items,
                               size_t smem_per_thread, const LaunchShape &shape, cudaStream_t stream,
                               GridDefault dflt = GridDefault{256, false})
{
    if (n_items == 0) return cudaSuccess;
    int threads = shape.threads > 0 ? shape.threads : dflt.threads;
    if (threads > 256) threads = 256;
    while (smem_per_thread * threads > 96 * 1024 && threads > 64) threads /= 2;
    const size_t smem = smem_per_thread * threads;
    KernelFit fit;
    cudaError_t err = kernel_fit(reinterpret_cast<const void *>(kernel), threads, smem, &fit);
    if (err != cudaSuccess) return err;
    if (fit.occupancy < 1) return cudaErrorLaunchOutOfResources;
    const uint64_t need = (n_items + threads - 1) / threads;
    uint64_t grid = need;
    const bool persistent = shape.blocks_per_sm > 0 || (shape.blocks_per_sm == 0 && dflt.persistent);
    if (persistent) {   // otherwise one trip per thread
        int bps = fit.occupancy;
        if (shape.blocks_per_sm > 0 && shape.blocks_per_sm < bps) bps = shape.blocks_per_sm;
        const uint64_t resident = static_cast<uint64_t>(shape.sm_count > 0 ? shape.sm_count : 148) * bps;
        if (grid > resident) grid = resident;
    }
    if (grid > 0x7FFFFFFFull) grid = 0x7FFFFFFFull;
    kernel<<<static_cast<unsigned>(grid), threads, smem, stream>>>(args);
    count_launch();
    return cudaGetLastError();
}

}  // namespace wash
