// Translation unit of the shared-memory-staged streaming shuffles (bulk copies; cp.async).
#include "wash_shuffle_tma.cuh"
#include "wash_shuffle_async.cuh"

namespace wash {

cudaError_t launch_shuffle_staged(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                  cudaStream_t stream, bool *supported)
{
    return launch_shuffle_tma(args, a_dtype, b_dtype, shape, stream, supported);
}

cudaError_t launch_shuffle_async_staged(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                        cudaStream_t stream, bool *supported)
{
    return launch_shuffle_async<true>(args, a_dtype, b_dtype, shape, stream, supported);
}

// sparse mode: the same kernel without the up-front copies
cudaError_t launch_shuffle_sparse(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                  cudaStream_t stream, bool *supported)
{
    return launch_shuffle_async<false>(args, a_dtype, b_dtype, shape, stream, supported);
}

}  // namespace wash
