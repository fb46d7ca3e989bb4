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
    return launch_shuffle_async(args, a_dtype, b_dtype, shape, stream, supported);
}

}  // namespace wash
