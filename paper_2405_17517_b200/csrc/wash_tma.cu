// Translation unit of the shared-memory-staged streaming shuffles (bulk copies; cp.async) and of the sparse shuffle.
#include "wash_shuffle_tma.cuh"
#include "wash_shuffle_async.cuh"
#include "wash_shuffle_sparse.cuh"

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

// sparse mode: mask first, only selected coordinates touched (wash_shuffle_sparse.cuh)
cudaError_t launch_shuffle_sparse(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                  cudaStream_t stream, bool *supported)
{
    return launch_shuffle_sparse_tiles(args, a_dtype, b_dtype, shape, stream, supported);
}

}  // namespace wash
