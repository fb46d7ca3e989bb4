// Translation unit of the two shuffle kernels: the streaming one (stack staged through shared
// memory by cp.async) and the sparse one (mask first, only selected coordinates touched).
#include "wash_shuffle_async.cuh"
#include "wash_shuffle_sparse.cuh"

namespace wash {

cudaError_t launch_shuffle_stream(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                  cudaStream_t stream, bool *supported)
{
    return launch_shuffle_async(args, a_dtype, b_dtype, shape, stream, supported);
}

cudaError_t launch_shuffle_sparse(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                  cudaStream_t stream, bool *supported)
{
    return launch_shuffle_sparse_tiles(args, a_dtype, b_dtype, shape, stream, supported);
}

}  // namespace wash
