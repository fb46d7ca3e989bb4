// Translation unit of the resident-warp streaming shuffle (small groups).
#include "wash_shuffle_loop.cuh"

namespace wash {

cudaError_t launch_shuffle_stream_loop(const ShuffleArgs &args, int a_dtype, int b_dtype, const LaunchShape &shape,
                                       cudaStream_t stream, bool *supported)
{
    return launch_shuffle_loop(args, a_dtype, b_dtype, shape, stream, supported);
}

}  // namespace wash
