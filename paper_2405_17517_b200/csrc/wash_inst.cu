// One translation unit per population size: compiled with -DWASH_N=<n> for every n of
// WASH_N_LIST (unrolled kernels) and with -DWASH_N=0 (run-time-N kernels, which include
// the reduce kernels for population sizes without an unrolled instantiation).
#include "wash_shuffle.cuh"
#include "wash_reduce.cuh"

#ifndef WASH_N
#error "compile with -DWASH_N=<population size> (0 = run-time N)"
#endif

#define WASH_CAT2(a, b) a##b
#define WASH_CAT(a, b) WASH_CAT2(a, b)

namespace wash {

#if WASH_N > 0
cudaError_t WASH_CAT(launch_shuffle_stream_n, WASH_N)(const ShuffleArgs &args, int a_dtype, int b_dtype,
                                                      const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    return launch_shuffle_n<WASH_N, true>(args, a_dtype, b_dtype, shape, stream, supported);
}
#endif

cudaError_t WASH_CAT(launch_reduce_n, WASH_N)(const ReduceArgs &args, int op, int dtype, int out_dtype,
                                              const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    return launch_reduce_n<WASH_N>(args, op, dtype, out_dtype, shape, stream, supported);
}

}  // namespace wash
