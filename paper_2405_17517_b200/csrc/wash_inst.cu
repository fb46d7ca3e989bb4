// One translation unit per population size for the dense operators (EMA, average, PAPA-all,
// consensus distance): compiled with -DWASH_N=<n> for every n of WASH_N_LIST (loops over the
// models unrolled) and with -DWASH_N=0 (run-time N, for the other population sizes).
#include "wash_reduce.cuh"

#ifndef WASH_N
#error "compile with -DWASH_N=<population size> (0 = run-time N)"
#endif

#define WASH_CAT2(a, b) a##b
#define WASH_CAT(a, b) WASH_CAT2(a, b)

namespace wash {

cudaError_t WASH_CAT(launch_reduce_n, WASH_N)(const ReduceArgs &args, int op, int dtype, int out_dtype,
                                              const LaunchShape &shape, cudaStream_t stream, bool *supported)
{
    return launch_reduce_n<WASH_N>(args, op, dtype, out_dtype, shape, stream, supported);
}

}  // namespace wash
