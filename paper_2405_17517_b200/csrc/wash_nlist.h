// Population sizes with fully unrolled (register-resident) kernels.  Other sizes up to
// WASH_MAX_N run the run-time-N kernels.  The build compiles wash_inst.cu once per
// entry (-DWASH_N=<n>) and once with -DWASH_N=0 for the run-time-N kernels.
#pragma once
#define WASH_N_LIST(X) X(2) X(3) X(4) X(5) X(6) X(8) X(10) X(12) X(16) X(20) X(24) X(32)
