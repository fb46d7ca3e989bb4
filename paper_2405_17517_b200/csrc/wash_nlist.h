// Population sizes whose dense operators (EMA, average, PAPA-all, consensus distance) are
// compiled with the loops over the models unrolled.  Other sizes up to WASH_MAX_N run the
// run-time-N instantiation.  The build compiles wash_inst.cu once per entry (-DWASH_N=<n>)
// and once with -DWASH_N=0.
#pragma once
#define WASH_N_LIST(X) X(2) X(3) X(4) X(5) X(6) X(8) X(10) X(12) X(16) X(20) X(24) X(32)
