// Instantiates the forward kernels of ONE activation (FEWBIT_ACT_ID, given on
// the compiler command line) so that the seven activations build in parallel.
#include "fewbit_fwd.cuh"

#ifndef FEWBIT_ACT_ID
#error "compile with -DFEWBIT_ACT_ID=<0..8>"
#endif

namespace fewbit {

#define FEWBIT_CAT2(a, b) a##b
#define FEWBIT_CAT(a, b) FEWBIT_CAT2(a, b)

const FwdLaunchers &FEWBIT_CAT(fwd_launchers_act, FEWBIT_ACT_ID)() {
    static const FwdLaunchers l = make_fwd_launchers<FEWBIT_ACT_ID>();
    return l;
}

}  // namespace fewbit
