// Definitions shared by the translation units of the library (not installed).
#pragma once

#include <cstdint>

#include "fewbit.h"

#include <atomic>

namespace fewbit {
constexpr int kMaxBits = 4;
constexpr int kMaxLevels = 1 << kMaxBits;   // K <= 16

extern std::atomic<uint64_t> g_launches;     // kernels launched by the library in this process
extern thread_local int t_last_cuda_error;   // cudaError_t behind this thread's last FEWBIT_ERR_CUDA
}  // namespace fewbit

// The parameters s and y of Eq. 2, as binary32.  Unused boundary slots hold
// +inf (never below any x), unused level slots 0.
struct fewbit_table {
    fewbit_act act;
    int bits;
    double objective;                  // value of Eq. 3 reached by the solver
    float s[fewbit::kMaxLevels];       // s[0 .. K-2]
    float lev[fewbit::kMaxLevels];     // lev[0 .. K-1]
};
