// Device evaluation of the activations f (Sec. 2).  activation<ACT, T>(x)
// returns f(x) as a binary32 value that the caller rounds to the storage type
// T.  The result must stay within 2 ulp of T from the exactly rounded value:
//   T = float    : evaluated in binary64 (errors far below a binary32 ulp);
//   T = bfloat16 : evaluated in binary32 (errors far below a bfloat16 ulp),
//                  in forms that keep RELATIVE accuracy in the tails, since
//                  bfloat16 has the exponent range of binary32.
#pragma once

#include <cuda_bf16.h>

#include "fewbit.h"

namespace fewbit {

// ---- binary64 evaluation (T = float) ---------------------------------------
template <int ACT>
__device__ __forceinline__ float act_f64(float xf) {
    const double x = static_cast<double>(xf);
    double r;
    if constexpr (ACT == FEWBIT_GELU) {
        r = 0.5 * x * erfc(-x * 0.70710678118654752440);
    } else if constexpr (ACT == FEWBIT_SILU) {
        const double e = exp(-fabs(x));
        r = (x >= 0.0 ? x : x * e) / (1.0 + e);
    } else if constexpr (ACT == FEWBIT_SIGMOID) {
        const double e = exp(-fabs(x));
        r = (x >= 0.0 ? 1.0 : e) / (1.0 + e);
    } else if constexpr (ACT == FEWBIT_TANH) {
        r = tanh(x);
    } else if constexpr (ACT == FEWBIT_ELU) {
        r = x > 0.0 ? x : expm1(x);
    } else if constexpr (ACT == FEWBIT_SOFTPLUS) {
        r = fmax(x, 0.0) + log1p(exp(-fabs(x)));
    } else {
        r = x > 0.0 ? x : 0.01 * x;
    }
    return static_cast<float>(r);
}

// ---- binary32 evaluation (T = bfloat16) ------------------------------------
template <int ACT>
__device__ __forceinline__ float act_f32(float x) {
    if constexpr (ACT == FEWBIT_GELU) {
        return 0.5f * x * erfcf(-x * 0.70710678f);
    } else if constexpr (ACT == FEWBIT_SILU) {
        const float e = expf(-fabsf(x));
        return (x >= 0.0f ? x : x * e) / (1.0f + e);
    } else if constexpr (ACT == FEWBIT_SIGMOID) {
        const float e = expf(-fabsf(x));
        return (x >= 0.0f ? 1.0f : e) / (1.0f + e);
    } else if constexpr (ACT == FEWBIT_TANH) {
        return tanhf(x);
    } else if constexpr (ACT == FEWBIT_ELU) {
        return x > 0.0f ? x : expm1f(x);
    } else if constexpr (ACT == FEWBIT_SOFTPLUS) {
        return fmaxf(x, 0.0f) + log1pf(expf(-fabsf(x)));
    } else {
        return x > 0.0f ? x : 0.01f * x;
    }
}

template <int ACT, typename T>
__device__ __forceinline__ float activation(float x) {
    if constexpr (sizeof(T) == 4) return act_f64<ACT>(x);
    else return act_f32<ACT>(x);
}

}  // namespace fewbit
