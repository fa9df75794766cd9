// Device evaluation of the activations f (Sec. 2).
//
// activation<ACT, T>(x) returns f(x) as a binary32 value that the caller
// rounds once (nearest-even) to the storage type T.  The rounded result must
// stay within 2 ulp of T from the correctly rounded value, over the whole
// input range -- including the tails, where f(x) is tiny but still a normal
// number of T (bfloat16 has the exponent range of binary32).
//
//   T = bfloat16 : binary32 arithmetic with hardware approximations (ex2, rcp,
//                  tanh: relative error <= 2^-11, far below the 2^-9 that
//                  one bfloat16 ulp allows).  Every form is written so that
//                  the small quantity is computed as a product, never as a
//                  difference of nearly equal numbers:
//                      e^{-|x|} and friends are produced as E * 2^64 (so that
//                      ex2.approx.ftz never flushes them) and the factor
//                      2^-64 is folded into the last fused multiply-add, whose
//                      IEEE gradual underflow gives correct subnormals.
//   T = half     : as bfloat16 where the hardware approximation is 2^-22 (ex2, rcp), with a
//                  tighter GELU fit (3.4e-5) and tanh / expm1 from ex2 and a short series near 0
//                  instead of tanh.approx (2^-11 is not enough for 11 significant bits).
//   T = float    : binary32 arithmetic built on an exponential good to ~0.7 ulp, with the
//                  rounding error of every step that would reach the result carried along as a
//                  second binary32 term (fused multiply-add residuals).  GELU against the
//                  binary64 erfc form over all 2^32 inputs: 96.7 % equal, 2.9 % off by 1 ulp,
//                  0.007 % by 2, none by more.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "fewbit.h"

namespace fewbit {

// ---- hardware approximations ------------------------------------------------
__device__ __forceinline__ float ex2_ftz(float a) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a)); return r; }
__device__ __forceinline__ float rcp_ftz(float a) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a)); return r; }
__device__ __forceinline__ float tanh_apx(float a) { float r; asm("tanh.approx.f32 %0, %1;" : "=f"(r) : "f"(a)); return r; }

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kScaleUp = 64.0f;                      // exponent offset S
constexpr float kScaleDown = 5.421010862427522e-20f;   // 2^-64
constexpr float kSeluScale = 1.0507009873554805f;       // lambda
constexpr float kSeluScaleAlpha = 1.7580993408473766f;  // lambda * alpha

// ---- packed binary32 pairs (sm_100: two FMAs per issued instruction) ----------
__device__ __forceinline__ float2 splat(float c) { return make_float2(c, c); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 relu2(float2 x) { return make_float2(fmaxf(x.x, 0.0f), fmaxf(x.y, 0.0f)); }
// |x| = 2 max(x,0) - x, exact
__device__ __forceinline__ float2 abs2_from_relu(float2 relu, float2 x) { return fma2(relu, splat(2.0f), make_float2(-x.x, -x.y)); }
__device__ __forceinline__ float2 ex2_2(float2 a) { return make_float2(ex2_ftz(a.x), ex2_ftz(a.y)); }
__device__ __forceinline__ float2 rcp_2(float2 a) { return make_float2(rcp_ftz(a.x), rcp_ftz(a.y)); }

// ---- binary32 evaluation for bfloat16 storage, two elements at a time ---------
template <int ACT>
__device__ __forceinline__ float2 act_bf16(float2 x) {
    if constexpr (ACT == FEWBIT_GELU) {
        // x Phi(x) = max(x,0) - t Phi(-t), t = |x|, and t Phi(-t) = 16 s 2^{L(s)} with
        // s = min(t, 16) / 16 (one saturating multiply) and L(s) = log2 Phi(-16 s) a degree-7
        // polynomial (fit_coefficients.py: relative error of the product 8.7e-4 up to t = 14.6, where
        // it leaves the bfloat16 range; bounded beyond -- a quarter of a bfloat16 ulp: over all 65 536
        // inputs 511 results are one ulp from the rounded exact value, none further; degree 8 had 227,
        // degree 6 would have 18 757).  One ex2 per element and no reciprocal.
        // The constant term carries log2(16) and the exponent offset S.
        const float2 relu = relu2(x);
        const float2 s = make_float2(__saturatef(fabsf(x.x) * 0.0625f), __saturatef(fabsf(x.y) * 0.0625f));
        float2 l = fma2(s, splat(-58.7093277f), splat(224.208511f));
        l = fma2(l, s, splat(-358.452332f));
        l = fma2(l, s, splat(315.201569f));
        l = fma2(l, s, splat(-170.588593f));
        l = fma2(l, s, splat(-122.484428f));
        l = fma2(l, s, splat(-18.2224369f));
        l = fma2(l, s, splat(-1.00125074f + 4.0f + kScaleUp));
        return fma2(mul2(s, ex2_2(l)), splat(-kScaleDown), relu);
    } else if constexpr (ACT == FEWBIT_SILU) {
        // x / (1 + e^{-x}) with e^{-x} carried as e^{-x} 2^-64 (finite down to x = -133, below the
        // last x whose result is a bfloat16 subnormal; flushed to 0 where 1 + e^{-x} = 1 anyway), so
        // that r = 2^64 sigmoid(x) is a normal number over that range.  sigmoid(x) = 2^-64 r is then
        // formed first: it may be a binary32 subnormal (x < -87), but keeps at least 9 more bits than
        // the bfloat16 product can hold, and a tiny x meets an exact 0.5.
        const float2 e = ex2_2(fma2(x, splat(-kLog2e), splat(-kScaleUp)));
        const float2 r = rcp_2(add2(e, splat(kScaleDown)));
        return mul2(x, mul2(r, splat(kScaleDown)));
    } else if constexpr (ACT == FEWBIT_SIGMOID) {
        // 1 / (1 + e^{-x}), same scaling: 2^-64 r
        const float2 e = ex2_2(fma2(x, splat(-kLog2e), splat(-kScaleUp)));
        const float2 r = rcp_2(add2(e, splat(kScaleDown)));
        return mul2(r, splat(kScaleDown));
    } else if constexpr (ACT == FEWBIT_TANH) {
        return make_float2(tanh_apx(x.x), tanh_apx(x.y));
    } else if constexpr (ACT == FEWBIT_ELU) {
        // e^x - 1 = 2u / (1 - u), u = tanh(x/2): no cancellation for x <= 0
        const float2 h = mul2(x, splat(0.5f));
        const float2 u = make_float2(tanh_apx(h.x), tanh_apx(h.y));
        const float2 m = mul2(add2(u, u), rcp_2(fma2(u, splat(-1.0f), splat(1.0f))));
        return make_float2(x.x > 0.0f ? x.x : m.x, x.y > 0.0f ? x.y : m.y);
    } else if constexpr (ACT == FEWBIT_SOFTPLUS) {
        // max(x,0) + log(1 + E), E = e^{-|x|}, and log(1 + E) = E h(E) with h(u) = log(1 + u) / u a
        // degree-5 polynomial on [0, 1] (fit_coefficients.py: relative error 8.4e-6): one ex2 per
        // element, no logarithm, and the relative accuracy of the small results (x << 0) comes for free.
        // E is carried scaled by 2^64 so that the product does not lose its low bits to underflow.
        const float2 relu = relu2(x);
        const float2 t = abs2_from_relu(relu, x);
        const float2 e = ex2_2(fma2(t, splat(-kLog2e), splat(kScaleUp)));
        const float2 es = mul2(e, splat(kScaleDown));                  // E; where it underflows h is its constant term
        float2 h = fma2(es, splat(-0.0238690935f), splat(0.101222135f));
        h = fma2(h, es, splat(-0.210048556f));
        h = fma2(h, es, splat(0.325206637f));
        h = fma2(h, es, splat(-0.499361366f));
        h = fma2(h, es, splat(0.999991596f));
        return fma2(mul2(e, h), splat(kScaleDown), relu);
    } else if constexpr (ACT == FEWBIT_LEAKY_RELU) {
        const float2 m = mul2(x, splat(0.01f));
        return make_float2(fmaxf(x.x, m.x), fmaxf(x.y, m.y));
    } else if constexpr (ACT == FEWBIT_RELU) {
        return relu2(x);
    } else {
        // SELU: lambda x for x > 0, lambda alpha (e^x - 1) otherwise; e^x - 1 = 2u / (1 - u), u = tanh(x/2)
        const float2 h = mul2(x, splat(0.5f));
        const float2 u = make_float2(tanh_apx(h.x), tanh_apx(h.y));
        const float2 m = mul2(mul2(add2(u, u), splat(kSeluScaleAlpha)), rcp_2(fma2(u, splat(-1.0f), splat(1.0f))));
        const float2 p = mul2(x, splat(kSeluScale));
        return make_float2(x.x > 0.0f ? p.x : m.x, x.y > 0.0f ? p.y : m.y);
    }
}

// ---- binary64 evaluation for binary32 storage --------------------------------
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
    } else if constexpr (ACT == FEWBIT_LEAKY_RELU) {
        r = x > 0.0 ? x : 0.01 * x;
    } else if constexpr (ACT == FEWBIT_RELU) {
        r = x > 0.0 ? x : 0.0;
    } else {
        r = 1.0507009873554804934193349852946 * (x > 0.0 ? x : 1.6732632423543772848170429916717 * expm1(x));
    }
    return static_cast<float>(r);
}

// ---- binary32 evaluation for binary32 storage, two elements at a time ---------
// Everything that must be accurate to a fraction of a binary32 ulp is built on one
// exponential with ~0.7 ulp error; the quotient E / (1 + E) is refined with the
// exact rounding error of the sum 1 + E, so the logistic function ends near 1 ulp.

// e^a = (1 + s) * 2^n for a <= 0 (a is clamped at -131, far below the last value that matters:
// every result that uses it has reached its limit in binary32 by then).  Cody-Waite reduction by
// ln 2 in two pieces, degree-6 polynomial (fit in fit_coefficients.py: 0.05 ulp).  Returns s; *t
// holds 1.5 * 2^23 + n, i.e. the integer n in its low mantissa bits.
template <bool CLAMP = true>                 // CLAMP = false: the caller has already bounded a from below
__device__ __forceinline__ float2 exp_reduced_f32(float2 a, float2 *t_out) {
    if constexpr (CLAMP) a = make_float2(fmaxf(a.x, -131.0f), fmaxf(a.y, -131.0f));
    const float2 t = fma2(a, splat(kLog2e), splat(12582912.0f));
    const float2 n = add2(t, splat(-12582912.0f));
    float2 r = fma2(n, splat(-0.693145751953125f), a);                      // ln 2, high 12 bits
    r = fma2(n, splat(-1.428606765330187e-06f), r);                         // ln 2, the rest
    float2 q = fma2(r, splat(0.0013814608100801706f), splat(0.008368746377527714f));
    q = fma2(q, r, splat(0.04166838899254799f));
    q = fma2(q, r, splat(0.1666652113199234f));
    q = fma2(q, r, splat(0.4999999403953552f));
    *t_out = t;
    return fma2(mul2(r, r), q, r);                                           // e^r - 1
}

// 2^(n + bias - 127) from t = 1.5 * 2^23 + n, with integers
__device__ __forceinline__ float2 pow2_from_t(float2 t, uint32_t bias) {
    return make_float2(__uint_as_float((__float_as_uint(t.x) << 23) + (bias << 23)),
                       __uint_as_float((__float_as_uint(t.y) << 23) + (bias << 23)));
}

// E * 2^64 for E = e^a, a <= 0
__device__ __forceinline__ float2 exp_scaled_f32(float2 a) {
    float2 t;
    const float2 s = exp_reduced_f32(a, &t);
    return mul2(add2(s, splat(1.0f)), pow2_from_t(t, 127u + 64u));
}

// e^a - 1 for a <= 0:  2^n (1 + s) - 1 = 2^n s + (2^n - 1), and 2^n - 1 is exact.  The result is
// -1 in binary32 long before a = -80, where a is clamped so that 2^n stays a normal number.
__device__ __forceinline__ float2 expm1_nonpos_f32(float2 a) {
    a = make_float2(fmaxf(a.x, -80.0f), fmaxf(a.y, -80.0f));
    float2 t;
    const float2 s = exp_reduced_f32<false>(a, &t);
    const float2 p2 = pow2_from_t(t, 127u);
    return fma2(p2, s, add2(p2, splat(-1.0f)));
}

// -(E / (1 + E)) * 2^64 for E = e^{-|x|}: Newton-corrected quotient with the rounding error of
// 1 + E taken into account (Dh + Dl = 1 + E exactly).
__device__ __forceinline__ float2 neg_logistic_tail_scaled_f32(float2 x) {
    const float2 es = exp_scaled_f32(make_float2(-fabsf(x.x), -fabsf(x.y)));
    const float2 e = mul2(es, splat(kScaleDown));
    const float2 dh = add2(e, splat(1.0f));
    const float2 dl = fma2(add2(dh, splat(-1.0f)), splat(-1.0f), e);
    const float2 rn = make_float2(rcp_ftz(-dh.x), rcp_ftz(-dh.y));           // -1 / Dh
    const float2 qn = mul2(es, rn);                                          // -q0
    float2 res = fma2(dh, qn, es);                                           // E - Dh q0
    res = fma2(dl, qn, res);                                                 //   - Dl q0
    return fma2(res, rn, qn);                                                // -(q0 + res / Dh)
}

// GELU for binary32 storage in binary32 arithmetic, two elements at a time.
//   x Phi(x) = max(x,0) - T,   T = t Phi(-t) = t e^{-t^2/2} Q(t),   t = min(|x|, 15),
//   Q(t) = Phi(-t) e^{t^2/2} = w G(w),   w = 1/(1 + p t),   p = 0.2f,
// G a degree-9 polynomial in u = w - 1/2 (relative error 1e-8, fit_coefficients.py).  Beyond
// t = 14.6 the subtracted term is 0 in binary32.  Every step whose rounding error would reach the
// result carries its error term along:
//   * -t^2/2 = a + al exactly (fused multiply-add residual); al enters the reduced argument of e^r;
//   * 1 + p t = d + dl (the residual of one fused multiply-add).  The hardware reciprocal w0 of d
//     is used as it is: w0 = 1/(1 + p t0) exactly for a nearby t0 with t - t0 = -rho d / p,
//     rho = 1 - (d + dl) w0 (|rho| < 2^-22), and Q' = t Q - 1/sqrt(2 pi) gives the first-order step
//     from Q(t0) = w0 G(w0) to Q(t).  u = w0 - 1/2 is exact for w0 in [1/4, 1];
//   * the constant term of G is a two-piece constant;
//   * t w0 and its product with G are kept as value + residual, and the factor 1 + s of
//     e^{-t^2/2} = 2^n (1 + s) is applied with one fused multiply-add, so the binary32 product is
//     rounded once.
// The signs are arranged so that no negation is needed: tn = -t, wn = -w0 = rcp(-d), un = -u.
__device__ __forceinline__ float2 neg2(float2 a) { return make_float2(-a.x, -a.y); }
__device__ __forceinline__ float2 gelu_f32_pair(float2 x) {
    constexpr float kP = 0.2f;
    const float2 relu = relu2(x);
    const float2 t = make_float2(fminf(fabsf(x.x), 15.0f), fminf(fabsf(x.y), 15.0f));
    const float2 tn = make_float2(fmaxf(-fabsf(x.x), -15.0f), fmaxf(-fabsf(x.y), -15.0f));
    // a + al = -t^2/2 exactly
    const float2 c = mul2(t, splat(0.5f));
    const float2 b = mul2(c, t);
    const float2 a = neg2(b);
    const float2 al = fma2(c, tn, b);
    // e^a = 2^n (1 + s)
    const float2 tt = fma2(a, splat(kLog2e), splat(12582912.0f));
    const float2 n = add2(tt, splat(-12582912.0f));
    float2 r = fma2(n, splat(-0.693145751953125f), a);
    r = add2(r, fma2(n, splat(-1.428606765330187e-06f), al));
    float2 q = fma2(r, splat(0.0013814608100801706f), splat(0.008368746377527714f));
    q = fma2(q, r, splat(0.04166838899254799f));
    q = fma2(q, r, splat(0.1666652113199234f));
    q = fma2(q, r, splat(0.4999999403953552f));
    const float2 s = fma2(mul2(r, r), q, r);
    // d + dl = 1 + p t; wn = -w0 ~ -1/d; rho = 1 - (d + dl) w0
    const float2 d = fma2(t, splat(kP), splat(1.0f));
    const float2 dl = fma2(t, splat(kP), fma2(d, splat(-1.0f), splat(1.0f)));
    const float2 wn = make_float2(rcp_ftz(-d.x), rcp_ftz(-d.y));
    const float2 rho = fma2(dl, wn, fma2(d, wn, splat(1.0f)));
    // gh = G(w0) less the low piece of its constant term; Horner in un = -u
    const float2 un = add2(wn, splat(0.5f));
    float2 g = fma2(un, splat(0.0419610143f), splat(-0.0491418652f));
    g = fma2(g, un, splat(-0.0756255537f));
    g = fma2(g, un, splat(0.267188549f));
    g = fma2(g, un, splat(-0.442362875f));
    g = fma2(g, un, splat(0.528021038f));
    g = fma2(g, un, splat(-0.501653731f));
    g = fma2(g, un, splat(0.396245152f));
    g = fma2(g, un, splat(-0.266153008f));
    const float2 gh = fma2(g, un, splat(0.153838605f));
    // P + Pl = t w0 (gh + 5.85e-9)
    const float2 A = mul2(tn, wn);
    const float2 nA = neg2(A);
    const float2 P = mul2(A, gh);
    float2 Pl = fma2(A, gh, mul2(nA, gh));
    Pl = fma2(fma2(tn, wn, nA), gh, Pl);
    Pl = fma2(A, splat(5.8476104e-09f), Pl);
    // + t (t - t0) (t0 Q(t0) - 1/sqrt(2 pi)) = (rho d t) (1/sqrt(2 pi) - P) / p
    Pl = fma2(mul2(mul2(rho, d), t), fma2(P, splat(-4.99999993f), splat(1.99471137f)), Pl);
    // T = (P + Pl) (1 + s) 2^n
    Pl = fma2(s, Pl, Pl);
    const float2 T = add2(P, fma2(s, P, Pl));
    return fma2(mul2(T, pow2_from_t(tt, 127u + 64u)), splat(-kScaleDown), relu);
}

template <int ACT>
__device__ __forceinline__ float2 act_f32(float2 x) {
    if constexpr (ACT == FEWBIT_GELU) {
        return gelu_f32_pair(x);
    } else if constexpr (ACT == FEWBIT_SILU) {
        // x < 0: x q;  x >= 0: x - x q   with q = E / (1 + E)
        // below -131 the product is 0 in binary32; clamping there keeps |x| E from growing again
        // once E itself has been clamped
        const float2 xc = make_float2(fmaxf(x.x, -131.0f), fmaxf(x.y, -131.0f));
        const float2 u = mul2(xc, neg_logistic_tail_scaled_f32(xc));         // -x q 2^64
        const float2 c = make_float2(copysignf(kScaleDown, x.x), copysignf(kScaleDown, x.y));
        return fma2(u, make_float2(c.x, c.y), relu2(x));
    } else if constexpr (ACT == FEWBIT_SIGMOID) {
        // x < 0: q;  x >= 0: 1 - q
        const float2 qn = neg_logistic_tail_scaled_f32(x);
        const float2 step = make_float2(x.x >= 0.0f ? 1.0f : 0.0f, x.y >= 0.0f ? 1.0f : 0.0f);
        const float2 c = fma2(step, splat(2.0f * kScaleDown), splat(-kScaleDown));
        return fma2(qn, c, step);
    } else if constexpr (ACT == FEWBIT_TANH) {
        return make_float2(tanhf(x.x), tanhf(x.y));                          // library: <= 2 ulp
    } else if constexpr (ACT == FEWBIT_ELU) {
        const float2 m = expm1_nonpos_f32(make_float2(fminf(x.x, 0.0f), fminf(x.y, 0.0f)));
        return make_float2(x.x > 0.0f ? x.x : m.x, x.y > 0.0f ? x.y : m.y);
    } else if constexpr (ACT == FEWBIT_SOFTPLUS) {
        // max(x,0) + log(1 + E),  E = e^{-|x|} in (0, 1]:  log(1 + E) = 2 atanh(s),  s = E / (2 + E) <= 1/3.
        // The sum 2 + E is kept as d + dl (exact), the quotient gets one Newton step with the
        // residual E - (d + dl) s0, and atanh(s) = s + s^3 P(s^2) with P of degree 4 (1e-10).
        const float2 e = mul2(exp_scaled_f32(make_float2(-fabsf(x.x), -fabsf(x.y))), splat(kScaleDown));
        const float2 d = add2(e, splat(2.0f));
        const float2 nd = fma2(e, splat(-1.0f), splat(-2.0f));                  // -d
        const float2 ndl = fma2(e, splat(-1.0f), add2(d, splat(-2.0f)));        // -dl = (d - 2) - E
        const float2 rc = rcp_2(d);
        const float2 s0 = mul2(e, rc);
        const float2 res = fma2(ndl, s0, fma2(nd, s0, e));
        const float2 sq = fma2(res, rc, s0);
        const float2 z = mul2(sq, sq);
        float2 p = fma2(z, splat(0.12150468f), splat(0.10713829f));
        p = fma2(p, z, splat(0.14308442f));
        p = fma2(p, z, splat(0.19999439f));
        p = fma2(p, z, splat(0.33333337f));
        const float2 h = fma2(mul2(sq, z), p, sq);                               // atanh(s)
        return fma2(h, splat(2.0f), relu2(x));
    } else if constexpr (ACT == FEWBIT_LEAKY_RELU) {
        const float2 m = mul2(x, splat(0.01f));
        return make_float2(fmaxf(x.x, m.x), fmaxf(x.y, m.y));
    } else if constexpr (ACT == FEWBIT_RELU) {
        return relu2(x);
    } else if constexpr (ACT == FEWBIT_SELU) {
        const float2 m = mul2(expm1_nonpos_f32(make_float2(fminf(x.x, 0.0f), fminf(x.y, 0.0f))), splat(kSeluScaleAlpha));
        const float2 p = mul2(x, splat(kSeluScale));
        return make_float2(x.x > 0.0f ? p.x : m.x, x.y > 0.0f ? p.y : m.y);
    } else {
        return make_float2(act_f64<ACT>(x.x), act_f64<ACT>(x.y));
    }
}

// ---- binary32 evaluation for binary16 storage, two elements at a time ----------
template <int ACT>
__device__ __forceinline__ float2 act_f16(float2 x) {
    if constexpr (ACT == FEWBIT_GELU) {
        // as for bfloat16: t Phi(-t) = 6 s 2^{L(s)}, s = min(t, 6) / 6, L(s) = log2 Phi(-6 s) of degree 6
        // (relative error of the product 3.4e-5 up to t = 5.7; beyond, the product is below half the
        // smallest binary16 subnormal and stays there: 6 * 2^L(1) = 6e-9)
        const float2 relu = relu2(x);
        const float2 s = make_float2(__saturatef(fabsf(x.x) * 0.16666667f), __saturatef(fabsf(x.y) * 0.16666667f));
        float2 l = fma2(s, splat(1.16089976f), splat(-4.98774767f));
        l = fma2(l, s, splat(9.55984306f));
        l = fma2(l, s, splat(-11.1624165f));
        l = fma2(l, s, splat(-16.5841904f));
        l = fma2(l, s, splat(-6.90263224f));
        l = fma2(l, s, splat(-1.00004601f + 2.5849625f + kScaleUp));
        return fma2(mul2(s, ex2_2(l)), splat(-kScaleDown), relu);
    } else if constexpr (ACT == FEWBIT_TANH) {
        // |x| >= 1/32: 2 / (1 + E) - 1 with E = e^{-2x} for the signed x (E = inf gives -1, E = 0
        // gives 1; the difference keeps 2^-16 relative accuracy down to 1/32); below: x - x^3/3
        // (relative error 2 x^4 / 15 < 2e-7)
        const float2 e = ex2_2(mul2(x, splat(-2.0f * kLog2e)));
        const float2 big = fma2(rcp_2(add2(e, splat(1.0f))), splat(2.0f), splat(-1.0f));
        const float2 x2 = mul2(x, x);
        const float2 small = fma2(mul2(x2, x), splat(-0.33333334f), x);
        return make_float2(fabsf(x.x) < 0.03125f ? small.x : big.x, fabsf(x.y) < 0.03125f ? small.y : big.y);
    } else if constexpr (ACT == FEWBIT_ELU || ACT == FEWBIT_SELU) {
        // e^x - 1 for x <= 0 to binary16 accuracy: e^x - 1 by the hardware exponential below -1/32
        // (the difference keeps 2^-17 there), x (1 + x/2 + x^2/6) above (next term x^3/24: 1.3e-6)
        const float2 big = add2(ex2_2(mul2(x, splat(kLog2e))), splat(-1.0f));
        const float2 small = mul2(x, fma2(x, fma2(x, splat(0.16666667f), splat(0.5f)), splat(1.0f)));
        float2 m = make_float2(x.x < -0.03125f ? big.x : small.x, x.y < -0.03125f ? big.y : small.y);
        float2 p = x;
        if constexpr (ACT == FEWBIT_SELU) {
            m = mul2(m, splat(kSeluScaleAlpha));
            p = mul2(x, splat(kSeluScale));
        }
        return make_float2(x.x > 0.0f ? p.x : m.x, x.y > 0.0f ? p.y : m.y);
    } else {
        return act_bf16<ACT>(x);                    // ex2 / rcp forms: hardware error 2^-22
    }
}

// two neighbouring elements at once
template <int ACT, typename T>
__device__ __forceinline__ float2 activation2(float2 x) {
    if constexpr (sizeof(T) == 4) return act_f32<ACT>(x);
    else if constexpr (std::is_same<T, __half>::value) return act_f16<ACT>(x);
    else return act_bf16<ACT>(x);
}

template <int ACT, typename T>
__device__ __forceinline__ float activation(float x) { return activation2<ACT, T>(make_float2(x, x)).x; }

}  // namespace fewbit
