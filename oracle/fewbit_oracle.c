/*
 * Few-Bit Backward -- reference oracle (TEST INFRASTRUCTURE, not the product).
 *
 * A plain, slow, single-threaded CPU statement of what the hot path computes,
 * written from the paper (arXiv 2202.00441) so that a reader can check it
 * against the equations by eye.  It shares no code with the CUDA library and
 * is only ever called from tests, the smoke check and the benchmark's CPU
 * baseline.  Everything floating point is binary64 unless the contract fixes
 * a narrower type (the fp32 compare in the bucketize step and the fp32
 * multiply in the backward step).
 *
 * Parts and the passage each follows:
 *   fbo_act / fbo_act_deriv   Sec. 2 (pointwise f, chain rule Eq. 1); the
 *                             activations of Table 1 plus ELU / LeakyReLU
 *   fbo_dp_solve              Eq. 7 (discrete DP, k-1 on the right-hand side as
 *                             in Eq. 6), Eq. 8-9 (prefix integrals), Eq. 4
 *                             (optimal levels), uniform weight Eq. 10
 *   fbo_bruteforce            Eq. 3 minimised by exhaustive search on the grid
 *   fbo_objective             Eq. 3 for a given boundary set (levels by Eq. 4)
 *   *_w variants              the same with the weight w chosen: 0 = indicator of
 *                             [A,B] (Eq. 10), 1 = standard normal density cut to
 *                             [A,B] (the other practical choice named under Eq. 3)
 *   fbo_loss_at               Eq. 3 and its gradient Eq. 5 at arbitrary (off-grid)
 *                             boundaries, levels by Eq. 4
 *   fbo_finetune              gradient descent on the boundaries started from the
 *                             DP result (Sec. 3, "Dynamic programming" paragraph)
 *   fbo_fwd_*                 Listing 1 "forward": y = f(x); code = position
 *                             of x among the boundaries s (Eq. 2); only
 *                             log2(K) bits per element are kept (Sec. 2)
 *   fbo_fwd_*_fold            the same with the position of |x| (caption of
 *                             Fig. 3: for an even f' only the positive half-axis
 *                             is quantised, the table lives on [0, B])
 *   fbo_bwd_*                 Listing 1 "backward": grad_in = grad_out * y[code]
 *   fbo_bias_add_*            an extension in front of Listing 1: the activation's
 *                             input is x + bias (one bias per column), the exact
 *                             sum rounded once to the storage type
 *
 * Every function here is pinned by tests/test_oracle_*.py against Table 1,
 * brute force, closed forms and library routines; none is "parity unpinned"
 * except the boundary indices of degenerate (piecewise-constant f') tables,
 * where every zero-error table is equally correct.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum {
    FBO_GELU = 0,      /* x * Phi(x), erf form */
    FBO_SILU = 1,      /* x * sigmoid(x) (Swish) */
    FBO_SIGMOID = 2,
    FBO_TANH = 3,
    FBO_ELU = 4,       /* alpha = 1 */
    FBO_SOFTPLUS = 5,  /* beta = 1, no threshold */
    FBO_LEAKY_RELU = 6,/* slope 0.01 */
    FBO_RELU = 7,      /* Table 1 row, pin only */
    FBO_SELU = 8       /* Table 1 row, pin only */
};

#define SELU_LAMBDA 1.0507009873554804934193349852946
#define SELU_ALPHA  1.6732632423543772848170429916717

static double sigmoid64(double x)
{
    /* 1/(1+e^-x), written so that neither branch overflows */
    if (x >= 0.0) return 1.0 / (1.0 + exp(-x));
    double e = exp(x);
    return e / (1.0 + e);
}

static double std_normal_cdf(double x) { return 0.5 * erfc(-x * M_SQRT1_2); }
static double std_normal_pdf(double x) { return exp(-0.5 * x * x) / sqrt(2.0 * M_PI); }

/* f(x), Sec. 2. */
double fbo_act(int act, double x)
{
    switch (act) {
    case FBO_GELU:       return x * std_normal_cdf(x);
    case FBO_SILU:       return x * sigmoid64(x);
    case FBO_SIGMOID:    return sigmoid64(x);
    case FBO_TANH:       return tanh(x);
    case FBO_ELU:        return x > 0.0 ? x : expm1(x);
    case FBO_SOFTPLUS:   return (x > 0.0 ? x : 0.0) + log1p(exp(-fabs(x)));
    case FBO_LEAKY_RELU: return x > 0.0 ? x : 0.01 * x;
    case FBO_RELU:       return x > 0.0 ? x : 0.0;
    case FBO_SELU:       return SELU_LAMBDA * (x > 0.0 ? x : SELU_ALPHA * expm1(x));
    default:             return NAN;
    }
}

/* f'(x), the factor of the chain rule, Eq. 1. */
double fbo_act_deriv(int act, double x)
{
    double s;
    switch (act) {
    case FBO_GELU:       return std_normal_cdf(x) + x * std_normal_pdf(x);
    case FBO_SILU:       s = sigmoid64(x); return s * (1.0 + x * (1.0 - s));
    case FBO_SIGMOID:    s = sigmoid64(x); return s * (1.0 - s);
    case FBO_TANH:       s = tanh(x); return 1.0 - s * s;
    case FBO_ELU:        return x > 0.0 ? 1.0 : exp(x);
    case FBO_SOFTPLUS:   return sigmoid64(x);
    case FBO_LEAKY_RELU: return x > 0.0 ? 1.0 : 0.01;
    case FBO_RELU:       return x > 0.0 ? 1.0 : 0.0;
    case FBO_SELU:       return SELU_LAMBDA * (x > 0.0 ? 1.0 : SELU_ALPHA * exp(x));
    default:             return NAN;
    }
}

/* ------------------------------------------------------------------------ */
/* Prefix integrals of Eq. 8-9 with the uniform weight of Eq. 10 on [A,B].   */
/*   W(i)  = t_i - A                       (integral of w)                   */
/*   FW(i) = f(t_i) - f(A)                 (integral of f' w, closed form)   */
/*   F2(i) = F2(i-1) + int_cell f'^2       (4-point Gauss-Legendre per cell; */
/*           the nodes are interior, so a jump of f' at a grid point is      */
/*           never sampled)                                                  */
/* ------------------------------------------------------------------------ */
typedef struct {
    int n;
    double *t, *W, *FW, *F2;
} prefix_t;

/* w(x) on [A,B]: weight 0 -> 1, weight 1 -> standard normal density */
static double weight_at(int weight, double x) { return weight ? std_normal_pdf(x) : 1.0; }

static int prefix_build(prefix_t *p, int act, double A, double B, int n, int weight)
{
    static const double gl_x[4] = { -0.86113631159405257522, -0.33998104358485626480,
                                     0.33998104358485626480,  0.86113631159405257522 };
    static const double gl_w[4] = {  0.34785484513745385737,  0.65214515486254614263,
                                     0.65214515486254614263,  0.34785484513745385737 };
    p->n = n;
    p->t  = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    p->W  = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    p->FW = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    p->F2 = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    if (!p->t || !p->W || !p->FW || !p->F2) return -1;
    double fA = fbo_act(act, A);
    for (int i = 0; i <= n; ++i) {
        p->t[i]  = A + (B - A) * (double)i / (double)n;
        if (!weight) {                      /* closed forms for w = 1 */
            p->W[i]  = p->t[i] - A;
            p->FW[i] = fbo_act(act, p->t[i]) - fA;
        }
    }
    p->t[n] = B;
    p->F2[0] = 0.0;
    if (weight) { p->W[0] = 0.0; p->FW[0] = 0.0; }
    for (int i = 0; i < n; ++i) {
        double a = p->t[i], b = p->t[i + 1];
        double mid = 0.5 * (a + b), half = 0.5 * (b - a), acc = 0.0, accw = 0.0, accfw = 0.0;
        for (int q = 0; q < 4; ++q) {
            double xq = mid + half * gl_x[q];
            double d = fbo_act_deriv(act, xq), wq = weight_at(weight, xq);
            acc += gl_w[q] * d * d * wq;
            accw += gl_w[q] * wq;
            accfw += gl_w[q] * d * wq;
        }
        p->F2[i + 1] = p->F2[i] + half * acc;
        if (weight) {                       /* Eq. 9, all three by quadrature */
            p->W[i + 1]  = p->W[i] + half * accw;
            p->FW[i + 1] = p->FW[i] + half * accfw;
        }
    }
    return 0;
}

static void prefix_free(prefix_t *p)
{
    free(p->t); free(p->W); free(p->FW); free(p->F2);
}

/* y(j,i) of Eq. 8: the optimal level (Eq. 4) of the bin [t_j, t_i]. */
static double bin_level(const prefix_t *p, int j, int i)
{
    return (p->FW[i] - p->FW[j]) / (p->W[i] - p->W[j]);
}

/* T(j,i) of Eq. 8: the error of the bin [t_j, t_i] under its optimal level.
 * It is a sum of squares, so a negative value can only be rounding noise and
 * is clamped to zero. */
static double bin_cost(const prefix_t *p, int j, int i)
{
    double y = bin_level(p, j, i);
    double c = p->F2[i] - p->F2[j] - y * y * (p->W[i] - p->W[j]);
    return c > 0.0 ? c : 0.0;
}

/*
 * Discrete dynamic programme, Eq. 7:
 *     DP(i,k) = min_j DP(j,k-1) + T(j,i),   DP(0,0) = 0,
 * i = grid index of the right end, k = number of constant pieces used on
 * [A, t_i].  The answer is DP(n,K); the first minimiser wins a tie.
 * Outputs: idx_out[K-1] interior boundary grid indices (increasing),
 * s_out[K-1] = t[idx], lev_out[K] by Eq. 4 with s_0 = A and s_K = B,
 * *objective = DP(n,K).  Returns 0 on success.
 */
int fbo_dp_solve_w(int act, double A, double B, int n, int K, int weight,
                   double *s_out, double *lev_out, double *objective, int *idx_out);

int fbo_dp_solve(int act, double A, double B, int n, int K,
                 double *s_out, double *lev_out, double *objective, int *idx_out)
{
    return fbo_dp_solve_w(act, A, B, n, K, 0, s_out, lev_out, objective, idx_out);
}

int fbo_dp_solve_w(int act, double A, double B, int n, int K, int weight,
                   double *s_out, double *lev_out, double *objective, int *idx_out)
{
    if (n < 1 || K < 1 || K > n || !(A < B)) return -1;
    prefix_t p;
    if (prefix_build(&p, act, A, B, n, weight)) return -2;
    size_t stride = (size_t)(n + 1);
    double *dp  = (double *)malloc(sizeof(double) * stride * (size_t)(K + 1));
    int    *arg = (int *)malloc(sizeof(int) * stride * (size_t)(K + 1));
    if (!dp || !arg) return -2;
    for (size_t q = 0; q < stride * (size_t)(K + 1); ++q) { dp[q] = INFINITY; arg[q] = -1; }
    dp[0] = 0.0; /* DP(0,0) */
    for (int k = 1; k <= K; ++k) {
        for (int i = k; i <= n; ++i) {
            double best = INFINITY; int bestj = -1;
            for (int j = k - 1; j < i; ++j) {
                double prev = dp[(size_t)(k - 1) * stride + (size_t)j];
                if (prev == INFINITY) continue;
                double v = prev + bin_cost(&p, j, i);
                if (v < best) { best = v; bestj = j; }
            }
            dp[(size_t)k * stride + (size_t)i] = best;
            arg[(size_t)k * stride + (size_t)i] = bestj;
        }
    }
    if (objective) *objective = dp[(size_t)K * stride + (size_t)n];
    /* back-track the right ends of pieces K, K-1, ..., 1 */
    int *ends = (int *)malloc(sizeof(int) * (size_t)(K + 1));
    ends[K] = n;
    for (int k = K; k >= 1; --k) ends[k - 1] = arg[(size_t)k * stride + (size_t)ends[k]];
    /* ends[0] == 0 by construction */
    for (int m = 1; m < K; ++m) {
        if (idx_out) idx_out[m - 1] = ends[m];
        if (s_out)   s_out[m - 1] = p.t[ends[m]];
    }
    if (lev_out)
        for (int m = 0; m < K; ++m) lev_out[m] = bin_level(&p, ends[m], ends[m + 1]);
    free(ends); free(dp); free(arg);
    prefix_free(&p);
    return 0;
}

/* Eq. 3 for the boundary grid indices idx[0..K-2] (levels by Eq. 4). */
int fbo_objective_w(int act, double A, double B, int n, int K, int weight, const int *idx, double *objective);

int fbo_objective(int act, double A, double B, int n, int K, const int *idx, double *objective)
{
    return fbo_objective_w(act, A, B, n, K, 0, idx, objective);
}

int fbo_objective_w(int act, double A, double B, int n, int K, int weight, const int *idx, double *objective)
{
    prefix_t p;
    if (prefix_build(&p, act, A, B, n, weight)) return -2;
    double total = 0.0;
    int left = 0;
    for (int m = 0; m < K; ++m) {
        int right = (m == K - 1) ? n : idx[m];
        if (right <= left) { prefix_free(&p); return -1; }
        total += bin_cost(&p, left, right);
        left = right;
    }
    *objective = total;
    prefix_free(&p);
    return 0;
}

/*
 * Exhaustive search: every increasing (K-1)-subset of the interior grid
 * points 1..n-1, each scored by Eq. 3 with the levels of Eq. 4.  The
 * lexicographically first minimiser is kept.  Only for tiny n.
 */
int fbo_bruteforce_w(int act, double A, double B, int n, int K, int weight, int *idx_out, double *objective);

int fbo_bruteforce(int act, double A, double B, int n, int K, int *idx_out, double *objective)
{
    return fbo_bruteforce_w(act, A, B, n, K, 0, idx_out, objective);
}

int fbo_bruteforce_w(int act, double A, double B, int n, int K, int weight, int *idx_out, double *objective)
{
    if (K < 1 || K > n) return -1;
    prefix_t p;
    if (prefix_build(&p, act, A, B, n, weight)) return -2;
    int m = K - 1;
    int *c = (int *)malloc(sizeof(int) * (size_t)(m + 1));
    for (int q = 0; q < m; ++q) c[q] = q + 1;
    double best = INFINITY;
    for (;;) {
        double total = 0.0;
        int left = 0;
        for (int q = 0; q <= m; ++q) {
            int right = (q == m) ? n : c[q];
            total += bin_cost(&p, left, right);
            left = right;
        }
        if (total < best) {
            best = total;
            for (int q = 0; q < m; ++q) idx_out[q] = c[q];
        }
        /* next combination of {1..n-1} choose m */
        int q = m - 1;
        while (q >= 0 && c[q] == (n - 1) - (m - 1 - q)) --q;
        if (q < 0) break;
        ++c[q];
        for (int r = q + 1; r < m; ++r) c[r] = c[r - 1] + 1;
    }
    *objective = best;
    free(c);
    prefix_free(&p);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Off-grid boundaries: Eq. 3 with the levels of Eq. 4, its gradient Eq. 5,  */
/* and gradient descent from the DP result.                                  */
/* ------------------------------------------------------------------------ */

/* integrals of w, f' w and f'^2 w over [a,b]: 4-point Gauss-Legendre on panels no wider than 2^-8 */
static void bin_integrals(int act, int weight, double a, double b, double *iw, double *ifw, double *if2w)
{
    static const double gx[4] = { -0.86113631159405257522, -0.33998104358485626480,
                                   0.33998104358485626480,  0.86113631159405257522 };
    static const double gw[4] = {  0.34785484513745385737,  0.65214515486254614263,
                                   0.65214515486254614263,  0.34785484513745385737 };
    int panels = (int)ceil((b - a) * 256.0);
    if (panels < 1) panels = 1;
    double h = (b - a) / panels, sw = 0.0, sfw = 0.0, sf2 = 0.0;
    for (int k = 0; k < panels; ++k) {
        double mid = a + (k + 0.5) * h, half = 0.5 * h;
        for (int q = 0; q < 4; ++q) {
            double x = mid + half * gx[q];
            double d = fbo_act_deriv(act, x), w = weight_at(weight, x);
            sw += gw[q] * w * half; sfw += gw[q] * d * w * half; sf2 += gw[q] * d * d * w * half;
        }
    }
    *iw = sw; *ifw = sfw; *if2w = sf2;
}

/*
 * L(s, y(s)) of Eq. 3 for K-1 increasing boundaries s in (A,B), with
 * y_i by Eq. 4; grad_out[i] = dL/ds_i by Eq. 5:
 *     (2 f'(s_i) - y_i - y_{i-1}) (y_i - y_{i-1}) w(s_i),
 * y_{i-1} the level left of s_i and y_i the level right of it.
 * lev_out (K) and grad_out (K-1) may be NULL.  Returns L, or NAN if s is not increasing.
 */
double fbo_loss_at(int act, double A, double B, int weight, int K, const double *s,
                   double *lev_out, double *grad_out)
{
    double lev[64];
    double total = 0.0, left = A;
    if (K > 64) return NAN;
    for (int m = 0; m < K; ++m) {
        double right = (m == K - 1) ? B : s[m];
        if (!(right > left)) return NAN;
        double iw, ifw, if2;
        bin_integrals(act, weight, left, right, &iw, &ifw, &if2);
        lev[m] = ifw / iw;                                  /* Eq. 4 */
        total += if2 - lev[m] * lev[m] * iw;                /* int (f' - y)^2 w  with the optimal y */
        left = right;
    }
    if (lev_out) for (int m = 0; m < K; ++m) lev_out[m] = lev[m];
    if (grad_out)
        for (int i = 0; i < K - 1; ++i)
            grad_out[i] = (2.0 * fbo_act_deriv(act, s[i]) - lev[i + 1] - lev[i]) * (lev[i + 1] - lev[i])
                          * weight_at(weight, s[i]);
    return total;
}

/*
 * Gradient descent on the boundaries.  Each component of Eq. 5 is divided by the positive factor
 * |y_i - y_{i-1}| w(s_i) it contains (a diagonal scaling: the direction is still a descent
 * direction, and what is left is the stationarity residual 2 f'(s_i) - y_i - y_{i-1}, so flat
 * outer bins move as fast as steep inner ones).  The step is halved until L decreases.  At most
 * max_iter steps; stops when every scaled component is below 1e-10.  s_inout: the DP boundaries
 * on entry, the fine-tuned ones on exit.  Returns the number of steps taken, negative on error.
 */
int fbo_finetune(int act, double A, double B, int weight, int K, double *s_inout, int max_iter,
                 double *lev_out, double *objective_out)
{
    double g[64], lev[64], dir[64], trial[64];
    if (K > 64) return -1;
    double cur = fbo_loss_at(act, A, B, weight, K, s_inout, lev, g);
    if (isnan(cur)) return -1;
    double step = 0.25;
    int it = 0;
    for (; it < max_iter; ++it) {
        double dmax = 0.0;
        for (int i = 0; i < K - 1; ++i) {
            double scale = fabs(lev[i + 1] - lev[i]) * weight_at(weight, s_inout[i]);
            dir[i] = scale > 1e-300 ? g[i] / scale : 0.0;
            if (fabs(dir[i]) > dmax) dmax = fabs(dir[i]);
        }
        if (dmax < 1e-10) break;
        int moved = 0;
        for (int half = 0; half < 60; ++half) {
            for (int i = 0; i < K - 1; ++i) trial[i] = s_inout[i] - step * dir[i];
            double l = fbo_loss_at(act, A, B, weight, K, trial, NULL, NULL);
            if (!isnan(l) && l < cur) { cur = l; moved = 1; break; }
            step *= 0.5;
        }
        if (!moved) break;
        for (int i = 0; i < K - 1; ++i) s_inout[i] = trial[i];
        fbo_loss_at(act, A, B, weight, K, s_inout, lev, g);
        step *= 2.0;                                        /* try a longer step next time */
    }
    cur = fbo_loss_at(act, A, B, weight, K, s_inout, lev_out, NULL);
    if (objective_out) *objective_out = cur;
    return it;
}

/* ------------------------------------------------------------------------ */
/* Rounding binary64 -> storage dtype, round-to-nearest-even, in ONE step.   */
/* ------------------------------------------------------------------------ */

/* bfloat16: 8 exponent bits, 7 stored mantissa bits.  The value is scaled so
 * that one bfloat16 ulp becomes 1.0, rounded with nearbyint (nearest-even in
 * the default rounding mode) and scaled back; both scalings are exact. */
uint16_t fbo_f64_to_bf16(double d)
{
    if (isnan(d)) return 0x7fc0;
    if (isinf(d)) return d > 0 ? 0x7f80 : 0xff80;
    double r = 0.0;
    if (d != 0.0) {
        int e = ilogb(d);
        if (e < -126) e = -126;           /* subnormal range: fixed spacing 2^-133 */
        double ulp = ldexp(1.0, e - 7);
        r = nearbyint(d / ulp) * ulp;
    } else {
        r = d;                             /* keeps the sign of zero */
    }
    float f = (float)r;                    /* exact, or +-inf past the largest finite bf16 */
    if (fabs(r) >= ldexp(1.0, 128)) f = r > 0 ? INFINITY : -INFINITY;
    uint32_t u; memcpy(&u, &f, 4);
    if (r == 0.0 && signbit(d)) u = 0x80000000u;
    return (uint16_t)(u >> 16);
}

double fbo_bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return (double)f;
}

/* IEEE binary16: 5 exponent bits, 10 stored mantissa bits, subnormals below 2^-14, same method. */
uint16_t fbo_f64_to_f16(double d)
{
    if (isnan(d)) return 0x7e00;
    if (isinf(d)) return d > 0 ? 0x7c00 : 0xfc00;
    uint16_t sign = signbit(d) ? 0x8000 : 0;
    double a = fabs(d);
    if (a == 0.0) return sign;
    int e = ilogb(a);
    if (e < -14) e = -14;                        /* subnormal range: fixed spacing 2^-24 */
    double ulp = ldexp(1.0, e - 10);
    double r = nearbyint(a / ulp) * ulp;         /* exact scaling, nearest-even */
    if (r >= 65520.0) return sign | 0x7c00;      /* past the largest finite value 65504 (+ half an ulp) */
    if (r == 0.0) return sign;
    int er = ilogb(r);
    if (er < -14) return sign | (uint16_t)nearbyint(r / ldexp(1.0, -24));          /* subnormal */
    uint16_t mant = (uint16_t)nearbyint(r / ldexp(1.0, er - 10)) & 0x3ff;
    return sign | (uint16_t)((er + 15) << 10) | mant;
}

double fbo_f16_to_f64(uint16_t h)
{
    int e = (h >> 10) & 0x1f, m = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp(1.0 + m / 1024.0, e - 15);
    return (h & 0x8000) ? -v : v;
}

static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16; float f; memcpy(&f, &u, 4); return f;
}

/* ------------------------------------------------------------------------ */
/* Forward, Listing 1: y = f(x); X_pos = position of x among s; save X_pos   */
/* in log2(K) bits.  Position = number of boundaries strictly below x, so    */
/* bin i is (s_i, s_{i+1}] and values outside [A,B] fall in the end bins.    */
/* Bit layout of the saved tensor: one flat bit stream, element e occupies   */
/* bits [e*bits, e*bits+bits), least significant bit first, stored in        */
/* little-endian 32-bit words; unused bits of the last word are zero.        */
/* ------------------------------------------------------------------------ */
static uint32_t bucketize(const float *s, int nb, float x)
{
    uint32_t c = 0;
    for (int j = 0; j < nb; ++j) if (s[j] < x) ++c;
    return c;
}

static void put_code(uint32_t *packed, size_t e, int bits, uint32_t code)
{
    for (int b = 0; b < bits; ++b) {
        size_t pos = e * (size_t)bits + (size_t)b;
        if ((code >> b) & 1u) packed[pos >> 5] |= (uint32_t)1 << (pos & 31);
    }
}

static uint32_t get_code(const uint32_t *packed, size_t e, int bits)
{
    uint32_t code = 0;
    for (int b = 0; b < bits; ++b) {
        size_t pos = e * (size_t)bits + (size_t)b;
        code |= ((packed[pos >> 5] >> (pos & 31)) & 1u) << b;
    }
    return code;
}

size_t fbo_packed_words(size_t n, int bits) { return (n * (size_t)bits + 31) / 32; }

void fbo_pack(int bits, const uint8_t *codes, uint32_t *packed, size_t n)
{
    memset(packed, 0, 4 * fbo_packed_words(n, bits));
    for (size_t e = 0; e < n; ++e) put_code(packed, e, bits, codes[e]);
}

void fbo_unpack(int bits, const uint32_t *packed, uint8_t *codes, size_t n)
{
    for (size_t e = 0; e < n; ++e) codes[e] = (uint8_t)get_code(packed, e, bits);
}

/* fold != 0: the table approximates an even f' on [0, B] and the code is the position of |x|
 * (caption of Fig. 3).  y is unaffected. */
void fbo_fwd_f32_fold(int act, int bits, int fold, const float *s, const float *x, float *y,
                      uint32_t *packed, size_t n)
{
    int nb = (1 << bits) - 1;
    memset(packed, 0, 4 * fbo_packed_words(n, bits));
    for (size_t e = 0; e < n; ++e) {
        y[e] = (float)fbo_act(act, (double)x[e]);
        put_code(packed, e, bits, bucketize(s, nb, fold ? fabsf(x[e]) : x[e]));
    }
}

void fbo_fwd_bf16_fold(int act, int bits, int fold, const float *s, const uint16_t *x, uint16_t *y,
                       uint32_t *packed, size_t n)
{
    int nb = (1 << bits) - 1;
    memset(packed, 0, 4 * fbo_packed_words(n, bits));
    for (size_t e = 0; e < n; ++e) {
        float xf = bf16_to_f32(x[e]);
        y[e] = fbo_f64_to_bf16(fbo_act(act, fbo_bf16_to_f64(x[e])));
        put_code(packed, e, bits, bucketize(s, nb, fold ? fabsf(xf) : xf));
    }
}

void fbo_fwd_f16_fold(int act, int bits, int fold, const float *s, const uint16_t *x, uint16_t *y,
                      uint32_t *packed, size_t n)
{
    int nb = (1 << bits) - 1;
    memset(packed, 0, 4 * fbo_packed_words(n, bits));
    for (size_t e = 0; e < n; ++e) {
        double xd = fbo_f16_to_f64(x[e]);
        float xf = (float)xd;                                /* exact: binary16 is a subset of binary32 */
        y[e] = fbo_f64_to_f16(fbo_act(act, xd));
        put_code(packed, e, bits, bucketize(s, nb, fold ? fabsf(xf) : xf));
    }
}

void fbo_fwd_f32(int act, int bits, const float *s, const float *x, float *y,
                 uint32_t *packed, size_t n)
{
    fbo_fwd_f32_fold(act, bits, 0, s, x, y, packed, n);
}

void fbo_fwd_bf16(int act, int bits, const float *s, const uint16_t *x, uint16_t *y,
                  uint32_t *packed, size_t n)
{
    fbo_fwd_bf16_fold(act, bits, 0, s, x, y, packed, n);
}

/* ------------------------------------------------------------------------ */
/* Backward, Listing 1: grad_in = grad_out * y[X_pos].  The product is one   */
/* binary32 multiply (levels are binary32), then one rounding to the dtype.  */
/* ------------------------------------------------------------------------ */
void fbo_bwd_f32(int bits, const float *lev, const uint32_t *packed, const float *grad_out,
                 float *grad_in, size_t n)
{
    for (size_t e = 0; e < n; ++e) {
        volatile float p = grad_out[e] * lev[get_code(packed, e, bits)];
        grad_in[e] = p;
    }
}

void fbo_bwd_bf16(int bits, const float *lev, const uint32_t *packed, const uint16_t *grad_out,
                  uint16_t *grad_in, size_t n)
{
    for (size_t e = 0; e < n; ++e) {
        volatile float p = bf16_to_f32(grad_out[e]) * lev[get_code(packed, e, bits)];
        grad_in[e] = fbo_f64_to_bf16((double)p);
    }
}

void fbo_bwd_f16(int bits, const float *lev, const uint32_t *packed, const uint16_t *grad_out,
                 uint16_t *grad_in, size_t n)
{
    for (size_t e = 0; e < n; ++e) {
        volatile float p = (float)fbo_f16_to_f64(grad_out[e]) * lev[get_code(packed, e, bits)];
        grad_in[e] = fbo_f64_to_f16((double)p);
    }
}

void fbo_f64_to_f16_array(const double *x, uint16_t *y, size_t n)
{
    for (size_t e = 0; e < n; ++e) y[e] = fbo_f64_to_f16(x[e]);
}

/* Elementwise helpers for the Python side. */
void fbo_act_array(int act, const double *x, double *y, size_t n)
{
    for (size_t e = 0; e < n; ++e) y[e] = fbo_act(act, x[e]);
}

void fbo_act_deriv_array(int act, const double *x, double *y, size_t n)
{
    for (size_t e = 0; e < n; ++e) y[e] = fbo_act_deriv(act, x[e]);
}

void fbo_f64_to_bf16_array(const double *x, uint16_t *y, size_t n)
{
    for (size_t e = 0; e < n; ++e) y[e] = fbo_f64_to_bf16(x[e]);
}

/* ------------------------------------------------------------------------- */
/* Bias add in front of the activation (an extension: the paper's Listing 1    */
/* starts at the activation's input).  z[r][c] = x[r][c] + bias[c], the exact  */
/* sum rounded once to the storage type -- what an unfused framework op that   */
/* adds the bias and stores the result would hand to the activation.  The sum */
/* of two binary64 numbers is formed in binary64; it is exact whenever the two */
/* exponents are less than 29 (binary32) apart, and beyond that the smaller    */
/* term cannot move the rounding of the larger one, which is itself a value of */
/* the storage type, so the single rounding below is the IEEE sum.             */
/* ------------------------------------------------------------------------- */
void fbo_bias_add_f32(const float *x, const float *bias, size_t rows, size_t cols, float *z)
{
    for (size_t r = 0; r < rows; ++r)
        for (size_t c = 0; c < cols; ++c)
            z[r * cols + c] = (float)((double)x[r * cols + c] + (double)bias[c]);
}

void fbo_bias_add_bf16(const uint16_t *x, const uint16_t *bias, size_t rows, size_t cols, uint16_t *z)
{
    for (size_t r = 0; r < rows; ++r)
        for (size_t c = 0; c < cols; ++c)
            z[r * cols + c] = fbo_f64_to_bf16(fbo_bf16_to_f64(x[r * cols + c]) + fbo_bf16_to_f64(bias[c]));
}

void fbo_bias_add_f16(const uint16_t *x, const uint16_t *bias, size_t rows, size_t cols, uint16_t *z)
{
    for (size_t r = 0; r < rows; ++r)
        for (size_t c = 0; c < cols; ++c)
            z[r * cols + c] = fbo_f64_to_f16(fbo_f16_to_f64(x[r * cols + c]) + fbo_f16_to_f64(bias[c]));
}
