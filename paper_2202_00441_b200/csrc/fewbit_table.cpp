// Host side of the library: the table object and the offline solver that
// finds the optimal piecewise-constant approximation of f' (Eq. 3) by the
// dynamic programme of Eq. 7 over prefix integrals (Eq. 8-9), with the
// levels of Eq. 4.  Pure C++17, no CUDA.
#include "fewbit_internal.h"

#include <cmath>
#include <cstring>
#include <limits>
#include <map>
#include <memory>
#include <mutex>
#include <new>
#include <tuple>
#include <vector>

namespace fewbit {
namespace {

// ---------------------------------------------------------------------------
// f and f' in binary64 (Sec. 2; Eq. 1 needs f', the closed form of Eq. 9's
// FW needs f).
// ---------------------------------------------------------------------------
inline double logistic(double x) {
    if (x >= 0.0) return 1.0 / (1.0 + std::exp(-x));
    const double e = std::exp(x);
    return e / (1.0 + e);
}

constexpr double kSeluScale = 1.0507009873554804934193349852946;
constexpr double kSeluAlpha = 1.6732632423543772848170429916717;

inline double Phi(double x) { return 0.5 * std::erfc(-x * 0.70710678118654752440); }
inline double phi(double x) { return 0.39894228040143267794 * std::exp(-0.5 * x * x); }

double value(fewbit_act a, double x) {
    switch (a) {
    case FEWBIT_GELU: return x * Phi(x);
    case FEWBIT_SILU: return x * logistic(x);
    case FEWBIT_SIGMOID: return logistic(x);
    case FEWBIT_TANH: return std::tanh(x);
    case FEWBIT_ELU: return x > 0.0 ? x : std::expm1(x);
    case FEWBIT_SOFTPLUS: return std::fmax(x, 0.0) + std::log1p(std::exp(-std::fabs(x)));
    case FEWBIT_LEAKY_RELU: return x > 0.0 ? x : 0.01 * x;
    case FEWBIT_RELU: return x > 0.0 ? x : 0.0;
    case FEWBIT_SELU: return kSeluScale * (x > 0.0 ? x : kSeluAlpha * std::expm1(x));
    }
    return std::numeric_limits<double>::quiet_NaN();
}

double slope(fewbit_act a, double x) {
    switch (a) {
    case FEWBIT_GELU: return Phi(x) + x * phi(x);
    case FEWBIT_SILU: { const double g = logistic(x); return g + x * g * (1.0 - g); }
    case FEWBIT_SIGMOID: { const double g = logistic(x); return g * (1.0 - g); }
    case FEWBIT_TANH: { const double t = std::tanh(x); return (1.0 - t) * (1.0 + t); }
    case FEWBIT_ELU: return x > 0.0 ? 1.0 : std::exp(x);
    case FEWBIT_SOFTPLUS: return logistic(x);
    case FEWBIT_LEAKY_RELU: return x > 0.0 ? 1.0 : 0.01;
    case FEWBIT_RELU: return x > 0.0 ? 1.0 : 0.0;
    case FEWBIT_SELU: return kSeluScale * (x > 0.0 ? 1.0 : kSeluAlpha * std::exp(x));
    }
    return std::numeric_limits<double>::quiet_NaN();
}

// ---------------------------------------------------------------------------
// One solved grid: every layer DP(., k), k = 1..kMaxLevels, with its argmin,
// so that tables for 1, 2, 3 and 4 bits come out of a single run.
// ---------------------------------------------------------------------------
struct Solved {
    int n = 0;
    double A = 0, B = 0;
    std::vector<double> F2, FW, Wt;             // prefix integrals of Eq. 8-9 (uniform weight, Eq. 10)
    std::vector<double> best_at_n;              // DP(n, k)
    std::vector<std::vector<int32_t>> from;     // from[k][i] = argmin_j of Eq. 7

    double level(int j, int i) const { return (FW[i] - FW[j]) / (Wt[i] - Wt[j]); }
};

// the weight w of Eq. 3 on [A,B]: 1 (Eq. 10) or the standard normal density
inline double weight_at(int weight, double x) { return weight == FEWBIT_WEIGHT_NORMAL ? phi(x) : 1.0; }

std::shared_ptr<const Solved> solve_grid(fewbit_act act, double A, double B, int n, int weight) {
    auto out = std::make_shared<Solved>();
    Solved &g = *out;
    g.n = n; g.A = A; g.B = B;
    g.F2.assign(n + 1, 0.0); g.FW.assign(n + 1, 0.0); g.Wt.assign(n + 1, 0.0);

    // Eq. 9: the three running integrals.  With w = 1 on [A,B] the integral of
    // f' is f itself; the integral of f'^2 uses a 4-node Gauss-Legendre rule
    // per cell, whose nodes never touch a grid point (f' may jump there).
    const double node[2] = {0.33998104358485626480, 0.86113631159405257522};
    const double wght[2] = {0.65214515486254614263, 0.34785484513745385737};
    const double fA = value(act, A);
    double left = A;
    for (int i = 1; i <= n; ++i) {
        const double right = (i == n) ? B : A + (B - A) * (static_cast<double>(i) / n);
        const double c = 0.5 * (left + right), r = 0.5 * (right - left);
        double q = 0.0, qf = 0.0;
        for (int m = 0; m < 2; ++m) {
            const double xm = c - r * node[m], xp = c + r * node[m];
            const double dm = slope(act, xm), dp = slope(act, xp);
            const double wm = weight_at(weight, xm), wp = weight_at(weight, xp);
            q += wght[m] * (dm * dm * wm + dp * dp * wp);
            qf += wght[m] * (dm * wm + dp * wp);
        }
        g.F2[i] = g.F2[i - 1] + r * q;
        if (weight == FEWBIT_WEIGHT_NORMAL) {
            g.FW[i] = g.FW[i - 1] + r * qf;              // no closed form: same quadrature
            g.Wt[i] = Phi(right) - Phi(A);               // closed form
        } else {
            g.FW[i] = value(act, right) - fA;
            g.Wt[i] = right - A;
        }
        left = right;
    }

    // Eq. 7 with Eq. 8's O(1) cost: cost(j,i) = dF2 - dFW^2 / dW, never below 0.
    const double inf = std::numeric_limits<double>::infinity();
    std::vector<double> prev(n + 1, inf), cur(n + 1, inf);
    prev[0] = 0.0;                                  // zero pieces cover [A, A]
    g.best_at_n.assign(kMaxLevels + 1, inf);
    g.from.assign(kMaxLevels + 1, {});
    const int layers = std::min(kMaxLevels, n);
    for (int k = 1; k <= layers; ++k) {
        std::vector<int32_t> &arg = g.from[k];
        arg.assign(n + 1, -1);
        std::fill(cur.begin(), cur.end(), inf);
        for (int i = k; i <= n; ++i) {
            const double f2i = g.F2[i], fwi = g.FW[i], wi = g.Wt[i];
            double best = inf;
            int32_t best_j = -1;
            for (int j = k - 1; j < i; ++j) {
                const double dfw = fwi - g.FW[j];
                double cost = (f2i - g.F2[j]) - dfw * (dfw / (wi - g.Wt[j]));
                cost = cost > 0.0 ? cost : 0.0;
                const double total = prev[j] + cost;
                if (total < best) { best = total; best_j = j; }
            }
            cur[i] = best;
            arg[i] = best_j;
        }
        g.best_at_n[k] = cur[n];
        prev.swap(cur);
    }
    return out;
}

std::mutex g_cache_mutex;
std::map<std::tuple<int, double, double, int, int>, std::shared_ptr<const Solved>> g_cache;

std::shared_ptr<const Solved> solved_for(fewbit_act act, double A, double B, int n, int weight) {
    const auto key = std::make_tuple(static_cast<int>(act), A, B, n, weight);
    {
        std::lock_guard<std::mutex> lock(g_cache_mutex);
        auto it = g_cache.find(key);
        if (it != g_cache.end()) return it->second;
    }
    auto fresh = solve_grid(act, A, B, n, weight);
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    if (g_cache.size() >= 64) g_cache.clear();
    return g_cache.emplace(key, fresh).first->second;
}

// ---------------------------------------------------------------------------
// Off-grid refinement (Sec. 3 proposes gradient-based fine-tuning of the grid optimum the DP returns).
// ---------------------------------------------------------------------------
struct BinSums { double w, fw, f2w; };

// integrals of w, f'w, f'^2 w over [a,b]; Gauss-Legendre (4 nodes) on panels of width <= 2^-8
BinSums integrate_bin(fewbit_act act, int weight, double a, double b) {
    const double node[2] = {0.33998104358485626480, 0.86113631159405257522};
    const double wght[2] = {0.65214515486254614263, 0.34785484513745385737};
    const int panels = std::max(1, static_cast<int>(std::ceil((b - a) * 256.0)));
    const double h = (b - a) / panels;
    BinSums out{0.0, 0.0, 0.0};
    for (int k = 0; k < panels; ++k) {
        const double c = a + (k + 0.5) * h, r = 0.5 * h;
        for (int m = 0; m < 2; ++m)
            for (int sgn = -1; sgn <= 1; sgn += 2) {
                const double x = c + sgn * r * node[m];
                const double d = slope(act, x), w = weight_at(weight, x) * wght[m] * r;
                out.w += w; out.fw += d * w; out.f2w += d * d * w;
            }
    }
    return out;
}

// Eq. 3 at boundaries s (levels by Eq. 4 into lev); grad = Eq. 5 when not null.  NaN if s is not increasing.
double loss_at(fewbit_act act, int weight, double A, double B, int K, const double *s, double *lev, double *grad) {
    double total = 0.0, left = A;
    for (int m = 0; m < K; ++m) {
        const double right = (m == K - 1) ? B : s[m];
        if (!(right > left)) return std::numeric_limits<double>::quiet_NaN();
        const BinSums b = integrate_bin(act, weight, left, right);
        lev[m] = b.fw / b.w;
        total += b.f2w - lev[m] * lev[m] * b.w;
        left = right;
    }
    if (grad != nullptr)
        for (int i = 0; i + 1 < K; ++i)
            grad[i] = (2.0 * slope(act, s[i]) - lev[i + 1] - lev[i]) * (lev[i + 1] - lev[i]) * weight_at(weight, s[i]);
    return total;
}

// Descent along Eq. 5 with each component divided by its positive factor |y_i - y_{i-1}| w(s_i)
// (what remains is the stationarity residual 2 f'(s_i) - y_i - y_{i-1}); step halved until Eq. 3 decreases.
double finetune(fewbit_act act, int weight, double A, double B, int K, double *s, double *lev, int max_iter) {
    double grad[kMaxLevels], dir[kMaxLevels], trial[kMaxLevels], tl[kMaxLevels];
    double cur = loss_at(act, weight, A, B, K, s, lev, grad);
    double step = 0.25;
    for (int it = 0; it < max_iter && !std::isnan(cur); ++it) {
        double largest = 0.0;
        for (int i = 0; i + 1 < K; ++i) {
            const double scale = std::fabs(lev[i + 1] - lev[i]) * weight_at(weight, s[i]);
            dir[i] = scale > 1e-300 ? grad[i] / scale : 0.0;
            largest = std::max(largest, std::fabs(dir[i]));
        }
        if (largest < 1e-10) break;
        bool moved = false;
        for (int halvings = 0; halvings < 60 && !moved; ++halvings) {
            for (int i = 0; i + 1 < K; ++i) trial[i] = s[i] - step * dir[i];
            const double l = loss_at(act, weight, A, B, K, trial, tl, nullptr);
            if (!std::isnan(l) && l < cur) { cur = l; moved = true; } else { step *= 0.5; }
        }
        if (!moved) break;
        for (int i = 0; i + 1 < K; ++i) s[i] = trial[i];
        loss_at(act, weight, A, B, K, s, lev, grad);
        step *= 2.0;
    }
    return loss_at(act, weight, A, B, K, s, lev, nullptr);
}

// code(x) = #{ j : s[j] < x } by a plain scan (host side, table set-up only)
inline unsigned code_of(const float *s, int nb, float x) {
    unsigned c = 0;
    for (int j = 0; j < nb; ++j) c += (s[j] < x) ? 1u : 0u;
    return c;
}

inline float from_bits(uint32_t u) { float f; std::memcpy(&f, &u, 4); return f; }

void encode_runs(const std::vector<uint8_t> &lut, CodeRuns *out) {
    out->count = 0;
    for (size_t c = 0; c < lut.size(); ++c) {
        if (c == 0 || lut[c] != lut[c - 1]) {
            if (out->count == kMaxRuns) { out->count = 0; return; }     // too fragmented: no look-up table
            out->run[out->count++] = static_cast<uint32_t>(c) | (static_cast<uint32_t>(lut[c]) << 24);
        }
    }
}

bool valid_act(int a) { return a >= 0 && a < FEWBIT_NUM_ACTS; }
bool valid_bits(int b) { return b >= 1 && b <= 4; }

}  // namespace

// Eq. 2's interval search as a table over bit patterns: the code is a step
// function of x with at most K-1 steps, so it is constant on long runs of
// patterns.
// IEEE binary16 pattern -> value
float f16_bits_to_float(uint32_t h) {
    const int e = (h >> 10) & 0x1f, m = h & 0x3ff;
    float v;
    if (e == 0) v = std::ldexp(static_cast<float>(m), -24);
    else if (e == 31) v = m ? std::numeric_limits<float>::quiet_NaN() : std::numeric_limits<float>::infinity();
    else v = std::ldexp(1.0f + m / 1024.0f, e - 15);
    return (h & 0x8000u) ? -v : v;
}

void build_code_runs(const float *s, int bits, bool folded, CodeRuns *bf16_runs, CodeRuns *f32_runs, CodeRuns *f16_runs) {
    const int nb = (1 << bits) - 1;
    const auto mag = [folded](float v) { return folded ? std::fabs(v) : v; };   // |NaN| stays NaN: code 0
    {   // bfloat16: exact code of every one of the 65 536 patterns
        std::vector<uint8_t> lut(1u << kCellBitsBf16);
        for (uint32_t p = 0; p < lut.size(); ++p) lut[p] = static_cast<uint8_t>(code_of(s, nb, mag(from_bits(p << 16))));
        encode_runs(lut, bf16_runs);
    }
    {   // binary16: exact code of every one of the 65 536 patterns
        std::vector<uint8_t> lut(1u << 16);
        for (uint32_t p = 0; p < lut.size(); ++p) lut[p] = static_cast<uint8_t>(code_of(s, nb, mag(f16_bits_to_float(p))));
        encode_runs(lut, f16_runs);
    }
    {   // binary32: per cell of 2^19 consecutive patterns, the smaller of the codes of its two
        // end points when they differ by at most one (codes are monotone across a cell)
        std::vector<uint8_t> lut(1u << kCellBitsF32);
        const int shift = 32 - kCellBitsF32;
        for (uint32_t p = 0; p < lut.size(); ++p) {
            const unsigned a = code_of(s, nb, mag(from_bits(p << shift)));
            const unsigned b = code_of(s, nb, mag(from_bits((p << shift) | ((1u << shift) - 1u))));
            const unsigned lo = a < b ? a : b, hi = a < b ? b : a;
            // a cell that mixes infinity with NaNs (code 0) is dense unless K-1 <= 1
            lut[p] = static_cast<uint8_t>((hi - lo <= 1) ? lo : kCellDense);
        }
        encode_runs(lut, f32_runs);
    }
}

// For a bfloat16 x and any binary32 s:  s < x  <=>  floor_bf16(s) < x, where floor_bf16(s) is the
// largest bfloat16 not above s.  The forward kernel compares two bfloat16 elements per instruction
// against these rounded-down boundaries.
void build_bf16_thresholds(const float *s, uint32_t *s_bf16x2) {
    for (int j = 0; j < kMaxLevels; ++j) {
        uint32_t u;
        std::memcpy(&u, &s[j], 4);
        uint32_t h = u >> 16;
        if ((u & 0xffffu) != 0 && (u >> 31) != 0 && !std::isnan(s[j])) h += 1;   // negative and inexact: one step further from zero
        s_bf16x2[j] = h | (h << 16);
    }
}

// The same for IEEE binary16: the largest binary16 value not above s[j] (by bisection over the
// 63 489 ordered finite-or-infinite patterns; -inf when s[j] is below every finite value).
void build_f16_thresholds(const float *s, uint32_t *s_f16x2) {
    // ordered index k in [0, 2*0x7c00]: k < 0x7c00 -> negative pattern 0x8000 | (0x7c00 - k); else positive pattern k - 0x7c00
    const auto pattern = [](int k) -> uint32_t { return k < 0x7c00 ? (0x8000u | static_cast<uint32_t>(0x7c00 - k)) : static_cast<uint32_t>(k - 0x7c00); };
    for (int j = 0; j < kMaxLevels; ++j) {
        int lo = 0, hi = 2 * 0x7c00;              // pattern(lo) = -inf, pattern(hi) = +inf
        if (std::isnan(s[j]) || !(f16_bits_to_float(pattern(hi)) > s[j])) lo = hi;   // s = +inf (unused slot)
        while (hi - lo > 1) {                    // invariant: value(lo) <= s < value(hi)
            const int mid = (lo + hi) / 2;
            if (f16_bits_to_float(pattern(mid)) <= s[j]) lo = mid; else hi = mid;
        }
        uint32_t h = pattern(lo);
        if (h == 0x8000u) h = 0;                  // -0 and +0 compare equal; keep one pattern
        s_f16x2[j] = h | (h << 16);
    }
}

}  // namespace fewbit

using fewbit::kMaxLevels;

extern "C" {

static fewbit_status solve_into_table(fewbit_act act, int bits, double A, double B, int n_cells, bool folded,
                                      fewbit_table **out, int weight = FEWBIT_WEIGHT_UNIFORM, int finetune_iters = 0) {
    if (out == nullptr) return FEWBIT_ERR_INVALID_ARG;
    *out = nullptr;
    if (!fewbit::valid_act(act) || !fewbit::valid_bits(bits)) return FEWBIT_ERR_INVALID_ARG;
    const int K = 1 << bits;
    if (!(A < B) || !std::isfinite(A) || !std::isfinite(B) || n_cells < K || n_cells > 65536 || finetune_iters < 0 ||
        (weight != FEWBIT_WEIGHT_UNIFORM && weight != FEWBIT_WEIGHT_NORMAL))
        return FEWBIT_ERR_INVALID_ARG;
    try {
        auto g = fewbit::solved_for(act, A, B, n_cells, weight);
        // walk the argmins back from (n, K): right ends of pieces K, K-1, ..., 1
        int ends[kMaxLevels + 1];
        ends[K] = g->n;
        for (int k = K; k >= 1; --k) ends[k - 1] = g->from[k][ends[k]];
        auto *t = new fewbit_table();
        t->act = act;
        t->bits = bits;
        t->folded = folded ? 1 : 0;
        t->objective = (folded ? 2.0 : 1.0) * g->best_at_n[K];     // both half-axes
        for (int m = 0; m < kMaxLevels; ++m) { t->s[m] = std::numeric_limits<float>::infinity(); t->lev[m] = 0.0f; }
        double sd[kMaxLevels], levd[kMaxLevels];
        for (int m = 1; m < K; ++m) {
            const int i = ends[m];
            sd[m - 1] = (i == g->n) ? B : A + (B - A) * (static_cast<double>(i) / g->n);
        }
        for (int m = 0; m < K; ++m) levd[m] = g->level(ends[m], ends[m + 1]);                         // Eq. 4
        if (finetune_iters > 0) {                                                                     // Eq. 5
            const double refined = fewbit::finetune(act, weight, A, B, K, sd, levd, finetune_iters);
            if (!std::isnan(refined)) t->objective = (folded ? 2.0 : 1.0) * refined;
        }
        for (int m = 1; m < K; ++m) t->s[m - 1] = static_cast<float>(sd[m - 1]);
        for (int m = 0; m < K; ++m) t->lev[m] = static_cast<float>(levd[m]);
        fewbit::build_code_runs(t->s, bits, folded, &t->runs_bf16, &t->runs_f32, &t->runs_f16);
        fewbit::build_bf16_thresholds(t->s, t->s_bf16x2);
        fewbit::build_f16_thresholds(t->s, t->s_f16x2);
        *out = t;
        return FEWBIT_OK;
    } catch (const std::bad_alloc &) {
        return FEWBIT_ERR_ALLOC;
    } catch (...) {
        return FEWBIT_ERR_UNSUPPORTED;
    }
}

fewbit_status fewbit_table_create_ex(fewbit_act act, int bits, double A, double B, int n_cells,
                                     fewbit_table **out) {
    return solve_into_table(act, bits, A, B, n_cells, false, out);
}

fewbit_status fewbit_table_create_folded(fewbit_act act, int bits, double B, int n_cells, fewbit_table **out) {
    if (out != nullptr) *out = nullptr;
    if (act != FEWBIT_SIGMOID && act != FEWBIT_TANH) return FEWBIT_ERR_UNSUPPORTED;   // f' must be even
    return solve_into_table(act, bits, 0.0, B, n_cells, true, out);
}

fewbit_status fewbit_table_create_opt(fewbit_act act, int bits, const fewbit_solver_options *opt, fewbit_table **out) {
    if (out != nullptr) *out = nullptr;
    if (opt == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (opt->folded) {
        if (act != FEWBIT_SIGMOID && act != FEWBIT_TANH) return FEWBIT_ERR_UNSUPPORTED;
        if (opt->A != 0.0) return FEWBIT_ERR_INVALID_ARG;
    }
    return solve_into_table(act, bits, opt->A, opt->B, opt->n_cells, opt->folded != 0, out, opt->weight,
                            opt->finetune_iters);
}

int fewbit_table_is_folded(const fewbit_table *table) { return table != nullptr && table->folded; }

fewbit_table *fewbit_table_create(fewbit_act act, int bits) {
    fewbit_table *t = nullptr;
    if (fewbit_table_create_ex(act, bits, -8.0, 8.0, 4096, &t) != FEWBIT_OK) return nullptr;
    return t;
}

fewbit_status fewbit_table_from_arrays(fewbit_act act, int bits, const float *s, const float *lev,
                                       fewbit_table **out) {
    return fewbit_table_from_arrays_ex(act, bits, s, lev, 0, out);
}

fewbit_status fewbit_table_from_arrays_ex(fewbit_act act, int bits, const float *s, const float *lev, int folded,
                                          fewbit_table **out) {
    if (out == nullptr) return FEWBIT_ERR_INVALID_ARG;
    *out = nullptr;
    if (folded && act != FEWBIT_SIGMOID && act != FEWBIT_TANH) return FEWBIT_ERR_UNSUPPORTED;
    if (!fewbit::valid_act(act) || !fewbit::valid_bits(bits) || s == nullptr || lev == nullptr)
        return FEWBIT_ERR_INVALID_ARG;
    const int K = 1 << bits;
    for (int m = 0; m < K - 1; ++m) {
        if (std::isnan(s[m])) return FEWBIT_ERR_INVALID_ARG;
        if (m > 0 && s[m] < s[m - 1]) return FEWBIT_ERR_INVALID_ARG;
    }
    auto *t = new (std::nothrow) fewbit_table();
    if (t == nullptr) return FEWBIT_ERR_ALLOC;
    t->act = act;
    t->bits = bits;
    t->folded = folded ? 1 : 0;
    t->objective = std::numeric_limits<double>::quiet_NaN();
    for (int m = 0; m < kMaxLevels; ++m) { t->s[m] = std::numeric_limits<float>::infinity(); t->lev[m] = 0.0f; }
    // +0 and -0 compare equal; store +0 so that every kernel variant sees one pattern
    for (int m = 0; m < K - 1; ++m) t->s[m] = (s[m] == 0.0f) ? 0.0f : s[m];
    for (int m = 0; m < K; ++m) t->lev[m] = lev[m];
    fewbit::build_code_runs(t->s, bits, folded != 0, &t->runs_bf16, &t->runs_f32, &t->runs_f16);
    fewbit::build_bf16_thresholds(t->s, t->s_bf16x2);
    fewbit::build_f16_thresholds(t->s, t->s_f16x2);
    *out = t;
    return FEWBIT_OK;
}

void fewbit_table_destroy(fewbit_table *table) { delete table; }

fewbit_status fewbit_table_get(const fewbit_table *table, int *act, int *bits, float *s_out,
                               float *lev_out, double *objective) {
    if (table == nullptr) return FEWBIT_ERR_INVALID_ARG;
    const int K = 1 << table->bits;
    if (act) *act = static_cast<int>(table->act);
    if (bits) *bits = table->bits;
    if (s_out) std::memcpy(s_out, table->s, sizeof(float) * (K - 1));
    if (lev_out) std::memcpy(lev_out, table->lev, sizeof(float) * K);
    if (objective) *objective = table->objective;
    return FEWBIT_OK;
}

size_t fewbit_packed_bytes(size_t n, int bits) {
    if (!fewbit::valid_bits(bits)) return 0;
    return 4 * ((n * static_cast<size_t>(bits) + 31) / 32);
}

const char *fewbit_status_string(fewbit_status status) {
    switch (status) {
    case FEWBIT_OK: return "ok";
    case FEWBIT_ERR_INVALID_ARG: return "invalid argument";
    case FEWBIT_ERR_UNSUPPORTED: return "unsupported";
    case FEWBIT_ERR_ALIGNMENT: return "buffer alignment";
    case FEWBIT_ERR_CUDA: return "CUDA error";
    case FEWBIT_ERR_ALLOC: return "allocation failed or workspace too small";
    case FEWBIT_ERR_TOO_LARGE: return "more elements than the fixed staging area of the allocation-free call holds";
    }
    return "unknown status";
}

}  // extern "C"
