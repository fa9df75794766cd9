"""Pins for the oracle's table solver (Eq. 3, 4, 5, 7-9) -- CPU only.

Each test ties the oracle to something other than itself: the values the paper
prints (Table 1), exhaustive search, numerical quadrature by scipy, numerical
differentiation by mpmath, closed forms and symmetries.
"""
import itertools
import os

import mpmath as mp
import numpy as np
import pytest
from scipy import integrate

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_error.txt")


def _table1_rows():
    rows = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, fold, *vals = line.split()
            for bits, v in enumerate(vals, 1):
                if v != "-":
                    rows.append((name, int(fold), bits, float(v)))
    return rows


@pytest.mark.parametrize("name,fold,bits,printed", _table1_rows())
def test_table1_values(name, fold, bits, printed):
    """Table 1: the DP optimum on [-10,10] equals every printed error to the
    printed precision (raw integral of Eq. 3, no normalisation)."""
    if fold:
        got = 2.0 * oracle.dp_solve(name, bits, 0.0, 10.0, 2000)["objective"]
    else:
        got = oracle.dp_solve(name, bits, -10.0, 10.0, 4000)["objective"]
    assert abs(got - printed) <= 1.0e-4, (name, bits, got, printed)


# --------------------------------------------------------------------------
# mpmath definitions of f (textbook forms, 40 digits) -- independent of the C
# --------------------------------------------------------------------------
mp.mp.dps = 40
MP_F = {
    "gelu": lambda x: x * mp.ncdf(x),
    "silu": lambda x: x / (1 + mp.exp(-x)),
    "sigmoid": lambda x: 1 / (1 + mp.exp(-x)),
    "tanh": lambda x: mp.tanh(x),
    "elu": lambda x: x if x > 0 else mp.expm1(x),
    "softplus": lambda x: mp.log1p(mp.exp(x)),
    "leaky_relu": lambda x: x if x > 0 else x / 100,
    "relu": lambda x: x if x > 0 else mp.mpf(0),
    "selu": lambda x: mp.mpf("1.0507009873554804934193349852946")
    * (x if x > 0 else mp.mpf("1.6732632423543772848170429916717") * mp.expm1(x)),
}
POINTS = [-30.0, -14.0, -9.5, -6.0, -3.3, -1.0, -0.3, -1e-3, -1e-9, 1e-9, 2e-3, 0.4, 1.0, 2.7, 5.5, 9.0, 20.0, 40.0]


@pytest.mark.parametrize("name", sorted(MP_F))
def test_activation_values_vs_mpmath(name):
    got = oracle.act(name, np.array(POINTS))
    for x, g in zip(POINTS, got):
        ref = MP_F[name](mp.mpf(x))
        # 1e-12 relative is 2^16 times finer than one binary32 ulp; the deep tails
        # (GELU at x = -30) lose a few digits to the rounded argument of erfc
        tol = abs(ref) * mp.mpf(10) ** -12 + mp.mpf(10) ** -320
        assert abs(mp.mpf(float(g)) - ref) <= tol, (name, x, g, ref)


@pytest.mark.parametrize("name", sorted(MP_F))
def test_activation_derivative_vs_numerical_differentiation(name):
    got = oracle.act_deriv(name, np.array(POINTS))
    for x, g in zip(POINTS, got):
        ref = mp.diff(MP_F[name], mp.mpf(x), h=mp.mpf(10) ** -15 * max(1, abs(x)) * mp.mpf("1e-3"))
        assert abs(mp.mpf(float(g)) - ref) <= 1e-12 * max(1, abs(ref)), (name, x, g, ref)


# --------------------------------------------------------------------------
# DP versus exhaustive search
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["gelu", "silu", "sigmoid", "elu", "softplus", "tanh", "selu"])
@pytest.mark.parametrize("n,K", [(10, 2), (12, 3), (12, 4), (16, 4), (16, 5), (20, 4), (14, 8)])
def test_dp_equals_bruteforce(name, n, K):
    """Eq. 7 finds the global minimum of Eq. 3 over the grid (asymmetric range,
    so the optimum is unique)."""
    A, B = -3.0, 5.0
    dp = oracle.dp_solve(name, A=A, B=B, n_cells=n, K=K)
    bf = oracle.bruteforce(name, K, A, B, n)
    assert dp["objective"] == pytest.approx(bf["objective"], abs=1e-15, rel=1e-13)
    assert list(dp["idx"]) == list(bf["idx"])


def test_bruteforce_is_really_exhaustive():
    """The enumerator visits C(n-1, K-1) subsets: check the minimum against a
    Python itertools enumeration scored by the oracle's own Eq. 3 evaluator."""
    name, A, B, n, K = "gelu", -2.0, 3.0, 9, 4
    best = min((oracle.objective(name, c, A, B, n), c)
               for c in itertools.combinations(range(1, n), K - 1))
    bf = oracle.bruteforce(name, K, A, B, n)
    assert tuple(bf["idx"]) == best[1]
    assert bf["objective"] == pytest.approx(best[0], abs=1e-16)


@pytest.mark.parametrize("name", ["gelu", "silu", "sigmoid", "tanh", "elu", "softplus"])
def test_objective_equals_direct_quadrature(name):
    """Eq. 8's prefix form of T(j,i) equals the integral of (f'-q)^2 computed
    bin by bin with scipy's adaptive quadrature, and the levels equal the mean
    of f' over each bin (Eq. 4)."""
    A, B, n, bits = -8.0, 8.0, 512, 3
    r = oracle.dp_solve(name, bits, A, B, n)
    edges = np.concatenate([[A], r["s"], [B]])
    fprime = lambda x: float(oracle.act_deriv(name, np.array([x]))[0])
    total = 0.0
    for m in range(len(edges) - 1):
        a, b = edges[m], edges[m + 1]
        mean, _ = integrate.quad(fprime, a, b, epsabs=1e-13, epsrel=1e-13, limit=200)
        mean /= (b - a)
        assert r["lev"][m] == pytest.approx(mean, abs=1e-11)
        err, _ = integrate.quad(lambda x: (fprime(x) - r["lev"][m]) ** 2, a, b,
                                epsabs=1e-13, epsrel=1e-13, limit=200)
        total += err
    assert r["objective"] == pytest.approx(total, abs=2e-9)


@pytest.mark.parametrize("name", ["gelu", "silu", "sigmoid", "tanh", "elu", "softplus", "selu"])
def test_error_non_increasing_in_pieces(name):
    objs = [oracle.dp_solve(name, A=-8.0, B=8.0, n_cells=256, K=K)["objective"] for K in range(1, 18)]
    for a, b in zip(objs, objs[1:]):
        assert b <= a + 1e-15
    assert objs[-1] < 0.05 * objs[0]


@pytest.mark.parametrize("name,lo", [("relu", 0.0), ("leaky_relu", 0.01)])
def test_one_bit_relu_family_is_exact(name, lo):
    """Sec. 2 (ReLU paragraph): a two-valued derivative needs one bit; the
    table is {boundary 0; levels (lo, 1)} with zero error."""
    r = oracle.dp_solve(name, 1, -8.0, 8.0, 4096)
    assert r["s"][0] == 0.0
    assert r["lev"][0] == pytest.approx(lo, abs=1e-17)
    assert r["lev"][1] == 1.0
    assert abs(r["objective"]) <= 1e-15
    assert np.float32(r["lev"][0]) == np.float32(lo)


@pytest.mark.parametrize("name", ["relu", "leaky_relu"])
@pytest.mark.parametrize("bits", [2, 3, 4])
def test_relu_family_extra_bits_stay_exact(name, bits):
    r = oracle.dp_solve(name, bits, -8.0, 8.0, 4096)
    assert abs(r["objective"]) <= 1e-14
    assert 0.0 in list(r["s"])


@pytest.mark.parametrize("name", ["gelu", "silu", "softplus"])
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_symmetry_of_tables(name, bits):
    """f'(x) + f'(-x) = 1 for these activations, so the optimal table on a
    symmetric range is point-symmetric."""
    r = oracle.dp_solve(name, bits, -8.0, 8.0, 1024)
    s, lev = r["s"], r["lev"]
    np.testing.assert_allclose(s, -s[::-1], atol=0)
    np.testing.assert_allclose(lev + lev[::-1], 1.0, atol=1e-12)


@pytest.mark.parametrize("name", ["gelu", "silu", "sigmoid", "tanh", "softplus"])
@pytest.mark.parametrize("bits", [2, 3])
def test_stationarity_of_boundaries(name, bits):
    """Eq. 5: at an optimum 2 f'(s_i) = y_i + y_{i-1}; on a grid of step h the
    residual is O(h)."""
    n = 4096
    h = 16.0 / n
    r = oracle.dp_solve(name, bits, -8.0, 8.0, n)
    d = oracle.act_deriv(name, r["s"])
    resid = np.abs(2 * d - r["lev"][1:] - r["lev"][:-1])
    assert resid.max() <= 2.0 * h, resid


def test_elu_boundaries_are_negative():
    for bits in (1, 2, 3, 4):
        r = oracle.dp_solve("elu", bits, -8.0, 8.0, 1024)
        assert (r["s"] <= 0).all()
        assert 0.9 < r["lev"][-1] <= 1.0      # last bin = a sliver of e^x plus all of x > 0


def test_config1_table_values():
    """GELU 3-bit on [-8,8], 4096 cells: every boundary is a multiple of 2^-8
    (exact in binary32) and the middle one is 0."""
    r = oracle.dp_solve("gelu", 3, -8.0, 8.0, 4096)
    assert (r["s"] * 256 == np.round(r["s"] * 256)).all()
    assert r["s"][3] == 0.0
    assert (r["s"].astype(np.float32).astype(np.float64) == r["s"]).all()
    assert (np.diff(r["lev"][1:-1]) > 0).all()


# --------------------------------------------------------------------------
# even-derivative fold (caption of Fig. 3)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["sigmoid", "tanh"])
@pytest.mark.parametrize("bits", [1, 2, 3])
def test_folded_table_is_worth_about_one_more_bit(name, bits):
    """2^bits pieces on the half-axis are 2^(bits+1) symmetric pieces on the whole axis: the
    error lies between the unfolded optimum with 2^(bits+1) pieces (nothing symmetric can beat
    it) and the unfolded optimum with 2^bits pieces."""
    folded = oracle.dp_solve_folded(name, bits, 8.0, 512)["objective"]
    same_bits = oracle.dp_solve(name, bits, -8.0, 8.0, 1024)["objective"]
    one_more = oracle.dp_solve(name, bits + 1, -8.0, 8.0, 1024)["objective"]
    assert one_more - 1e-12 <= folded < same_bits
    assert folded < 0.6 * same_bits


@pytest.mark.parametrize("name", ["sigmoid", "tanh"])
def test_folded_levels_are_means_over_the_half_axis_bins(name):
    r = oracle.dp_solve_folded(name, 2, 8.0, 2048)
    edges = np.concatenate([[0.0], r["s"], [8.0]])
    assert (r["s"] > 0).all()
    for m in range(4):
        a, b = edges[m], edges[m + 1]
        mean = (float(MP_F[name](mp.mpf(b))) - float(MP_F[name](mp.mpf(a)))) / (b - a)
        assert r["lev"][m] == pytest.approx(mean, abs=1e-12)


# --------------------------------------------------------------------------
# normal weight (named under Eq. 3) and gradient fine-tuning (Eq. 5)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["gelu", "sigmoid", "elu"])
def test_normal_weight_levels_and_objective_by_quadrature(name):
    """Eq. 4 and Eq. 3 with w = standard normal density cut to [A,B], against scipy."""
    A, B, n, bits = -6.0, 6.0, 768, 2
    r = oracle.dp_solve(name, bits, A, B, n, weight="normal")
    edges = np.concatenate([[A], r["s"], [B]])
    fprime = lambda x: float(oracle.act_deriv(name, np.array([x]))[0])
    pdf = lambda x: float(np.exp(-0.5 * x * x) / np.sqrt(2 * np.pi))
    total = 0.0
    for m in range(len(edges) - 1):
        a, b = edges[m], edges[m + 1]
        num, _ = integrate.quad(lambda x: fprime(x) * pdf(x), a, b, epsabs=1e-14, epsrel=1e-13, limit=200)
        den, _ = integrate.quad(pdf, a, b, epsabs=1e-14, epsrel=1e-13, limit=200)
        assert r["lev"][m] == pytest.approx(num / den, abs=1e-10)
        err, _ = integrate.quad(lambda x: (fprime(x) - r["lev"][m]) ** 2 * pdf(x), a, b, epsabs=1e-14, epsrel=1e-13, limit=200)
        total += err
    assert r["objective"] == pytest.approx(total, abs=1e-10)


@pytest.mark.parametrize("name", ["gelu", "silu", "tanh"])
@pytest.mark.parametrize("n,K", [(12, 3), (16, 4), (14, 5)])
def test_normal_weight_dp_equals_bruteforce(name, n, K):
    dp = oracle.dp_solve(name, A=-3.0, B=4.0, n_cells=n, K=K, weight="normal")
    bf = oracle.bruteforce(name, K, -3.0, 4.0, n, weight="normal")
    assert dp["objective"] == pytest.approx(bf["objective"], abs=1e-16, rel=1e-13)
    assert list(dp["idx"]) == list(bf["idx"])


def test_normal_weight_moves_the_table_towards_the_origin():
    """With most of the weight near 0 the outer boundaries move inwards and the weighted error
    is far below the uniform-weight error (which pays for the whole of [-8,8])."""
    u = oracle.dp_solve("gelu", 3)
    w = oracle.dp_solve("gelu", 3, weight="normal")
    assert abs(w["s"][0]) < abs(u["s"][0]) and abs(w["s"][-1]) < abs(u["s"][-1])
    assert w["objective"] < 0.25 * u["objective"]
    np.testing.assert_allclose(w["s"], -w["s"][::-1], atol=0)


@pytest.mark.parametrize("weight", ["uniform", "normal"])
@pytest.mark.parametrize("name", ["gelu", "silu", "sigmoid", "softplus"])
def test_eq5_gradient_equals_finite_differences(name, weight):
    rng = np.random.default_rng(5)
    s = np.sort(rng.uniform(-3, 3, 7))
    _, _, grad = oracle.loss_at(name, s, -8.0, 8.0, weight)
    for i in range(s.size):
        h = 1e-4                     # truncation ~1e-9; below that the quadrature's own 1e-13 noise / h takes over
        sp, sm = s.copy(), s.copy()
        sp[i] += h
        sm[i] -= h
        fd = (oracle.loss_at(name, sp, -8.0, 8.0, weight)[0] - oracle.loss_at(name, sm, -8.0, 8.0, weight)[0]) / (2 * h)
        assert grad[i] == pytest.approx(fd, abs=1e-8), (name, weight, i)


def test_loss_at_grid_points_equals_the_dp_objective():
    r = oracle.dp_solve("silu", 3, -8.0, 8.0, 1024)
    val, lev, _ = oracle.loss_at("silu", r["s"])
    assert val == pytest.approx(r["objective"], abs=1e-12)
    np.testing.assert_allclose(lev, r["lev"], atol=1e-12)


@pytest.mark.parametrize("weight", ["uniform", "normal"])
@pytest.mark.parametrize("name", ["gelu", "silu", "tanh", "softplus"])
def test_finetuning_reaches_a_stationary_point_below_the_dp_value(name, weight):
    """Sec. 3: the DP result is a starting point for gradient methods.  After fine-tuning Eq. 5
    vanishes (2 f'(s_i) = y_i + y_{i-1} to 1e-6 instead of O(h) = 4e-3) and the error is not larger."""
    r = oracle.dp_solve(name, 3, weight=weight)
    ft = oracle.finetune(name, r["s"], weight=weight)
    assert ft["objective"] <= r["objective"] + 1e-15
    assert np.abs(ft["s"] - r["s"]).max() < 2 * 16.0 / 4096        # stays within two grid cells
    d = oracle.act_deriv(name, ft["s"])
    resid = np.abs(2 * d - ft["lev"][1:] - ft["lev"][:-1])
    assert resid.max() < 1e-6, resid
    assert (np.diff(ft["s"]) > 0).all()
