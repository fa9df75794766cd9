"""Pins for the oracle's forward / backward halves (Listing 1) -- CPU only.

The oracle is checked against library routines and exact arithmetic that it
does not itself use: numpy.searchsorted, numpy.packbits, Python Fractions,
mpmath at 40 digits, numpy's IEEE binary32 multiply.
"""
from fractions import Fraction

import mpmath as mp
import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(1234)


def bf16_bits_to_f32(h):
    return (np.asarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def all_finite_bf16():
    h = np.arange(65536, dtype=np.uint16)
    f = bf16_bits_to_f32(h)
    keep = np.isfinite(f)
    return h[keep], f[keep]


# --------------------------------------------------------------------------
# rounding to bfloat16
# --------------------------------------------------------------------------
def _exact_rne_bf16(d: float) -> int:
    """Nearest bfloat16 (ties to even mantissa) by exact rational arithmetic
    over the full list of finite bfloat16 values."""
    vals = _exact_rne_bf16.vals
    if d == 0:
        return 0x8000 if np.signbit(d) else 0
    x = Fraction(d)
    sign = 0x8000 if x < 0 else 0
    x = abs(x)
    lo, hi = 0, len(vals) - 1           # vals: non-negative finite bf16 as Fractions, index = bit pattern
    if x >= vals[hi]:
        top = vals[hi]
        step = top - vals[hi - 1]
        return sign | (0x7f80 if x >= top + step / 2 else hi)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if vals[mid] <= x:
            lo = mid
        else:
            hi = mid
    dl, dh = x - vals[lo], vals[hi] - x
    if dl < dh:
        return sign | lo
    if dh < dl:
        return sign | hi
    return sign | (lo if lo % 2 == 0 else hi)


_exact_rne_bf16.vals = [Fraction(float(v)) for v in bf16_bits_to_f32(np.arange(0x7f80, dtype=np.uint16))]


def test_bf16_rounding_against_exact_rationals():
    xs = np.concatenate([
        RNG.standard_normal(2000) * 3,
        RNG.standard_normal(500) * 1e-39,          # subnormal bf16 range
        RNG.standard_normal(500) * 1e38,           # near overflow
        10.0 ** RNG.uniform(-45, 39, 1000) * RNG.choice([-1, 1], 1000),
    ])
    # exact midpoints between neighbouring bf16 values, and their f64 neighbours
    h = RNG.integers(0, 0x7f7f, 600).astype(np.uint16)
    a = bf16_bits_to_f32(h).astype(np.float64)
    b = bf16_bits_to_f32(h + 1).astype(np.float64)
    mids = (a + b) / 2
    xs = np.concatenate([xs, mids, -mids, np.nextafter(mids, 1e300), np.nextafter(mids, -1e300),
                         [0.0, -0.0, 3.3895313892515355e38, 3.39e38, 3.4e38, -3.4e38, 1e-41, 4.5e-41, 4.6e-41]])
    got = oracle.f64_to_bf16(xs)
    for x, g in zip(xs, got):
        assert int(g) == _exact_rne_bf16(float(x)), (x, hex(int(g)))


def test_bf16_rounding_is_identity_on_bf16_values():
    h = np.arange(65536, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        f = bf16_bits_to_f32(h).astype(np.float64)
    got = oracle.f64_to_bf16(f)
    nan = np.isnan(f)
    assert (got[~nan] == h[~nan]).all()
    assert (got[nan] == 0x7fc0).all()
    np.testing.assert_array_equal(oracle.bf16_to_f64(h[~nan]), f[~nan])


# --------------------------------------------------------------------------
# bucketize (Eq. 2 / the sorted search of Listing 1)
# --------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_bucketize_equals_searchsorted_left(bits):
    K = 1 << bits
    s = np.sort(RNG.standard_normal(K - 1)).astype(np.float32)
    near = np.concatenate([s, np.nextafter(s, np.float32(np.inf)), np.nextafter(s, np.float32(-np.inf))])
    x = np.concatenate([RNG.standard_normal(5000).astype(np.float32) * 2, near,
                        np.array([0.0, -0.0, np.inf, -np.inf, 1e30, -1e30], dtype=np.float32)])
    _, packed = oracle.fwd("gelu", bits, s, x)
    codes = oracle.unpack(packed, bits, x.size)
    np.testing.assert_array_equal(codes, np.searchsorted(s, x, side="left"))


def test_bucketize_bf16_all_patterns():
    s = np.array([-2.390625, -0.7109375, -0.328125, 0.0, 0.328125, 0.7109375, 2.390625], dtype=np.float32)
    h, f = all_finite_bf16()
    _, packed = oracle.fwd("gelu", 3, s, h)
    np.testing.assert_array_equal(oracle.unpack(packed, 3, h.size), np.searchsorted(s, f, side="left"))


def test_nan_input_maps_to_code_zero():
    s = np.array([-1.0, 0.0, 1.0], dtype=np.float32)
    x = np.array([np.nan, 0.5], dtype=np.float32)
    _, packed = oracle.fwd("tanh", 2, s, x)
    assert list(oracle.unpack(packed, 2, 2)) == [0, 2]


def test_tie_goes_to_lower_bin():
    """x == s_j belongs to the bin on the left, so that a 1-bit ReLU-type
    table gives the framework's derivative at 0 (slope, not 1)."""
    s = np.array([0.0], dtype=np.float32)
    x = np.array([0.0, -0.0, np.float32(1e-45), -np.float32(1e-45)], dtype=np.float32)
    _, packed = oracle.fwd("leaky_relu", 1, s, x)
    assert list(oracle.unpack(packed, 1, 4)) == [0, 0, 1, 0]


# --------------------------------------------------------------------------
# bit stream layout
# --------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_pack_equals_numpy_packbits_little(bits):
    for n in list(range(0, 131)) + [1000, 4099]:
        codes = RNG.integers(0, 1 << bits, n).astype(np.uint8)
        packed = oracle.pack(codes, bits)
        assert packed.size == (n * bits + 31) // 32
        bit_matrix = ((codes[:, None] >> np.arange(bits)[None, :]) & 1).astype(np.uint8).reshape(-1)
        ref_bytes = np.packbits(bit_matrix, bitorder="little")
        ref = np.zeros(packed.size * 4, dtype=np.uint8)
        ref[:ref_bytes.size] = ref_bytes
        np.testing.assert_array_equal(packed, ref.view("<u4"))
        np.testing.assert_array_equal(oracle.unpack(packed, bits, n), codes)


def test_one_bit_stream_is_the_integer_sum():
    codes = RNG.integers(0, 2, 32).astype(np.uint8)
    assert int(oracle.pack(codes, 1)[0]) == sum(int(c) << e for e, c in enumerate(codes))


def test_three_bit_codes_straddle_words():
    codes = np.zeros(32, dtype=np.uint8)
    codes[10] = 0b101          # bits 30..32: two in word 0, one in word 1
    p = oracle.pack(codes, 3)
    assert p.size == 3 and int(p[0]) == (0b01 << 30) and int(p[1]) == 0b1 and int(p[2]) == 0


def test_padding_bits_are_zero():
    for bits in (1, 2, 3, 4):
        n = 2 ** 10 + 7
        x = (RNG.standard_normal(n) * 50).astype(np.float32)
        s = np.full((1 << bits) - 1, -1e30, dtype=np.float32)   # every code = K-1 (all ones)
        _, packed = oracle.fwd("tanh", bits, s, x)
        used = n * bits
        last = int(packed[-1])
        tail_bits = used - 32 * (packed.size - 1)
        assert last == (1 << tail_bits) - 1


# --------------------------------------------------------------------------
# forward values
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
}


def _ordered(bits, width):
    bits = bits.astype(np.int64)
    sign = 1 << (width - 1)
    return np.where(bits & sign, -(bits & (sign - 1)), bits)


@pytest.mark.parametrize("name", sorted(MP_F))
def test_forward_f32_is_the_rounded_exact_value(name):
    x = np.concatenate([RNG.standard_normal(300) * 2, -np.abs(RNG.standard_normal(100)) * 6,
                        [-14.0, -13.2, -9.0, 1e-20, -1e-20, 30.0, 88.0, -88.0]]).astype(np.float32)
    y, _ = oracle.fwd(name, 1, np.zeros(1, np.float32), x)
    ref = np.array([float(MP_F[name](mp.mpf(float(v)))) for v in x]).astype(np.float32)
    d = np.abs(_ordered(y.view(np.uint32), 32) - _ordered(ref.view(np.uint32), 32))
    assert d.max() <= 1 and (d == 0).mean() > 0.99, (name, d.max())


@pytest.mark.parametrize("name", sorted(MP_F))
def test_forward_bf16_is_the_rounded_exact_value(name):
    h = RNG.integers(0, 65536, 600).astype(np.uint16)
    h = h[np.isfinite(bf16_bits_to_f32(h))]
    y, _ = oracle.fwd(name, 1, np.zeros(1, np.float32), h)
    for hv, yv in zip(h, y):
        xv = float(bf16_bits_to_f32(np.array([hv]))[0])
        exact = MP_F[name](mp.mpf(xv))
        # rounding the 40-digit value through binary64 cannot move it across a
        # bf16 rounding boundary except on an exact tie, which these inputs avoid
        assert int(yv) == _exact_rne_bf16(float(exact)) or abs(exact) < mp.mpf(2) ** -140, (name, xv)


# --------------------------------------------------------------------------
# backward
# --------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_backward_f32_is_one_ieee_multiply(bits):
    K = 1 << bits
    n = 4099
    lev = RNG.standard_normal(K).astype(np.float32)
    codes = RNG.integers(0, K, n).astype(np.uint8)
    g = (RNG.standard_normal(n) * 10.0 ** RNG.uniform(-42, 3, n)).astype(np.float32)
    got = oracle.bwd(bits, lev, oracle.pack(codes, bits), g)
    ref = g * lev[codes]                      # numpy binary32 multiply
    np.testing.assert_array_equal(got.view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("bits", [1, 3])
def test_backward_bf16_multiplies_in_f32_then_rounds_once(bits):
    K = 1 << bits
    n = 3001
    lev = RNG.standard_normal(K).astype(np.float32)
    codes = RNG.integers(0, K, n).astype(np.uint8)
    gh = RNG.integers(0, 65536, n).astype(np.uint16)
    gh = np.where(np.isfinite(bf16_bits_to_f32(gh)), gh, 0x3f80).astype(np.uint16)
    got = oracle.bwd(bits, lev, oracle.pack(codes, bits), gh)
    prod = bf16_bits_to_f32(gh) * lev[codes]
    for p, o in zip(prod, got):
        assert int(o) == _exact_rne_bf16(float(p))


def test_backward_relu_family_equals_exact_derivative():
    """Sec. 2: with a 1-bit ReLU-type table the backward pass is the exact
    chain rule (Eq. 1), including at x = 0."""
    r = oracle.dp_solve("leaky_relu", 1)
    s, lev = r["s"].astype(np.float32), r["lev"].astype(np.float32)
    x = np.concatenate([RNG.standard_normal(5000), [0.0, -0.0]]).astype(np.float32)
    g = RNG.standard_normal(x.size).astype(np.float32)
    y, packed = oracle.fwd("leaky_relu", 1, s, x)
    gi = oracle.bwd(1, lev, packed, g)
    np.testing.assert_array_equal(gi, g * np.where(x > 0, np.float32(1.0), np.float32(0.01)))
    np.testing.assert_array_equal(y, np.where(x > 0, x, (0.01 * x.astype(np.float64)).astype(np.float32)))


def test_backward_applies_the_piecewise_constant_function():
    """Eq. 2: the factor applied to grad_out is q(x | s, y)."""
    r = oracle.dp_solve("silu", 2)
    s, lev = r["s"].astype(np.float32), r["lev"].astype(np.float32)
    x = (RNG.standard_normal(4000) * 1.5).astype(np.float32)
    g = np.ones_like(x)
    _, packed = oracle.fwd("silu", 2, s, x)
    gi = oracle.bwd(2, lev, packed, g)
    q = lev[np.searchsorted(s, x, side="left")]
    np.testing.assert_array_equal(gi, q)
    # and q tracks f' with the error the table promises (mean square under N(0,1.5^2) is small)
    assert np.mean((gi - oracle.act_deriv("silu", x)) ** 2) < 0.02


# --------------------------------------------------------------------------
# even-derivative fold
# --------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [1, 2, 4])
def test_folded_bucketize_is_searchsorted_of_abs(bits):
    r = oracle.dp_solve_folded("tanh", bits)
    s, lev = r["s"].astype(np.float32), r["lev"].astype(np.float32)
    x = np.concatenate([RNG.standard_normal(4000) * 2, s, -s, np.nextafter(s, np.float32(9)), -np.nextafter(s, np.float32(9)),
                        [0.0, -0.0, np.inf, -np.inf, np.nan]]).astype(np.float32)
    _, packed = oracle.fwd("tanh", bits, s, x, fold=True)
    codes = oracle.unpack(packed, bits, x.size)
    with np.errstate(invalid="ignore"):
        ref = np.searchsorted(s, np.abs(x), side="left")
    ref[np.isnan(x)] = 0
    np.testing.assert_array_equal(codes, ref)
    # the factor applied in the backward pass is an even function of x
    gi = oracle.bwd(bits, lev, packed, np.ones_like(x))
    _, packed_neg = oracle.fwd("tanh", bits, s, -x, fold=True)
    np.testing.assert_array_equal(gi, oracle.bwd(bits, lev, packed_neg, np.ones_like(x)))
    h, f = all_finite_bf16()
    _, pb = oracle.fwd("tanh", bits, s, h, fold=True)
    np.testing.assert_array_equal(oracle.unpack(pb, bits, h.size), np.searchsorted(s, np.abs(f), side="left"))


# --------------------------------------------------------------------------
# IEEE binary16 storage
# --------------------------------------------------------------------------
def test_f16_rounding_against_numpy_and_exact_rationals():
    """numpy converts binary64 -> float16 with one correct rounding; ties and the subnormal /
    overflow edges are checked against exact rational arithmetic as well."""
    xs = np.concatenate([RNG.standard_normal(20000) * 3, RNG.standard_normal(5000) * 1e-6, RNG.standard_normal(5000) * 3e4,
                         10.0 ** RNG.uniform(-9, 5, 5000) * RNG.choice([-1, 1], 5000)])
    allh = np.arange(0x7c00, dtype=np.uint16).view(np.float16).astype(np.float64)
    mids = (allh[:-1] + allh[1:]) / 2                       # every tie between neighbouring finite values
    xs = np.concatenate([xs, mids, -mids, np.nextafter(mids, 1e9), np.nextafter(mids, -1e9),
                         [0.0, -0.0, 65504.0, 65519.99, 65520.0, 1e9, -1e9, 2.0 ** -25, 2.0 ** -25 * 1.0000001, np.inf, -np.inf]])
    with np.errstate(over="ignore"):
        ref = xs.astype(np.float16)
    got = oracle.f64_to_f16(xs)
    np.testing.assert_array_equal(got.view(np.uint16), ref.view(np.uint16))
    vals = [Fraction(float(v)) for v in allh]
    for x, g in zip(mids[::97], oracle.f64_to_f16(mids[::97]).view(np.uint16)):
        lo = int(np.searchsorted(allh, x, side="right")) - 1
        assert vals[lo] < Fraction(float(x)) < vals[lo + 1] and Fraction(float(x)) - vals[lo] == vals[lo + 1] - Fraction(float(x))
        assert int(g) == (lo if lo % 2 == 0 else lo + 1)     # tie -> even pattern


def test_f16_forward_and_backward_follow_the_same_rules():
    h = np.arange(65536, dtype=np.uint16).view(np.float16)
    f = h.astype(np.float32)
    fin = np.isfinite(f)
    s = np.array([-2.390625, -0.7109375, -0.328125, 0.0, 0.328125, 0.7109375, 2.390625], dtype=np.float32)
    y, packed = oracle.fwd("gelu", 3, s, h)
    assert y.dtype == np.float16
    np.testing.assert_array_equal(oracle.unpack(packed, 3, h.size)[fin], np.searchsorted(s, f[fin], side="left"))
    ref = np.array([float(MP_F["gelu"](mp.mpf(float(v)))) for v in f[fin][::37]])
    with np.errstate(over="ignore"):
        np.testing.assert_array_equal(y[fin][::37].view(np.uint16), ref.astype(np.float16).view(np.uint16))
    lev = RNG.standard_normal(8).astype(np.float32)
    g = (RNG.standard_normal(h.size) * 10.0 ** RNG.uniform(-7, 4, h.size)).astype(np.float16)
    gi = oracle.bwd(3, lev, packed, g)
    codes = oracle.unpack(packed, 3, h.size)
    with np.errstate(over="ignore"):
        ref_gi = (g.astype(np.float32) * lev[codes]).astype(np.float64).astype(np.float16)
    np.testing.assert_array_equal(gi.view(np.uint16), ref_gi.view(np.uint16))


# --------------------------------------------------------------------------
# bias add in front of the activation
# --------------------------------------------------------------------------
def _rne_to_grid(value: Fraction, grid_vals, grid_bits):
    """Round an exact rational to the nearest value of a sorted list of representable numbers
    (ties to the even bit pattern); returns the bit pattern.  Written from the definition."""
    lo, hi = 0, len(grid_vals) - 1
    if value <= grid_vals[0]:
        return grid_bits[0]
    if value >= grid_vals[-1]:
        return grid_bits[-1]
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if grid_vals[mid] <= value:
            lo = mid
        else:
            hi = mid
    dl, dh = value - grid_vals[lo], grid_vals[hi] - value
    if dl != dh:
        return grid_bits[lo] if dl < dh else grid_bits[hi]
    return grid_bits[lo] if grid_bits[lo] % 2 == 0 else grid_bits[hi]


def test_bias_add_f32_is_numpy_single_precision_addition():
    rows, cols = 37, 64
    x = (RNG.standard_normal((rows, cols)) * 10.0 ** RNG.uniform(-20, 20, (rows, cols))).astype(np.float32)
    b = (RNG.standard_normal(cols) * 10.0 ** RNG.uniform(-20, 20, cols)).astype(np.float32)
    x[0, :6] = [0.0, -0.0, np.inf, -np.inf, 1e-45, 3e38]
    b[:6] = [-0.0, -0.0, -np.inf, 1.0, -1e-45, 3e38]
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x + b[None, :]                                  # IEEE binary32 addition, one rounding
    got = oracle.bias_add(x, b)
    ok = ~np.isnan(ref)
    np.testing.assert_array_equal(got.view(np.uint32)[ok], ref.view(np.uint32)[ok])
    assert np.isnan(got[~ok]).all()
    # the flat layout is the same thing
    np.testing.assert_array_equal(oracle.bias_add(x.reshape(-1), b).view(np.uint32)[ok.reshape(-1)],
                                  ref.reshape(-1).view(np.uint32)[ok.reshape(-1)])


def test_bias_add_f16_is_numpy_half_precision_addition_and_the_exact_sum_rounded_once():
    rows, cols = 64, 1024
    x = (RNG.standard_normal((rows, cols)) * 10.0 ** RNG.uniform(-6, 4, (rows, cols))).astype(np.float16)
    b = (RNG.standard_normal(cols) * 10.0 ** RNG.uniform(-6, 4, cols)).astype(np.float16)
    with np.errstate(over="ignore", invalid="ignore"):
        ref = x + b[None, :]
    got = oracle.bias_add(x, b)
    ok = ~np.isnan(ref)
    np.testing.assert_array_equal(got.view(np.uint16)[ok], ref.view(np.uint16)[ok])
    # exact rationals on a subset, ties included: 1 + 2^-11 is half way between two float16 values
    allh = np.arange(0x7c00, dtype=np.uint16)
    vals = [Fraction(float(v)) for v in allh.view(np.float16)]
    grid_vals = [-v for v in vals[:0:-1]] + vals
    grid_bits = [int(h) | 0x8000 for h in allh[:0:-1]] + [int(h) for h in allh]
    xs = np.array([1.0, 1.0, 2048.0, -1.0, 6.1e-5, 0.333], dtype=np.float16)
    bs = np.array([2.0 ** -11, 3 * 2.0 ** -11, 1.0, 2.0 ** -11, 5.96e-8, 0.667], dtype=np.float16)
    for xv, bv in zip(xs, bs):
        z = oracle.bias_add(np.array([xv]), np.array([bv]))
        want = _rne_to_grid(Fraction(float(xv)) + Fraction(float(bv)), grid_vals, grid_bits)
        assert int(z.view(np.uint16)[0]) == want, (xv, bv)


def test_bias_add_bf16_is_the_exact_sum_rounded_once():
    allh = np.arange(0x7f80, dtype=np.uint16)                # non-negative finite bfloat16 patterns
    vals = [Fraction(float(v)) for v in bf16_bits_to_f32(allh)]
    grid_vals = [-v for v in vals[:0:-1]] + vals
    grid_bits = [int(h) | 0x8000 for h in allh[:0:-1]] + [int(h) for h in allh]
    n = 600
    xb = RNG.integers(0x3000, 0x4800, n).astype(np.uint16) | (RNG.integers(0, 2, n).astype(np.uint16) << 15)
    bb = RNG.integers(0x3000, 0x4800, n).astype(np.uint16) | (RNG.integers(0, 2, n).astype(np.uint16) << 15)
    # ties: 1 + 2^-8 lies half way between 1 and the next bfloat16; and a pair 30 binades apart
    xb[:4] = [0x3f80, 0x3f80, 0xbf80, 0x4e80]
    bb[:4] = [0x3b80, 0x3c40, 0x3b80, 0x3f80]
    got = oracle.bias_add(xb, bb)                             # one row, n columns
    for i in range(n):
        exact = Fraction(float(bf16_bits_to_f32(xb[i:i + 1])[0])) + Fraction(float(bf16_bits_to_f32(bb[i:i + 1])[0]))
        want = _rne_to_grid(exact, grid_vals, grid_bits)
        if exact == 0:
            assert int(got[i]) & 0x7fff == 0
        else:
            assert int(got[i]) == want, (hex(xb[i]), hex(bb[i]))
    # broadcasting over rows: every row gets the same bias
    x2 = np.tile(xb, (3, 1))
    np.testing.assert_array_equal(oracle.bias_add(x2, bb), np.tile(got, (3, 1)))
    # and it equals binary32 addition followed by one rounding to bfloat16 (no double-rounding case exists)
    f = bf16_bits_to_f32(xb) + bf16_bits_to_f32(bb)
    np.testing.assert_array_equal(oracle.f64_to_bf16(f.astype(np.float64)), got)
