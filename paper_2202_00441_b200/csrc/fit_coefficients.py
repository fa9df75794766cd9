"""Reproduces the polynomial coefficients hard-coded in fewbit_math.cuh.

Run by hand (needs numpy and mpmath); prints the constants.  Not used at
build or run time.

1. GELU for bfloat16 and binary16 storage, one exponential and no reciprocal.
   x Phi(x) = max(x,0) - t Phi(-t), t = |x|, and
   t Phi(-t) = t 2^{L(t)},  L(t) = log2 Phi(-t), fitted by a polynomial in s = t / tmax on
   s in [0, 1] (Chebyshev basis, absolute error of L minimised where t Phi(-t) is still
   representable in the storage type, loosely beyond); the kernel evaluates
   s = min(|x|, tmax) / tmax with a saturating multiply.
   bfloat16: tmax = 16, degree 7, accurate up to t = 14.7 (relative error of t Phi(-t) 8.7e-4).
   binary16: tmax = 6, degree 6, accurate up to t = 5.7 (3.4e-5); beyond, t Phi(-t) is below
   half the smallest subnormal.

2. exp for binary32 storage.
   e^r = 1 + r + r^2 Q(r) on |r| <= ln(2)/2, Q of degree 4, relative error of
   e^r minimised the same way on Chebyshev nodes.

3. GELU for binary32 storage.
   Phi(-t) exp(t^2/2) = w G(w),  w = 1/(1 + p t) with p = float32(0.2),  G of
   degree 9 in u = w - 1/2, fitted on t in [0, 15] (w in [1/4, 1]) in the
   Chebyshev basis, relative error minimised; printed as monomials in u with
   the constant term split into a float32 value and the float32 remainder.

4. Softplus for bfloat16 and binary16 storage.
   log(1 + E) = E h(E), h(u) = log(1 + u) / u of degree 5 on u in [0, 1], relative
   error minimised on Chebyshev nodes (8.4e-6).
"""
import mpmath as mp
import numpy as np

mp.mp.dps = 40


def minimax_lstsq(A, target, weight_of_error, iters=60):
    w = np.ones(len(target))
    for _ in range(iters):
        c, *_ = np.linalg.lstsq(A * w[:, None], target * w, rcond=None)
        err = weight_of_error(A @ c - target)
        w = w * (1 + 4 * np.abs(err) / np.abs(err).max())
        w /= w.mean()
    return c, np.abs(err).max()


def fit_gelu_log2(tmax=16.0, deg=7, t_accurate=14.7, nodes=800):
    from numpy.polynomial import chebyshev as C, polynomial as P
    k = np.arange(nodes)
    z = np.cos(np.pi * (k + 0.5) / nodes)
    sv = (z + 1) / 2
    target = np.array([float(mp.log(mp.ncdf(-mp.mpf(tmax * v)), 2)) for v in sv])
    imp = np.where(tmax * sv <= t_accurate, 1.0, 0.02)
    w = np.ones(nodes)
    V = C.chebvander(z, deg)
    for _ in range(60):
        c, *_ = np.linalg.lstsq(V * (w * imp)[:, None], target * w * imp, rcond=None)
        err = (V @ c - target) * imp
        w = w * (1 + 4 * np.abs(err) / np.abs(err).max())
        w /= w.mean()
    mono = np.zeros(1)
    for cf in C.cheb2poly(c)[::-1]:
        mono = P.polyadd(P.polymul(mono, [-1.0, 2.0]), [cf])       # z = 2 s - 1
    return mono, np.abs(err).max()


def fit_exp_f32(deg_q=4):
    half = float(mp.log(2) / 2) * 1.0005
    k = np.arange(400)
    r = half * np.cos(np.pi * (k + 0.5) / 400)
    target = np.array([float((mp.exp(mp.mpf(x)) - 1 - mp.mpf(x)) / mp.mpf(x) ** 2) for x in r])
    A = np.stack([r ** i for i in range(deg_q + 1)], 1)
    return minimax_lstsq(A, target, lambda e: e * r ** 2 / np.exp(r))


def fit_gelu_f32(p=0.2, deg=9, centre=0.5, tmax=15.0, nodes=500):
    from numpy.polynomial import chebyshev as C, polynomial as P
    p = float(np.float32(p))
    wmin = 1 / (1 + p * tmax)
    k = np.arange(nodes)
    z = np.cos(np.pi * (k + 0.5) / nodes)
    w = (z + 1) / 2 * (1 - wmin) + wmin
    t = (1 / w - 1) / p
    g = np.array([float(mp.ncdf(-mp.mpf(tt)) * mp.exp(mp.mpf(tt) ** 2 / 2) / mp.mpf(ww)) for tt, ww in zip(t, w)])
    c, err = minimax_lstsq(C.chebvander(z, deg) / g[:, None], np.ones_like(g), lambda e: e)
    a, b = 2 / (1 - wmin), -(1 + wmin) / (1 - wmin)          # z = a w + b = a u + (a centre + b)
    mono = np.zeros(1)
    for cf in C.cheb2poly(c)[::-1]:
        mono = P.polyadd(P.polymul(mono, [a * centre + b, a]), [cf])
    return mono, err


def fit_softplus_16(deg=5, nodes=600):
    from numpy.polynomial import chebyshev as C, polynomial as P
    k = np.arange(nodes)
    z = np.cos(np.pi * (k + 0.5) / nodes)
    u = (z + 1) / 2
    target = np.array([float(mp.log1p(mp.mpf(v)) / mp.mpf(v)) for v in u])
    V = C.chebvander(z, deg)
    w = np.ones(nodes)
    for _ in range(80):
        c, *_ = np.linalg.lstsq(V * (w / target)[:, None], w, rcond=None)
        err = (V @ c - target) / target
        w = w * (1 + 4 * np.abs(err) / np.abs(err).max())
        w /= w.mean()
    mono = np.zeros(1)
    for cf in C.cheb2poly(c)[::-1]:
        mono = P.polyadd(P.polymul(mono, [-1.0, 2.0]), [cf])       # z = 2 u - 1
    return mono, np.abs(err).max()


if __name__ == "__main__":
    c, err = fit_gelu_log2()
    print("GELU bf16: L(16 s) coefficients (s^0..s^7):", ", ".join("%.9g" % np.float32(v) for v in c),
          "max error of L %.3e" % err)
    c, err = fit_gelu_log2(tmax=6.0, deg=6, t_accurate=5.7)
    print("GELU f16: L(6 s) coefficients (s^0..s^6):", ", ".join("%.9g" % np.float32(v) for v in c),
          "max error of L %.3e" % err)
    g, err = fit_gelu_f32()
    c0 = np.float32(g[0])
    print("GELU f32: p = float32(0.2), G in u = w - 1/2: c0 = %.9g + %.9g, c1..c9 =" % (c0, np.float32(g[0] - float(c0))),
          ", ".join("%.9g" % np.float32(v) for v in g[1:]), "max relative error %.3e" % err)
    q, err = fit_exp_f32()
    print("exp f32: Q coefficients (r^0..r^4):", [float(np.float32(v)) for v in q],
          "max relative error of e^r %.3e (%.3f binary32 ulp)" % (err, err / 2 ** -24))
    # Cody-Waite split of ln 2: the high part keeps 15 significant bits, so n * hi is exact for |n| < 512
    ln2 = mp.log(2)
    bits = np.array([float(ln2)], dtype=np.float32).view(np.uint32) & np.uint32(0xfffffe00)
    hi = float(bits.view(np.float32)[0])
    print("ln 2 split: hi = %.15g, lo = %.15g" % (hi, float(ln2 - mp.mpf(hi))))
    h, err = fit_softplus_16()
    print("softplus 16-bit: h coefficients (u^0..u^5):", ", ".join("%.9g" % np.float32(v) for v in h),
          "max relative error %.3e" % err)
