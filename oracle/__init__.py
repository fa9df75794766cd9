"""Few-Bit Backward reference oracle -- TEST INFRASTRUCTURE, not the product.

A ctypes view of ``fewbit_oracle.c`` (plain C, binary64 arithmetic, written
from the paper).  Only the tests, the smoke check and the benchmark's CPU
baseline may import this package; the CUDA library never does and shares no
code with it.

The shared object is compiled with ``gcc -O2 -ffp-contract=off`` (no fused
multiply-add contraction, no fast-math) the first time it is needed.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fewbit_oracle.c")
_LIB = os.path.join(_HERE, "libfewbit_oracle.so")

ACTS = {
    "gelu": 0, "silu": 1, "sigmoid": 2, "tanh": 3, "elu": 4, "softplus": 5,
    "leaky_relu": 6, "relu": 7, "selu": 8,
}

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call([
            "gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
            "-D_GNU_SOURCE", "-o", tmp, _SRC, "-lm",
        ])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        c_dp = ctypes.POINTER(ctypes.c_double)
        c_ip = ctypes.POINTER(ctypes.c_int)
        vp = ctypes.c_void_p
        sz = ctypes.c_size_t
        lib.fbo_act.restype = ctypes.c_double
        lib.fbo_act.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.fbo_act_deriv.restype = ctypes.c_double
        lib.fbo_act_deriv.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.fbo_dp_solve.restype = ctypes.c_int
        lib.fbo_dp_solve.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                     ctypes.c_int, c_dp, c_dp, c_dp, c_ip]
        lib.fbo_objective.restype = ctypes.c_int
        lib.fbo_objective.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                      ctypes.c_int, c_ip, c_dp]
        lib.fbo_bruteforce.restype = ctypes.c_int
        lib.fbo_bruteforce.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                       ctypes.c_int, c_ip, c_dp]
        lib.fbo_dp_solve_w.restype = ctypes.c_int
        lib.fbo_dp_solve_w.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, c_dp, c_dp, c_dp, c_ip]
        lib.fbo_bruteforce_w.restype = ctypes.c_int
        lib.fbo_bruteforce_w.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, c_ip, c_dp]
        lib.fbo_loss_at.restype = ctypes.c_double
        lib.fbo_loss_at.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                    c_dp, c_dp, c_dp]
        lib.fbo_finetune.restype = ctypes.c_int
        lib.fbo_finetune.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                     c_dp, ctypes.c_int, c_dp, c_dp]
        lib.fbo_packed_words.restype = sz
        lib.fbo_packed_words.argtypes = [sz, ctypes.c_int]
        lib.fbo_pack.restype = None
        lib.fbo_pack.argtypes = [ctypes.c_int, vp, vp, sz]
        lib.fbo_unpack.restype = None
        lib.fbo_unpack.argtypes = [ctypes.c_int, vp, vp, sz]
        for name in ("fbo_fwd_f32", "fbo_fwd_bf16"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, sz]
        for name in ("fbo_fwd_f32_fold", "fbo_fwd_bf16_fold", "fbo_fwd_f16_fold"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, sz]
        for name in ("fbo_bwd_f32", "fbo_bwd_bf16", "fbo_bwd_f16"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [ctypes.c_int, vp, vp, vp, vp, sz]
        for name in ("fbo_act_array", "fbo_act_deriv_array"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [ctypes.c_int, vp, vp, sz]
        lib.fbo_f64_to_bf16_array.restype = None
        lib.fbo_f64_to_bf16_array.argtypes = [vp, vp, sz]
        lib.fbo_f64_to_f16_array.restype = None
        lib.fbo_f64_to_f16_array.argtypes = [vp, vp, sz]
        for name in ("fbo_bias_add_f32", "fbo_bias_add_bf16", "fbo_bias_add_f16"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [vp, vp, sz, sz, vp]
        _lib = lib
        return lib


def _act_id(act) -> int:
    return ACTS[act] if isinstance(act, str) else int(act)


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


# ----------------------------------------------------------------------------
# activations (binary64)
# ----------------------------------------------------------------------------
def act(name, x) -> np.ndarray:
    """f(x) in binary64 (Sec. 2)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    _load().fbo_act_array(_act_id(name), _ptr(x), _ptr(y), x.size)
    return y


def act_deriv(name, x) -> np.ndarray:
    """f'(x) in binary64 (Eq. 1)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    _load().fbo_act_deriv_array(_act_id(name), _ptr(x), _ptr(y), x.size)
    return y


def f64_to_bf16(x) -> np.ndarray:
    """binary64 -> bfloat16 bit patterns (uint16), one round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty(x.shape, dtype=np.uint16)
    _load().fbo_f64_to_bf16_array(_ptr(x), _ptr(y), x.size)
    return y


def f64_to_f16(x) -> np.ndarray:
    """binary64 -> IEEE binary16 (numpy float16), one round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty(x.shape, dtype=np.uint16)
    _load().fbo_f64_to_f16_array(_ptr(x), _ptr(y), x.size)
    return y.view(np.float16)


def bf16_to_f64(h) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.uint16)
    return (h.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ----------------------------------------------------------------------------
# tables (Eq. 3, 4, 7-9)
# ----------------------------------------------------------------------------
WEIGHTS = {"uniform": 0, "normal": 1}


def dp_solve(name, bits=None, A=-8.0, B=8.0, n_cells=4096, K=None, weight="uniform"):
    """Optimal K-piece constant approximation of f' on the grid (Eq. 7).

    ``weight``: "uniform" (Eq. 10 on [A,B]) or "normal" (standard normal
    density cut to [A,B]).  Returns a dict with ``s`` (K-1 boundaries, f64),
    ``lev`` (K levels, f64), ``idx`` (grid indices of the boundaries) and
    ``objective`` (Eq. 3)."""
    if K is None:
        K = 1 << int(bits)
    s = np.zeros(max(K - 1, 1), dtype=np.float64)
    lev = np.zeros(K, dtype=np.float64)
    idx = np.zeros(max(K - 1, 1), dtype=np.int32)
    obj = ctypes.c_double(0.0)
    rc = _load().fbo_dp_solve_w(
        _act_id(name), float(A), float(B), int(n_cells), int(K), WEIGHTS[weight],
        s.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
        lev.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
        ctypes.byref(obj),
        idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int)))
    if rc != 0:
        raise ValueError(f"fbo_dp_solve failed with {rc}")
    return {"s": s[:K - 1].copy(), "lev": lev, "idx": idx[:K - 1].copy(), "objective": obj.value}


def objective(name, idx, A, B, n_cells) -> float:
    """Eq. 3 for boundaries at the grid indices ``idx`` (levels by Eq. 4)."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    K = idx.size + 1
    obj = ctypes.c_double(0.0)
    rc = _load().fbo_objective(_act_id(name), float(A), float(B), int(n_cells), K,
                               idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), ctypes.byref(obj))
    if rc != 0:
        raise ValueError(f"fbo_objective failed with {rc}")
    return obj.value


def bruteforce(name, K, A, B, n_cells, weight="uniform"):
    """Exhaustive minimiser of Eq. 3 over all boundary subsets of the grid."""
    idx = np.zeros(max(K - 1, 1), dtype=np.int32)
    obj = ctypes.c_double(0.0)
    rc = _load().fbo_bruteforce_w(_act_id(name), float(A), float(B), int(n_cells), int(K), WEIGHTS[weight],
                                  idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), ctypes.byref(obj))
    if rc != 0:
        raise ValueError(f"fbo_bruteforce failed with {rc}")
    return {"idx": idx[:K - 1].copy(), "objective": obj.value}


def loss_at(name, s, A=-8.0, B=8.0, weight="uniform"):
    """Eq. 3 at arbitrary boundaries ``s`` (levels by Eq. 4); returns
    (L, levels, gradient by Eq. 5)."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    K = s.size + 1
    lev = np.zeros(K, dtype=np.float64)
    grad = np.zeros(max(K - 1, 1), dtype=np.float64)
    c_dp = ctypes.POINTER(ctypes.c_double)
    val = _load().fbo_loss_at(_act_id(name), float(A), float(B), WEIGHTS[weight], K, s.ctypes.data_as(c_dp),
                              lev.ctypes.data_as(c_dp), grad.ctypes.data_as(c_dp))
    return val, lev, grad[:K - 1]


def finetune(name, s, A=-8.0, B=8.0, weight="uniform", max_iter=2000):
    """Gradient descent (Eq. 5) on the boundaries, started from ``s``."""
    s = np.array(s, dtype=np.float64)
    K = s.size + 1
    lev = np.zeros(K, dtype=np.float64)
    obj = ctypes.c_double(0.0)
    c_dp = ctypes.POINTER(ctypes.c_double)
    it = _load().fbo_finetune(_act_id(name), float(A), float(B), WEIGHTS[weight], K, s.ctypes.data_as(c_dp),
                              int(max_iter), lev.ctypes.data_as(c_dp), ctypes.byref(obj))
    if it < 0:
        raise ValueError("fbo_finetune failed")
    return {"s": s, "lev": lev, "objective": obj.value, "iterations": it}


# ----------------------------------------------------------------------------
# bit stream
# ----------------------------------------------------------------------------
def packed_words(n: int, bits: int) -> int:
    return (int(n) * int(bits) + 31) // 32


def pack(codes, bits: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.zeros(packed_words(codes.size, bits), dtype=np.uint32)
    _load().fbo_pack(int(bits), _ptr(codes), _ptr(out), codes.size)
    return out


def unpack(packed, bits: int, n: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    assert packed.size >= packed_words(n, bits)
    out = np.zeros(n, dtype=np.uint8)
    _load().fbo_unpack(int(bits), _ptr(packed), _ptr(out), n)
    return out


# ----------------------------------------------------------------------------
# hot path (Listing 1)
# ----------------------------------------------------------------------------
def _check_tables(bits, s=None, lev=None):
    K = 1 << int(bits)
    if s is not None:
        s = np.ascontiguousarray(s, dtype=np.float32)
        assert s.size == K - 1
    if lev is not None:
        lev = np.ascontiguousarray(lev, dtype=np.float32)
        assert lev.size == K
    return s, lev


def dp_solve_folded(name, bits, B=8.0, n_cells=2048):
    """Table for an even f' (caption of Fig. 3): 2^bits pieces on [0, B]; the
    error over [-B, B] is twice the half-axis optimum."""
    r = dp_solve(name, bits, 0.0, B, n_cells)
    r["objective"] = 2.0 * r["objective"]
    return r


def fwd(name, bits: int, s, x: np.ndarray, fold: bool = False):
    """Forward half: returns (y, packed).

    ``x`` is float32, float16, or uint16 holding bfloat16 bit patterns; ``y``
    has the same dtype.  ``s`` are the K-1 boundaries as binary32.  ``fold``:
    the code is the position of |x| (table on [0, B] for an even f')."""
    s, _ = _check_tables(bits, s=s)
    if s.size == 0:
        s = np.zeros(1, dtype=np.float32)
    x = np.ascontiguousarray(x)
    n = x.size
    packed = np.zeros(packed_words(n, bits), dtype=np.uint32)
    y = np.empty_like(x)
    lib = _load()
    if x.dtype == np.float32:
        lib.fbo_fwd_f32_fold(_act_id(name), int(bits), int(bool(fold)), _ptr(s), _ptr(x), _ptr(y), _ptr(packed), n)
    elif x.dtype == np.uint16:
        lib.fbo_fwd_bf16_fold(_act_id(name), int(bits), int(bool(fold)), _ptr(s), _ptr(x), _ptr(y), _ptr(packed), n)
    elif x.dtype == np.float16:
        lib.fbo_fwd_f16_fold(_act_id(name), int(bits), int(bool(fold)), _ptr(s), _ptr(x), _ptr(y), _ptr(packed), n)
    else:
        raise TypeError("x must be float32, float16 or uint16 (bfloat16 bits)")
    return y, packed


def bias_add(x: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """z[r, c] = x[r, c] + bias[c], the exact sum rounded once to the storage type (same dtype
    convention as ``fwd``: float32, float16, or uint16 holding bfloat16 bits).  ``x`` is
    (rows, cols) or flat with a length that is a multiple of ``bias.size``."""
    bias = np.ascontiguousarray(bias)
    x = np.ascontiguousarray(x)
    if x.dtype != bias.dtype:
        raise TypeError("x and bias must have the same dtype")
    cols = bias.size
    if cols == 0 or x.size % cols:
        raise ValueError("x.size must be a multiple of bias.size")
    z = np.empty_like(x)
    fn = {np.dtype(np.float32): "fbo_bias_add_f32", np.dtype(np.uint16): "fbo_bias_add_bf16",
          np.dtype(np.float16): "fbo_bias_add_f16"}.get(x.dtype)
    if fn is None:
        raise TypeError("x must be float32, float16 or uint16 (bfloat16 bits)")
    getattr(_load(), fn)(_ptr(x), _ptr(bias), x.size // cols, cols, _ptr(z))
    return z


def bwd(bits: int, lev, packed: np.ndarray, grad_out: np.ndarray, n: int | None = None):
    """Backward half: returns grad_in (same dtype convention as ``fwd``)."""
    _, lev = _check_tables(bits, lev=lev)
    grad_out = np.ascontiguousarray(grad_out)
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    if n is None:
        n = grad_out.size
    assert packed.size >= packed_words(n, bits)
    grad_in = np.empty_like(grad_out)
    lib = _load()
    if grad_out.dtype == np.float32:
        lib.fbo_bwd_f32(int(bits), _ptr(lev), _ptr(packed), _ptr(grad_out), _ptr(grad_in), n)
    elif grad_out.dtype == np.uint16:
        lib.fbo_bwd_bf16(int(bits), _ptr(lev), _ptr(packed), _ptr(grad_out), _ptr(grad_in), n)
    elif grad_out.dtype == np.float16:
        lib.fbo_bwd_f16(int(bits), _ptr(lev), _ptr(packed), _ptr(grad_out), _ptr(grad_in), n)
    else:
        raise TypeError("grad_out must be float32 or uint16 (bfloat16 bits)")
    return grad_in
