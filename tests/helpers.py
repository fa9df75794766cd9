"""Shared helpers for the test-suite (no arithmetic of the method)."""
from __future__ import annotations

import numpy as np


def ordered_int(bits: np.ndarray, width: int) -> np.ndarray:
    """Maps sign-magnitude float bit patterns to integers that are monotone in
    the float value (+0 and -0 coincide), so that |a - b| counts ulps."""
    b = bits.astype(np.int64)
    sign = 1 << (width - 1)
    return np.where(b & sign, -(b & (sign - 1)), b)


def ulp_distance(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    """Elementwise ulp distance between two float32 arrays or two uint16
    (bfloat16 bit pattern) arrays."""
    if a.dtype == np.float32:
        return np.abs(ordered_int(a.view(np.uint32), 32) - ordered_int(b.view(np.uint32), 32))
    if a.dtype == np.float16:
        return np.abs(ordered_int(a.view(np.uint16), 16) - ordered_int(b.view(np.uint16), 16))
    assert a.dtype == np.uint16
    return np.abs(ordered_int(a, 16) - ordered_int(b, 16))


def bf16_bits_to_f32(h) -> np.ndarray:
    return (np.asarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def finite_mask(x: np.ndarray) -> np.ndarray:
    if x.dtype == np.uint16:
        return np.isfinite(bf16_bits_to_f32(x))
    return np.isfinite(x)
