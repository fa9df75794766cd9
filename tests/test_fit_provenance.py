"""The polynomial constants hard-coded in csrc/fewbit_math.cuh are the ones
csrc/fit_coefficients.py produces.

The script is run as it stands and every coefficient it prints is looked up
among the floating-point literals of the header (signs may differ: the kernel
evaluates some polynomials in the negated variable).  The comparison allows
5e-6 relative: the fits are iteratively reweighted least squares, and the last
digits of the smallest coefficients move with the iteration count by far less
than the approximation error the fit reports.
"""
import os
import re
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2202_00441_b200", "csrc")

_NUM = r"[-+]?(?:\d+\.\d*|\.\d+|\d+)(?:[eE][-+]?\d+)?"


def _header_literals():
    text = open(os.path.join(CSRC, "fewbit_math.cuh")).read()
    text = re.sub(r"//.*", "", text)
    vals = [abs(float(m)) for m in re.findall(r"(?<![\w.])(" + _NUM + r")f?\b", text)]
    return np.array(sorted(set(v for v in vals if v != 0.0)))


def _printed_coefficients():
    out = subprocess.run([sys.executable, os.path.join(CSRC, "fit_coefficients.py")], capture_output=True, text=True,
                         timeout=600, check=True).stdout
    coefs = {}
    for line in out.splitlines():
        name, _, rest = line.partition(":")
        rest = re.split(r"max (?:relative )?error", rest)[0]            # drop the reported fit error
        rest = re.sub(r"\([^)]*\)", "", rest)                             # "(s^0..s^8)" and the like
        rest = re.sub(r"float32\([^)]*\)", "", rest)
        nums = [float(m) for m in re.findall(r"(?<![\w^.])(" + _NUM + r")(?![\w^])", rest)]
        coefs[name.strip()] = [v for v in nums if v != 0.0]
    return coefs


def test_every_fitted_constant_is_in_the_header():
    lits = _header_literals()
    coefs = _printed_coefficients()
    assert {"GELU bf16", "GELU f16", "GELU f32", "exp f32", "ln 2 split", "softplus 16-bit"} <= set(coefs)
    assert len(coefs["GELU bf16"]) == 8 and len(coefs["GELU f16"]) == 7 and len(coefs["exp f32"]) == 5
    assert len(coefs["softplus 16-bit"]) == 6 and len(coefs["GELU f32"]) >= 11
    missing = []
    for name, vals in coefs.items():
        for v in vals:
            if name == "GELU f32" and abs(v) in (0.5, 2.0, 1.0):          # "u = w - 1/2" in the label
                continue
            rel = np.abs(lits - abs(v)) / abs(v)
            if rel.min() > 5e-6:
                missing.append((name, v, float(lits[rel.argmin()])))
    assert not missing, missing
