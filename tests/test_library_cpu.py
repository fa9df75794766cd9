"""CPU-only checks of the library: it loads, exports what include/fewbit.h
declares, its host solver agrees with the oracle, and its argument checks
answer before anything touches a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2202_00441_b200 as fb
from paper_2202_00441_b200 import build as fb_build
from paper_2202_00441_b200.workloads import ACTIVATIONS, EXTRA_ACTIVATIONS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fb_build.build_library()
    return fb.load_library()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "fewbit.h")).read()
    names = re.findall(r"FEWBIT_API[^;]*?\b(fewbit_\w+)\s*\(", header)
    assert len(names) >= 14
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for code in range(6):
        assert lib.fewbit_status_string(code)
    assert lib.fewbit_status_string(99) == b"unknown status"


def test_packed_bytes(lib):
    for bits in (1, 2, 3, 4):
        for n in (0, 1, 31, 32, 33, 1000, 2 ** 24 + 7, 2 ** 28):
            assert fb.fewbit_packed_bytes(n, bits) == 4 * ((n * bits + 31) // 32)
    assert fb.fewbit_packed_bytes(100, 0) == 0 and fb.fewbit_packed_bytes(100, 5) == 0
    # the binding sizes its buffers without the foreign call: same numbers
    for n in (0, 1, 31, 32, 33, 1023, 1025, 2 ** 24 + 7, 2 ** 33 + 5):
        for bits in (1, 2, 3, 4):
            assert fb.binding._packed_bytes(n, bits) == fb.fewbit_packed_bytes(n, bits)


@pytest.mark.parametrize("act", ACTIVATIONS + EXTRA_ACTIVATIONS)
def test_solver_matches_oracle(lib, act):
    """The library's DP (Eq. 7-9) and the oracle's are separate programmes;
    they must reach the same optimum.  Smooth f': same boundaries, levels equal
    after rounding to binary32 (up to 1 ulp).  LeakyReLU
    (piecewise-constant f'): every zero-error table is optimal, so only the
    objective and the induced function q are compared."""
    for bits in (1, 2, 3, 4):
        t = fb.fewbit_table_create(act, bits)
        s, lev = t.arrays()
        r = oracle.dp_solve(act, bits, -8.0, 8.0, 4096)
        assert t.objective == pytest.approx(r["objective"], abs=1e-12)
        if act in ("leaky_relu", "relu"):
            probe = np.linspace(-7.99, 7.99, 4001)
            q_lib = lev[np.searchsorted(s, probe.astype(np.float32), side="left")]
            q_ref = r["lev"].astype(np.float32)[np.searchsorted(r["s"].astype(np.float32), probe.astype(np.float32), side="left")]
            np.testing.assert_allclose(q_lib, q_ref, atol=1e-7)
        else:
            rs, rlev = r["s"].astype(np.float32), r["lev"].astype(np.float32)
            if act in ("sigmoid", "tanh") and not np.array_equal(s, rs):
                # even f': a table and its mirror image have the same error,
                # rounding noise picks one; both are the optimum
                rs, rlev = -rs[::-1], rlev[::-1]
            np.testing.assert_array_equal(s, rs)
            np.testing.assert_allclose(lev, rlev, rtol=2e-7, atol=1e-9)


def test_solver_other_range_matches_oracle(lib):
    t = fb.fewbit_table_create_ex("silu", 3, -10.0, 10.0, 1000)
    r = oracle.dp_solve("silu", 3, -10.0, 10.0, 1000)
    assert t.objective == pytest.approx(r["objective"], abs=1e-12)
    np.testing.assert_allclose(t.arrays()[0], r["s"].astype(np.float32), rtol=1e-6)


def test_table_from_arrays_round_trip_and_validation(lib):
    s = np.array([-1.0, 0.5, 2.0], dtype=np.float32)
    lev = np.array([0.0, 0.25, 0.75, 1.0], dtype=np.float32)
    t = fb.fewbit_table_from_arrays("tanh", 2, s, lev)
    s2, lev2 = t.arrays()
    np.testing.assert_array_equal(s, s2)
    np.testing.assert_array_equal(lev, lev2)
    assert np.isnan(t.objective)
    with pytest.raises(fb.FewbitError):
        fb.fewbit_table_from_arrays("tanh", 2, s[::-1].copy(), lev)
    with pytest.raises(fb.FewbitError):
        fb.fewbit_table_from_arrays("tanh", 2, np.array([0, np.nan, 1], np.float32), lev)
    # equal boundaries (a degenerate table) are allowed
    fb.fewbit_table_from_arrays("tanh", 2, np.array([0, 0, 1], np.float32), lev)


def test_invalid_table_requests(lib):
    assert not lib.fewbit_table_create(0, 0)
    assert not lib.fewbit_table_create(0, 5)
    assert not lib.fewbit_table_create(9, 2)
    assert not lib.fewbit_table_create(-1, 2)
    out = ctypes.c_void_p()
    assert lib.fewbit_table_create_ex(0, 2, 1.0, 1.0, 100, ctypes.byref(out)) == 1
    assert lib.fewbit_table_create_ex(0, 2, -1.0, 1.0, 3, ctypes.byref(out)) == 1
    assert lib.fewbit_table_create_ex(0, 2, -1.0, 1.0, 100, None) == 1
    lib.fewbit_table_destroy(None)


def test_hot_path_argument_checks_need_no_gpu(lib):
    """NULL / misaligned / empty requests are answered on the host."""
    t = fb.fewbit_table_create("gelu", 3)
    h = t.handle
    A = 1 << 20                      # a fake, well aligned "device address"; never dereferenced
    assert lib.fewbit_fwd(None, A, A, A, 10, 0, None) == 1
    assert lib.fewbit_fwd(h, A, A, A, 10, 7, None) == 1
    assert lib.fewbit_fwd(h, None, A, A, 10, 0, None) == 1
    assert lib.fewbit_fwd(h, A, None, A, 10, 0, None) == 1
    assert lib.fewbit_fwd(h, A, A, None, 10, 0, None) == 1
    # the rule: element buffers 16-byte aligned, packed words 4-byte aligned (any dtype)
    assert lib.fewbit_fwd(h, A + 8, A, A, 10, 0, None) == 3
    assert lib.fewbit_fwd(h, A, A + 8, A, 10, 1, None) == 3
    assert lib.fewbit_fwd(h, A, A, A + 2, 10, 1, None) == 3
    assert lib.fewbit_fwd(h, A, A + 4, A, 10, 2, None) == 3
    assert lib.fewbit_fwd(h, None, None, None, 0, 0, None) == 0
    assert lib.fewbit_bwd(None, A, A, A, 10, 0, None) == 1
    assert lib.fewbit_bwd(h, None, A, A, 10, 0, None) == 1
    assert lib.fewbit_bwd(h, A, A + 2, A, 10, 1, None) == 3
    assert lib.fewbit_bwd(h, A, A, A + 8, 10, 0, None) == 3
    assert lib.fewbit_bwd(h, A + 1, A, A, 10, 0, None) == 3
    assert lib.fewbit_bwd(h, A, A, A, 0, 1, None) == 0
    assert lib.fewbit_fwd_host(h, A, A, A, 10, 0, None, 0) == 1
    assert lib.fewbit_fwd_host(h, A, A, A, 10, 0, A, 16) == 5
    assert lib.fewbit_bwd_host(h, A, A, A, 10, 0, A + 8, 1 << 20) == 3
    assert lib.fewbit_fwd_host(h, A, A, A, 0, 0, None, 0) == 0
    # f(x + bias): x, bias, y, packed, rows, cols
    assert lib.fewbit_fwd_bias(None, A, A, A, A, 4, 1024, 1, None) == 1
    assert lib.fewbit_fwd_bias(h, A, None, A, A, 4, 1024, 1, None) == 1
    assert lib.fewbit_fwd_bias(h, A, A, A, A, 4, 1020, 1, None) == 2         # a row is not a whole number of 8-element chunks
    assert lib.fewbit_fwd_bias(h, A, A, A, A, 4, 1 << 32, 1, None) == 2       # row length beyond 32 bits
    assert lib.fewbit_fwd_bias(h, A, A + 8, A, A, 4, 1024, 1, None) == 3
    assert lib.fewbit_fwd_bias(h, A, A, A, A + 2, 4, 1024, 1, None) == 3
    assert lib.fewbit_fwd_bias(h, A, A, A, A, 1 << 40, 1 << 30, 1, None) == 1  # rows * cols overflows
    assert lib.fewbit_fwd_bias(h, None, None, None, None, 0, 1024, 1, None) == 0
    tf = fb.fewbit_table_create_folded("tanh", 2)
    assert lib.fewbit_fwd_bias(tf.handle, A, A, A, A, 4, 1024, 1, None) == 2  # no folded tables with a bias
    # options: unknown option / value out of range are refused, valid ones read back
    assert lib.fewbit_set_option(99, 0) == 1 and lib.fewbit_get_option(99) == -1
    assert lib.fewbit_set_option(0, 3) == 1 and lib.fewbit_set_option(2, -1) == 1 and lib.fewbit_set_option(2, 65) == 1
    assert lib.fewbit_set_option(3, 17) == 1 and lib.fewbit_set_option(4, 2) == 1
    for opt, default, other in ((0, 0, 2), (1, 0, 1), (2, 0, 7), (3, 0, 4), (4, 1, 0), (5, 0, 1), (6, 0, 2)):
        assert lib.fewbit_get_option(opt) == default
        assert lib.fewbit_set_option(opt, other) == 0 and lib.fewbit_get_option(opt) == other
        assert lib.fewbit_set_option(opt, default) == 0
    assert lib.fewbit_tail_warp_count(None, 0) == 1
    # the accuracy scan: act, first pattern, count, result
    assert lib.fewbit_f32_activation_scan(99, 0, 16, A, None) == 1
    assert lib.fewbit_f32_activation_scan(0, 0, 16, None, None) == 1
    assert lib.fewbit_f32_activation_scan(0, 1 << 32, 1, A, None) == 1
    assert lib.fewbit_f32_activation_scan(0, 0, 16, A + 4, None) == 3


def test_host_workspace_bytes(lib):
    assert fb.fewbit_host_workspace_bytes(1, fb.binding.torch.float32, 3) == 3 * (2 * 4096 + 512)
    assert fb.fewbit_host_workspace_bytes(1 << 20, fb.binding.torch.bfloat16, 4) == 3 * (2 * (2 << 20) + (1 << 19))
    assert load_zero(lib) == 0


def load_zero(lib):
    return lib.fewbit_host_workspace_bytes(100, 0, 9)


def test_memory_ratio_reproduces_the_papers_accounting():
    """Appendix memory table: RoBERTa-base keeps 36.0 MB of pointwise-
    nonlinearity inputs out of 219.6 MB of activations; at b bits those shrink
    to b/32 of fp32, which gives the printed 16 / 15 / 15 / 14 % savings."""
    nonlin, total = 36.0, 219.6
    printed = {1: 16, 2: 15, 3: 15, 4: 14}
    for bits, pct in printed.items():
        saved = nonlin * (1 - fb.fewbit_packed_bytes(32, bits) / (32 * 4)) / total
        assert round(100 * saved) == pct


@pytest.mark.parametrize("act", ["sigmoid", "tanh"])
def test_folded_solver_matches_oracle(lib, act):
    """Even-derivative fold (caption of Fig. 3): the library's half-axis solve equals the oracle's."""
    for bits in (1, 2, 3, 4):
        t = fb.fewbit_table_create_folded(act, bits)
        assert t.folded
        s, lev = t.arrays()
        r = oracle.dp_solve_folded(act, bits, 8.0, 2048)
        assert t.objective == pytest.approx(r["objective"], abs=1e-12)
        np.testing.assert_array_equal(s, r["s"].astype(np.float32))
        np.testing.assert_allclose(lev, r["lev"].astype(np.float32), rtol=2e-7, atol=1e-9)
        assert (s > 0).all()
    assert not fb.fewbit_table_create(act, 2).folded


def test_folded_tables_need_an_even_derivative(lib):
    for act in ("gelu", "silu", "elu", "softplus", "leaky_relu"):
        with pytest.raises(fb.FewbitError) as e:
            fb.fewbit_table_create_folded(act, 2)
        assert e.value.status == 2
    with pytest.raises(fb.FewbitError):
        fb.fewbit_table_from_arrays("gelu", 1, [0.5], [0.1, 0.9], folded=True)
    assert fb.fewbit_table_from_arrays("tanh", 1, [0.5], [0.9, 0.1], folded=True).folded
    assert lib.fewbit_table_is_folded(None) == 0


@pytest.mark.parametrize("act", ["gelu", "silu", "tanh", "softplus"])
@pytest.mark.parametrize("weight", ["uniform", "normal"])
def test_weight_and_finetune_options_match_oracle(lib, act, weight):
    """Normal weight (named under Eq. 3) and Eq. 5 fine-tuning: the library's solver and the oracle's
    reach the same grid optimum and the same stationary point."""
    for bits in (2, 3):
        t = fb.fewbit_table_create_opt(act, bits, weight=weight)
        r = oracle.dp_solve(act, bits, weight=weight)
        assert t.objective == pytest.approx(r["objective"], abs=1e-12)
        start = r["s"]
        if act == "tanh" and not np.array_equal(t.arrays()[0], start.astype(np.float32)):
            start = -start[::-1]              # even f': the mirror image is the same optimum
        np.testing.assert_array_equal(t.arrays()[0], start.astype(np.float32))
        tf = fb.fewbit_table_create_opt(act, bits, weight=weight, finetune_iters=2000)
        f = oracle.finetune(act, start, weight=weight)
        assert tf.objective == pytest.approx(f["objective"], abs=1e-10)
        assert tf.objective <= t.objective + 1e-15
        np.testing.assert_allclose(tf.arrays()[0], f["s"], atol=1e-5)
        np.testing.assert_allclose(tf.arrays()[1], f["lev"], atol=1e-5)
        s64 = tf.arrays()[0].astype(np.float64)
        lev = tf.arrays()[1].astype(np.float64)
        resid = np.abs(2 * oracle.act_deriv(act, s64) - lev[1:] - lev[:-1])
        assert resid.max() < 1e-5


def test_solver_option_validation(lib):
    with pytest.raises(fb.FewbitError) as e:
        fb.fewbit_table_create_opt("gelu", 2, folded=True, A=0.0)
    assert e.value.status == 2
    with pytest.raises(fb.FewbitError):
        fb.fewbit_table_create_opt("tanh", 2, folded=True, A=-8.0)
    with pytest.raises(fb.FewbitError):
        fb.fewbit_table_create_opt("tanh", 2, finetune_iters=-1)
    t = fb.fewbit_table_create_opt("tanh", 2, A=0.0, n_cells=2048, folded=True, weight="normal", finetune_iters=200)
    assert t.folded and (t.arrays()[0] > 0).all()
    assert lib.fewbit_table_create_opt(0, 2, None, None) == 1
