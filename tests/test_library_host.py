"""CPU-only checks of the CUDA library: it loads, exports every symbol the header declares,
its host-side table builder agrees with the oracle's, and argument validation that needs no
device rejects bad calls."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
import paper_2305_14405_b200 as nm


@pytest.fixture(scope="module")
def lib():
    from paper_2305_14405_b200 import build
    build.build()
    return nm.load()


def test_every_declared_symbol_is_exported(lib):
    text = open(nm.HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(nm_[a-z0-9_]+)\s*\(", text))
    assert declared, "no declarations found in the header"
    assert declared == set(nm.EXPORTS), declared ^ set(nm.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert nm.status_string(0) == "NM_OK"
    assert nm.status_string(7) == "NM_ERR_TIMEOUT"
    assert nm.status_string(99) == "NM_ERR_UNKNOWN"


@pytest.mark.parametrize("func,lo,hi", [(nm.FUNC_GELU, -4.0, 4.0), (nm.FUNC_EXP, -8.0, 0.0), (nm.FUNC_RECIP, 8.0, 128.0),
                                        (nm.FUNC_RECIP, 32.0, 512.0), (nm.FUNC_RSQRT, 0.25, 4.0), (nm.FUNC_RELU, -5.0, 5.0),
                                        (nm.FUNC_SQRT, 0.5, 9.0), (nm.FUNC_IDENTITY, -1.0, 2.0)])
@pytest.mark.parametrize("n", [1, 2, 16, 64, 256])
def test_table_builder_matches_oracle_bitwise(lib, func, lo, hi, n):
    k, b = nm.pwl_table_build(func, n, lo, hi)
    t = oracle.Table.secant(func, n, lo, hi)
    assert np.array_equal(np.asarray(k, np.float32), t.k)
    assert np.array_equal(np.asarray(b, np.float32), t.b)


def test_table_builder_rejects_bad_requests(lib):
    k = (C.c_float * 4)()
    assert lib.nm_pwl_table_build(0, 0, -1.0, 1.0, k, k) == 2          # n < 1
    assert lib.nm_pwl_table_build(0, 257, -1.0, 1.0, k, k) == 2        # n too large
    assert lib.nm_pwl_table_build(0, 4, 1.0, 1.0, k, k) == 2           # empty range
    assert lib.nm_pwl_table_build(42, 4, -1.0, 1.0, k, k) == 1         # unknown function
    assert lib.nm_pwl_table_build(0, 4, -1.0, 1.0, None, k) == 1       # null output


def test_calls_reject_null_context(lib):
    assert lib.nm_pwl_table_load(None, 0, 4, -1.0, 1.0, (C.c_float * 4)(), (C.c_float * 4)()) == 1
    assert lib.nm_linear_pwl(None, None, None) == 1
    assert lib.nm_attention_pwl(None, None, None) == 1
    assert lib.nm_layernorm_pwl(None, None, None, None, None, 0, 0, 0.0, 0, 0, None) == 1
    assert lib.nm_layernorm_pwl_sqrt_recip(None, None, None, None, None, 0, 0, 0.0, 0, 0, 0, None) == 1
    assert lib.nm_maxpool2d_pwl(None, None, None, 0, 0, 0, 0, 0, 0, 0, 0, 0, None) == 1
    assert lib.nm_ctx_destroy(None) == 1
    cfg = nm.Context.encoder_cfg(2, 16, 64, 4, 128, nm.BF16)
    assert lib.nm_encoder_workspace_bytes(C.byref(cfg)) > 0
    bad = nm.Context.encoder_cfg(2, 16, 65, 4, 128, nm.BF16)      # hidden not divisible by heads
    assert lib.nm_encoder_workspace_bytes(C.byref(bad)) == 0


def test_product_does_not_import_the_oracle():
    root = os.path.dirname(nm.__file__)
    for dirpath, _, files in os.walk(root):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "nm_oracle" not in src, f


@pytest.mark.parametrize("func,lo,hi,dLx,dK", [(nm.FUNC_GELU, -4.0, 4.0, 0.5, 0.1), (nm.FUNC_GELU, -4.0, 4.0, 0.125, 0.02),
                                               (nm.FUNC_EXP, -8.0, 0.0, 0.125, 0.01), (nm.FUNC_RECIP, 1.0, 33.0, 0.25, 0.002),
                                               (nm.FUNC_SQRT, 0.25, 8.25, 0.0625, 0.01), (nm.FUNC_RSQRT, 0.25, 4.25, 0.03125, 0.02)])
@pytest.mark.parametrize("bias", [False, True])
def test_elastic_table_builder_matches_oracle_bitwise(lib, func, lo, hi, dLx, dK, bias):
    """Algorithms 2 and 3 in the library's host code against the oracle's (pinned) routines."""
    from util import oracle_elastic_table
    n, k, b, nseg = nm.pwl_table_build_elastic(func, lo, hi, dLx, dK, bias_correct=bias)
    t, nseg_ref = oracle_elastic_table(func, lo, hi, dLx, dK, bias_correct=bias)
    assert n == t.n and nseg == nseg_ref and nseg < n          # segments were merged
    assert np.array_equal(np.asarray(k, np.float32), t.k)
    assert np.array_equal(np.asarray(b, np.float32), t.b)


def test_elastic_table_builder_rejects_bad_requests(lib):
    k = (C.c_float * 256)()
    n, s = C.c_int(0), C.c_int(0)
    f = lib.nm_pwl_table_build_elastic
    assert f(0, -4.0, 4.0, 0.01, 0.1, 1, 0.0, C.byref(n), C.byref(s), k, k) == 2     # 800 primary cells > 256
    assert f(0, -4.0, 4.0, 0.3, 0.1, 1, 0.0, C.byref(n), C.byref(s), k, k) == 2      # range not a whole number of cells
    assert f(0, 4.0, -4.0, 0.5, 0.1, 1, 0.0, C.byref(n), C.byref(s), k, k) == 2
    assert f(9, -4.0, 4.0, 0.5, 0.1, 1, 0.0, C.byref(n), C.byref(s), k, k) == 1


def _np_func(func):
    import scipy.special
    return {nm.FUNC_GELU: lambda x: 0.5 * x * (1 + scipy.special.erf(x / np.sqrt(2.0))), nm.FUNC_EXP: np.exp,
            nm.FUNC_RECIP: lambda x: 1.0 / x, nm.FUNC_RSQRT: lambda x: 1.0 / np.sqrt(x), nm.FUNC_SQRT: np.sqrt,
            nm.FUNC_RELU: lambda x: np.maximum(x, 0.0), nm.FUNC_IDENTITY: lambda x: x}[func]


def _segments_of(k, b):
    """(first cell, one-past-last cell) of every run of equal (k, b) on the primary grid."""
    runs, s = [], 0
    for c in range(1, len(k) + 1):
        if c == len(k) or k[c] != k[s] or b[c] != b[s]:
            runs.append((s, c))
            s = c
    return runs


def test_elastic_builder_reproduces_the_papers_worked_example(lib):
    """Section 3.2.2, Fig. 3(a): GELU with primary length 0.5 and slope threshold 0.1 keeps one segment
    over [-2, -1].  Checked on the library's own output, no oracle involved."""
    n, k, b, nseg = nm.pwl_table_build_elastic(nm.FUNC_GELU, -4.0, 4.0, 0.5, 0.1, bias_correct=False)
    assert n == 16 and nseg < 16
    cells = [(-4.0 + 0.5 * s, -4.0 + 0.5 * e) for s, e in _segments_of(k, b)]
    assert (-2.0, -1.0) in cells and len(cells) == nseg
    # a straight line is one segment whatever the threshold
    n, k, b, nseg = nm.pwl_table_build_elastic(nm.FUNC_IDENTITY, -4.0, 4.0, 0.5, 0.1, bias_correct=True)
    assert nseg == 1 and np.all(np.asarray(k) == 1.0) and np.abs(np.asarray(b)).max() < 1e-7


@pytest.mark.parametrize("func,lo,hi,dLx", [(nm.FUNC_GELU, -4.0, 4.0, 0.5), (nm.FUNC_EXP, -8.0, 0.0, 0.5),
                                            (nm.FUNC_RECIP, 1.0, 8.0, 0.4375), (nm.FUNC_SQRT, 0.25, 4.0, 0.234375),
                                            (nm.FUNC_RSQRT, 0.25, 4.0, 0.234375)])
def test_elastic_builder_against_numerical_means(lib, func, lo, hi, dLx):
    """Algorithm 3 in the library's host code against facts that involve no other implementation: every
    kept segment's line is the secant through its end points shifted by dE, dE being the mean of f minus
    the mean of the secant over the segment (midpoint rule on numpy's own functions); with the threshold
    at zero nothing merges, and the shift removes ~5/6 of the squared error of the secant (Section 3.2.3
    reports 74-83 %)."""
    f = _np_func(func)
    n0, k0, b0, nseg0 = nm.pwl_table_build_elastic(func, lo, hi, dLx, 0.0, bias_correct=False)
    n, k, b, nseg = nm.pwl_table_build_elastic(func, lo, hi, dLx, 0.0, bias_correct=True)
    assert n == n0 == nseg0 == nseg                   # threshold 0: one segment per primary cell
    k0, b0, k, b = (np.asarray(v, np.float64) for v in (k0, b0, k, b))
    assert np.array_equal(k, k0)
    mse0 = mse1 = 0.0
    for c in range(n):
        xa, xb = lo + c * dLx, lo + (c + 1) * dLx
        ks = (f(xb) - f(xa)) / (xb - xa)
        bs = f(xa) - ks * xa
        tol = 4e-7 * (abs(ks) * max(abs(xa), abs(xb)) + abs(bs) + 1.0)     # k, b are stored in fp32
        assert abs(k0[c] - ks) <= tol and abs(b0[c] - bs) <= tol
        x = xa + (xb - xa) * (np.arange(100000) + 0.5) / 100000
        dE = (f(x) - (ks * x + bs)).mean()
        assert abs((b[c] - b0[c]) - dE) <= 2 * tol + 1e-6 * abs(dE), (func, c)
        mse0 += ((k0[c] * x + b0[c] - f(x)) ** 2).mean()
        mse1 += ((k[c] * x + b[c] - f(x)) ** 2).mean()
    red = 100 * (1 - mse1 / mse0)
    assert 70.0 < red < 84.0, red
    # with a large e_th no intercept moves
    _, _, b_off, _ = nm.pwl_table_build_elastic(func, lo, hi, dLx, 0.0, bias_correct=True, e_th=10.0)
    assert np.array_equal(np.asarray(b_off, np.float64), b0)
