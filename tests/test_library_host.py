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
