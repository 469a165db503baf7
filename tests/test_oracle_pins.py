"""Pins for the CPU oracle: every check compares it with something other than itself --
facts the paper states, closed forms, textbook bounds, library routines (numpy / scipy /
torch in fp64) in the special cases that reduce to them, and brute force on tiny inputs."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from oracle import Table
import nm_inputs

HERE = os.path.dirname(os.path.abspath(__file__))


def paper_facts():
    facts = {}
    with open(os.path.join(HERE, "golden", "paper_facts.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                facts[k.strip()] = float(v)
    return facts


def np_f(func):
    return {
        oracle.GELU: lambda x: 0.5 * x * (1 + scipy.special.erf(x / np.sqrt(2.0))),
        oracle.EXP: np.exp,
        oracle.RECIP: lambda x: 1.0 / x,
        oracle.RSQRT: lambda x: 1.0 / np.sqrt(x),
        oracle.RELU: lambda x: np.maximum(x, 0.0),
        oracle.SQRT: np.sqrt,
        oracle.IDENTITY: lambda x: x,
    }[func]


def np_f2max(func, lo, hi):
    """max |f''| on [lo, hi] from a dense numerical second difference (independent of the oracle)."""
    x = np.linspace(lo, hi, 200001)
    f = np_f(func)(x)
    h = x[1] - x[0]
    return np.max(np.abs(f[2:] - 2 * f[1:-1] + f[:-2])) / h ** 2


RANGES = {oracle.GELU: (-4.0, 4.0), oracle.EXP: (-8.0, 0.0), oracle.RECIP: (8.0, 128.0),
          oracle.RSQRT: (0.25, 4.0), oracle.SQRT: (0.25, 4.0)}


# ---------------------------------------------------------------- tables ---------

@pytest.mark.parametrize("func", list(RANGES))
@pytest.mark.parametrize("n", [7, 16, 64, 256])
def test_table_interpolates_and_is_continuous(func, n):
    """Section 3.2.1: the end of one segment is the start of the next, so at every breakpoint both
    neighbouring lines give f(x_i)."""
    lo, hi = RANGES[func]
    t = Table.secant(func, n, lo, hi)
    xs = lo + (hi - lo) * np.arange(n + 1) / n
    f = np_f(func)(xs)
    k = t.k.astype(np.float64)
    b = t.b.astype(np.float64)
    left = k * xs[:-1] + b       # segment i at its start
    right = k * xs[1:] + b       # segment i at its end
    scale = np.maximum(np.abs(f).max(), 1.0)
    # k, b are stored in fp32: interpolation holds to fp32 rounding of k*x and b
    tol = 4e-7 * (np.abs(k) * np.abs(xs[:-1]) + np.abs(b) + scale).max()
    assert np.abs(left - f[:-1]).max() <= tol
    assert np.abs(right - f[1:]).max() <= tol
    assert np.abs(right[:-1] - left[1:]).max() <= 2 * tol


@pytest.mark.parametrize("func", list(RANGES))
def test_table_error_bound_shrinks_16x(func):
    """Linear interpolation error is at most h^2/8 * max|f''|; four times the segments, a
    sixteenth of the error."""
    lo, hi = RANGES[func]
    f2 = np_f2max(func, lo, hi)
    x = np.linspace(lo, hi, 40001)
    errs = []
    for n in (16, 64, 256):
        t = Table.secant(func, n, lo, hi)
        y = t(x)
        err = np.abs(y - np_f(func)(x)).max()
        h = (hi - lo) / n
        assert err <= h * h / 8 * f2 * 1.02 + 1e-6
        errs.append(err)
    # the 16x law is asymptotic (h small against the curvature scale): strict at 64 -> 256
    assert 6 < errs[0] / errs[1] < 20
    assert 12 < errs[1] / errs[2] < 20


def test_relu_two_segments_exact():
    """Section 3: ReLU is already piecewise linear -- two segments reproduce it exactly, in and
    out of range."""
    t = Table.secant(oracle.RELU, 2, -6.0, 6.0)
    assert t.k.tolist() == [0.0, 1.0] and t.b.tolist() == [0.0, 0.0]
    x = np.concatenate([np.linspace(-100, 100, 4001), [0.0, -0.0, 6.0, -6.0, 1e30, -1e30]])
    assert np.array_equal(t(x), np.maximum(x, 0.0))


def test_identity_table_is_identity():
    t = Table.secant(oracle.IDENTITY, 64, -3.0, 5.0)
    assert np.all(t.k == 1.0) and np.all(np.abs(t.b) < 1e-6)


def test_gelu_tails_match_paper_statement():
    fx = paper_facts()
    lo, hi = fx["gelu_near_zero_at_or_below"], fx["gelu_near_identity_at_or_above"]
    x = np.linspace(-8, lo, 101)
    assert np.abs(oracle.exact(oracle.GELU, x)).max() < 5e-3
    x = np.linspace(hi, 8, 101)
    assert np.abs(oracle.exact(oracle.GELU, x) - x).max() < 5e-3
    # and the erf form itself, against scipy
    x = np.linspace(-6, 6, 1001)
    assert np.allclose(oracle.exact(oracle.GELU, x), np_f(oracle.GELU)(x), rtol=0, atol=1e-15)


def test_out_of_range_extends_end_lines():
    """Section 3.2.1: inputs outside the range share k, b with the first / last segment."""
    t = Table.secant(oracle.EXP, 8, -8.0, 0.0)
    x = np.array([-20.0, -8.5, 0.5, 3.0])
    y, idx = oracle.pwl_eval(t, x)
    assert idx.tolist() == [0, 0, 7, 7]
    exp = np.array([t.k[0] * x[0] + t.b[0], t.k[0] * x[1] + t.b[0], t.k[7] * x[2] + t.b[7],
                    t.k[7] * x[3] + t.b[7]], np.float64)
    assert np.allclose(y, exp, rtol=1e-15)
    # x exactly at x_max belongs to the last segment
    assert oracle.pwl_eval(t, np.array([0.0]))[1][0] == 7


def test_parameter_budget_order_of_magnitude():
    """Section 5.2: ~1.6 KB / 3.2 KB of extra parameters; 4 tables x 64 segments x (k,b) fp32 = 2 KB."""
    fx = paper_facts()
    ours = 4 * 64 * 2 * 4
    assert fx["extra_params_roberta_bytes"] / 2 <= ours <= fx["extra_params_resnet50_bytes"] * 2


# ---------------------------------------------------------------- index ----------

@pytest.mark.parametrize("func,n", [(oracle.GELU, 64), (oracle.EXP, 16), (oracle.RECIP, 256), (oracle.RSQRT, 37)])
def test_index_matches_linear_search_away_from_breakpoints(func, n):
    lo, hi = RANGES[func]
    t = Table.secant(func, n, lo, hi)
    bp = lo + (hi - lo) * np.arange(n + 1) / n
    rng = np.random.default_rng(3)
    x = rng.uniform(lo - 1, hi + 1, 20000).astype(np.float32)
    dist = np.abs(x[:, None].astype(np.float64) - bp[None, :]).min(axis=1)
    x = x[dist > 1e-4 * (hi - lo) / n * 64]
    _, idx = oracle.pwl_eval(t, x)
    brute = np.clip(np.searchsorted(bp, x.astype(np.float64), side="right") - 1, 0, n - 1)
    assert np.array_equal(idx, brute)


def test_index_is_one_correctly_rounded_fp32_fma():
    """The index is floor(fma(x, inv_h, off)) with a single fp32 rounding: checked against exact
    rational arithmetic."""
    t = Table.secant(oracle.GELU, 64, -4.0, 4.0)
    inv_h = np.float32(64 / 8.0)
    off = np.float32(4.0 * 64 / 8.0)
    t2 = Table.secant(oracle.RSQRT, 37, 0.25, 4.0)
    span = float(np.float32(4.0)) - float(np.float32(0.25))
    inv_h2 = np.float32(37 / span)
    off2 = np.float32(-0.25 * 37 / span)
    pts = nm_inputs.pwl_probe_points(-4.0, 4.0, 64, 500, 1)
    pts = pts[np.isfinite(pts)]
    for tab, ih, of, n in ((t, inv_h, off, 64), (t2, inv_h2, off2, 37)):
        for x in pts[:700]:
            exact_u = Fraction(float(x)) * Fraction(float(ih)) + Fraction(float(of))
            u = np.float32(exact_u)  # Fraction -> double -> float can double-round; guard below
            lo_ = np.nextafter(u, np.float32(-np.inf))
            hi_ = np.nextafter(u, np.float32(np.inf))
            cands = sorted({float(lo_), float(u), float(hi_)}, key=lambda c: abs(Fraction(c) - exact_u))
            u = cands[0]
            # skip exact ties between two floats (none expected for these constants)
            if len(cands) > 1 and abs(Fraction(cands[0]) - exact_u) == abs(Fraction(cands[1]) - exact_u):
                continue
            want = min(max(math.floor(u), 0), n - 1)
            assert int(tab.index(np.array([x]))[0]) == want


def test_index_nan_selects_segment_zero():
    t = Table.secant(oracle.GELU, 64, -4.0, 4.0)
    y, idx = oracle.pwl_eval(t, np.array([np.nan]))
    assert idx[0] == 0 and np.isnan(y[0])


def test_f32_eval_is_fma():
    t = Table.secant(oracle.EXP, 64, -8.0, 0.0)
    x = nm_inputs.pwl_probe_points(-8.0, 0.0, 64, 300, 5)
    x = x[np.isfinite(x)]
    y, idx = oracle.pwl_eval_f32(t, x)
    for xi, yi, s in zip(x[:400], y[:400], idx[:400]):
        ex = Fraction(float(t.k[s])) * Fraction(float(xi)) + Fraction(float(t.b[s]))
        # correctly rounded: no other float is closer
        for nb in (np.nextafter(yi, np.float32(np.inf)), np.nextafter(yi, np.float32(-np.inf))):
            assert abs(Fraction(float(yi)) - ex) <= abs(Fraction(float(nb)) - ex)


# ---------------------------------------------------------------- linear ---------

def test_linear_brute_force_tiny():
    rng = np.random.default_rng(0)
    A = rng.standard_normal((3, 5))
    W = rng.standard_normal((4, 5))
    bias = rng.standard_normal(4)
    res = rng.standard_normal((3, 4))
    out = oracle.linear(A, W, bias, res)
    for m in range(3):
        for j in range(4):
            s = sum(A[m, c] * W[j, c] for c in range(5)) + bias[j] + res[m, j]
            assert abs(out[m, j] - s) < 1e-13


def test_linear_matches_numpy_and_epilogue_order():
    """bias -> table -> residual: with the exact 2-segment ReLU table the result must be
    relu(A W^T + bias) + residual, computed by numpy."""
    rng = np.random.default_rng(1)
    A = rng.standard_normal((37, 53))
    W = rng.standard_normal((29, 53))
    bias = rng.standard_normal(29)
    res = rng.standard_normal((37, 29))
    relu = Table.secant(oracle.RELU, 2, -10.0, 10.0)
    out, idx = oracle.linear(A, W, bias, res, relu, want_idx=True)
    pre = A @ W.T + bias
    assert np.allclose(out, np.maximum(pre, 0) + res, rtol=1e-12, atol=1e-12)
    assert np.array_equal(idx, (pre.astype(np.float32) >= 0).astype(np.int32))
    ident = Table.secant(oracle.IDENTITY, 64, -3.0, 3.0)
    out2 = oracle.linear(A, W, bias, None, ident)
    assert np.allclose(out2, pre, rtol=1e-6, atol=1e-6)   # b of the identity table is O(1e-7)
    assert np.allclose(oracle.linear(A, W), A @ W.T, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- attention ------

def _torch_attention(qkv, B, L, h, d):
    H = h * d
    t = torch.from_numpy(qkv).reshape(B, L, 3, h, d)
    q, k, v = (t[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v)
    return o.permute(0, 2, 1, 3).reshape(B * L, H).numpy()


def test_attention_exact_mode_is_textbook_softmax_attention():
    B, L, h, d = 2, 24, 3, 8
    rng = np.random.default_rng(2)
    qkv = rng.standard_normal((B * L, 3 * h * d))
    out = oracle.attention(qkv, B, L, h, d, Table.exact(oracle.EXP), Table.exact(oracle.RECIP))
    assert np.allclose(out, _torch_attention(qkv, B, L, h, d), rtol=1e-10, atol=1e-12)


def test_attention_pwl_converges_to_exact_and_uses_final_max():
    B, L, h, d = 1, 32, 2, 16
    rng = np.random.default_rng(4)
    qkv = rng.standard_normal((B * L, 3 * h * d))
    ref = _torch_attention(qkv, B, L, h, d)
    errs = []
    for n in (16, 64, 256):
        te = Table.secant(oracle.EXP, n, -16.0, 0.0)
        tr = Table.secant(oracle.RECIP, n, 1.0, float(L))
        errs.append(np.abs(oracle.attention(qkv, B, L, h, d, te, tr) - ref).max())
    assert errs[0] > errs[1] > errs[2] and errs[2] < 2e-3
    # a row whose scores are all equal: e_j = PWLexp(0) for every j, sigma = L * PWLexp(0)
    q = np.zeros((L, 3 * h * d))
    q[:, 2 * h * d:] = rng.standard_normal((L, h * d))
    te = Table.secant(oracle.EXP, 64, -8.0, 0.0)
    tr = Table.secant(oracle.RECIP, 64, 2.0, 32.0)
    out = oracle.attention(q, 1, L, h, d, te, tr)
    e0 = te(np.array([0.0]))[0]
    r = tr(np.array([L * e0]))[0]
    want = (e0 * r) * q[:, 2 * h * d:].sum(axis=0, keepdims=True)
    assert np.allclose(out, np.repeat(want, L, axis=0), rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- layernorm ------

def test_layernorm_exact_mode_is_library_layer_norm():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((9, 48)) * 3 + 1
    g = rng.standard_normal(48)
    b = rng.standard_normal(48)
    y = oracle.layernorm(z, g, b, 1e-5, Table.exact(oracle.RSQRT))
    ref = torch.nn.functional.layer_norm(torch.from_numpy(z), (48,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    assert np.allclose(y, ref.numpy(), rtol=1e-11, atol=1e-12)


def test_layernorm_pwl_uses_table_on_variance_plus_eps():
    rng = np.random.default_rng(6)
    z = rng.standard_normal((5, 64))
    t = Table.secant(oracle.RSQRT, 64, 0.25, 4.0)
    y = oracle.layernorm(z, np.ones(64), np.zeros(64), 1e-5, t)
    assert np.abs(y.mean(axis=1)).max() < 1e-14
    v = z.var(axis=1)
    r = t(v + 1e-5)
    assert np.allclose(y.std(axis=1), np.sqrt(v) * r, rtol=1e-12)


def test_layernorm_sqrt_recip_exact_mode_is_library_layer_norm():
    """With both tables exact, 1/sqrt(v + eps) is recovered and the result is the textbook LayerNorm."""
    rng = np.random.default_rng(15)
    z = rng.standard_normal((7, 40)) * 2 - 0.5
    g = rng.standard_normal(40)
    b = rng.standard_normal(40)
    y = oracle.layernorm_sqrt_recip(z, g, b, 1e-5, Table.exact(oracle.SQRT), Table.exact(oracle.RECIP))
    ref = torch.nn.functional.layer_norm(torch.from_numpy(z), (40,), torch.from_numpy(g), torch.from_numpy(b), 1e-5)
    assert np.allclose(y, ref.numpy(), rtol=1e-11, atol=1e-12)


def test_layernorm_sqrt_recip_composes_the_two_tables_in_that_order():
    """r = recip_table(sqrt_table(v + eps)): checked through the row statistics of the output (gamma 1,
    beta 0: zero mean, standard deviation sqrt(v) * r), and against the swapped order, which differs."""
    rng = np.random.default_rng(16)
    z = rng.standard_normal((6, 64)) * np.array([[0.6], [0.9], [1.2], [1.5], [1.8], [2.1]])
    ts = Table.secant(oracle.SQRT, 16, 0.0625, 9.0)
    tr = Table.secant(oracle.RECIP, 16, 0.25, 3.0)
    y = oracle.layernorm_sqrt_recip(z, np.ones(64), np.zeros(64), 1e-5, ts, tr)
    assert np.abs(y.mean(axis=1)).max() < 1e-14
    v = z.var(axis=1)
    r = tr(ts(v + 1e-5))
    assert np.allclose(y.std(axis=1), np.sqrt(v) * r, rtol=1e-12)
    swapped = ts(tr(v + 1e-5))
    assert np.abs(swapped - r).max() > 1e-3


def test_layernorm_sqrt_recip_error_against_exact_is_within_the_secant_bounds():
    """|recip_t(sqrt_t(u)) - u^-1/2| <= e_r + e_s / s_min^2 with the secant-line bounds e = h^2/8 max|f''|
    (sqrt: |f''| = u^-3/2 / 4; 1/x: |f''| = 2 / x^3) and 1/x having slope at most 1/s_min^2."""
    a, b, n = 0.25, 9.0, 64
    sa, sb = 0.45, 3.05   # range of the sqrt table's values with margin for its error
    ts = Table.secant(oracle.SQRT, n, a, b)
    tr = Table.secant(oracle.RECIP, n, sa, sb)
    u = np.linspace(a, b, 20001)
    got = tr(ts(u))
    e_s = ((b - a) / n) ** 2 / 8 * (a ** -1.5 / 4)
    e_r = ((sb - sa) / n) ** 2 / 8 * (2 / sa ** 3)
    bound = e_r + e_s / sa ** 2
    err = np.abs(got - u ** -0.5)
    assert err.max() <= bound * (1 + 1e-6)
    assert err.max() > bound / 50   # the bound is not vacuous


# ---------------------------------------------------------------- encoder layer --

def _torch_encoder_layer(x, w, B, L, h):
    H = x.shape[1]
    F = w["W1"].shape[0]
    layer = torch.nn.TransformerEncoderLayer(H, h, F, dropout=0.0, activation="gelu", batch_first=True,
                                             norm_first=False, dtype=torch.float64)
    sd = {
        "self_attn.in_proj_weight": w["Wqkv"], "self_attn.in_proj_bias": w["bqkv"],
        "self_attn.out_proj.weight": w["Wo"], "self_attn.out_proj.bias": w["bo"],
        "linear1.weight": w["W1"], "linear1.bias": w["b1"], "linear2.weight": w["W2"], "linear2.bias": w["b2"],
        "norm1.weight": w["g1"], "norm1.bias": w["be1"], "norm2.weight": w["g2"], "norm2.bias": w["be2"],
    }
    layer.load_state_dict({k: torch.from_numpy(np.asarray(v, np.float64)) for k, v in sd.items()})
    layer.train(False)
    with torch.no_grad():
        torch.backends.mha.set_fastpath_enabled(False)
        y = layer(torch.from_numpy(np.asarray(x, np.float64)).reshape(B, L, H))
    return y.reshape(B * L, H).numpy()


def _exact_tables():
    return {"gelu": Table.exact(oracle.GELU), "exp": Table.exact(oracle.EXP),
            "recip": Table.exact(oracle.RECIP), "rsqrt": Table.exact(oracle.RSQRT)}


def _pwl_tables(cfg, n):
    r = cfg.ranges()
    return {"gelu": Table.secant(oracle.GELU, n, *r["gelu"]), "exp": Table.secant(oracle.EXP, n, *r["exp"]),
            "recip": Table.secant(oracle.RECIP, n, *r["recip"]), "rsqrt": Table.secant(oracle.RSQRT, n, *r["rsqrt"])}


def test_encoder_layer_exact_mode_is_library_post_ln_layer():
    cfg = nm_inputs.EncoderConfig("t", "f32", B=2, L=16, H=48, heads=4, F=96)
    x, layers = nm_inputs.encoder_inputs(cfg, seed=7, random_affine=True)
    w = {k: v * (5.0 if k.startswith("W") else 1.0) for k, v in layers[0].items()}
    y = oracle.encoder_layer(x, w, cfg.B, cfg.L, cfg.heads, _exact_tables(), eps=1e-5)
    ref = _torch_encoder_layer(x, w, cfg.B, cfg.L, cfg.heads)
    assert np.allclose(y, ref, rtol=1e-9, atol=1e-10)


def test_encoder_layer_pwl_approaches_exact_with_more_segments():
    cfg = nm_inputs.with_(nm_inputs.C1, B=1, L=32, H=64, heads=4, F=128)
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0)
    w = {k: v * (4.0 if k.startswith("W") else 1.0) for k, v in layers[0].items()}
    ref = oracle.encoder_layer(x, w, cfg.B, cfg.L, cfg.heads, _exact_tables())
    errs = [np.abs(oracle.encoder_layer(x, w, cfg.B, cfg.L, cfg.heads, _pwl_tables(cfg, n)) - ref).max()
            for n in (16, 64, 256)]
    assert errs[0] > errs[1] > errs[2]
    assert errs[2] < 1e-3


# ---------------------------------------------------------------- calibrated ranges (Section 3.2.1 step 1)

def test_calibrated_ranges_against_a_torch_run_of_the_exact_layer():
    """oracle.calibrate records the input range of each nonlinear function while running the exact model;
    here the same four ranges are taken from an independent fp64 torch run of a small two-layer encoder."""
    import oracle.calibrate as cal
    F = torch.nn.functional
    cfg = nm_inputs.EncoderConfig("t", "f32", B=2, L=16, H=48, heads=4, F=96, layers=2)
    x, layers = nm_inputs.encoder_inputs(cfg, seed=11, random_affine=True)
    layers = [{k: v * (5.0 if k.startswith("W") else 1.0) for k, v in w.items()} for w in layers]
    got = cal.encoder_input_ranges(x, layers, cfg.B, cfg.L, cfg.heads)
    lo = {k: np.inf for k in got}
    hi = {k: -np.inf for k in got}

    def see(k, t):
        lo[k] = min(lo[k], float(t.min()))
        hi[k] = max(hi[k], float(t.max()))

    y = torch.from_numpy(x.astype(np.float64)).reshape(cfg.B, cfg.L, cfg.H)
    d = cfg.H // cfg.heads
    for w in layers:
        t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in w.items()}
        qkv = y @ t["Wqkv"].T + t["bqkv"]
        q, k, v = (u.reshape(cfg.B, cfg.L, cfg.heads, d).transpose(1, 2) for u in qkv.split(cfg.H, dim=2))
        s = (q @ k.transpose(2, 3)) / np.sqrt(d)
        s = s - s.amax(dim=3, keepdim=True)
        see("exp", s)
        e = s.exp()
        see("recip", e.sum(dim=3))
        a = ((e / e.sum(dim=3, keepdim=True)) @ v).transpose(1, 2).reshape(cfg.B, cfg.L, cfg.H)
        z1 = y + a @ t["Wo"].T + t["bo"]
        see("rsqrt", z1.var(dim=2, unbiased=False) + 1e-5)
        x1 = F.layer_norm(z1, (cfg.H,), t["g1"], t["be1"], 1e-5)
        pre = x1 @ t["W1"].T + t["b1"]
        see("gelu", pre)
        z2 = x1 + F.gelu(pre) @ t["W2"].T + t["b2"]
        see("rsqrt", z2.var(dim=2, unbiased=False) + 1e-5)
        y = F.layer_norm(z2, (cfg.H,), t["g2"], t["be2"], 1e-5)
    for k in got:
        assert np.isclose(got[k][0], lo[k], rtol=1e-9, atol=1e-12), (k, got[k], lo[k])
        assert np.isclose(got[k][1], 0.0 if k == "exp" else hi[k], rtol=1e-9, atol=1e-12), (k, got[k], hi[k])
    assert got["exp"][1] == 0.0 and got["exp"][0] < 0 and 1.0 <= got["recip"][0] <= got["recip"][1] <= cfg.L


def test_stored_calibrated_ranges_reproduce_and_tighten_the_tables():
    """The stored file is what the committed script writes (checked for the small configuration), every table
    range contains its observed range, and with the calibrated ranges the 64-segment layer is closer to the
    exact layer than with the fixed ones (the purpose of step 1: segments are not spent outside the data)."""
    import json
    import oracle.calibrate as cal
    with open(cal.GOLDEN) as f:
        stored = json.load(f)
    again = cal.calibrate_config("c1")
    assert again == stored["c1"]
    for name in ("c1", "c2", "c3"):
        for k, (a, b) in stored[name]["table"].items():
            oa, ob = stored[name]["observed"][k]
            assert a <= oa and ob <= b, (name, k)
        assert nm_inputs.CONFIGS[name].ranges(calibrated=True) == {k: tuple(v) for k, v in stored[name]["table"].items()}
    cfg = nm_inputs.C1
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0)
    ref = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, _exact_tables())

    def err(r):
        tabs = {"gelu": Table.secant(oracle.GELU, 64, *r["gelu"]), "exp": Table.secant(oracle.EXP, 64, *r["exp"]),
                "recip": Table.secant(oracle.RECIP, 64, *r["recip"]), "rsqrt": Table.secant(oracle.RSQRT, 64, *r["rsqrt"])}
        return float(np.abs(oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, tabs) - ref).max())

    e_fixed, e_cal = err(cfg.ranges()), err(cfg.ranges(calibrated=True))
    print("C1 layer, 64 segments, max |PWL - exact|: fixed ranges %.3e, calibrated %.3e" % (e_fixed, e_cal))
    assert e_cal < 0.25 * e_fixed


# ---------------------------------------------------------------- int8 -----------

def test_int8_accumulators_and_epilogue():
    M, N, K = 19, 23, 96
    Aq = nm_inputs.int8_matrix((M, K), 1)
    Wq = nm_inputs.int8_matrix((N, K), 2)
    rng = np.random.default_rng(3)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    bias = (0.1 * rng.standard_normal(N)).astype(np.float32)
    a_scale = np.float32(0.031)
    t = Table.secant(oracle.GELU, 64, -4.0, 4.0)
    r = oracle.linear_i8(Aq, Wq, a_scale, ws, bias, None, t, out_scale=0.05)
    acc = Aq.astype(np.int64) @ Wq.astype(np.int64).T
    assert np.array_equal(r["acc"], acc.astype(np.int32))
    inv = np.float32(1.0) / np.float32(0.05)
    for m in range(0, M, 3):
        for j in range(0, N, 2):
            sc = np.float32(a_scale * ws[j])
            ex = Fraction(int(acc[m, j])) * Fraction(float(sc)) + Fraction(float(bias[j]))
            x = np.float32(float(ex))          # |ex| small, 53-bit double then float: check nearest below
            for nb in (np.nextafter(x, np.float32(np.inf)), np.nextafter(x, np.float32(-np.inf))):
                if abs(Fraction(float(nb)) - ex) < abs(Fraction(float(x)) - ex):
                    x = nb
            s = int(t.index(np.array([x]))[0])
            assert r["idx"][m, j] == s
            ey = Fraction(float(t.k[s])) * Fraction(float(x)) + Fraction(float(t.b[s]))
            y = r["y"][m, j]
            for nb in (np.nextafter(y, np.float32(np.inf)), np.nextafter(y, np.float32(-np.inf))):
                assert abs(Fraction(float(y)) - ey) <= abs(Fraction(float(nb)) - ey)
            q = float(np.clip(np.rint(np.float32(y * inv)), -127, 127))
            assert r["q"][m, j] == q


def test_quantize_round_half_even_and_clamp():
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 200.0, -200.0, 126.5, 127.4], np.float32)
    q = oracle.quantize_i8(x, 1.0)
    assert q.tolist() == [0, 2, 2, 0, -2, 127, -127, 126, 127]


# ---------------------------------------------------------------- CNN pieces -----

def test_conv_pool_match_torch():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((2, 9, 11, 5))
    W = rng.standard_normal((7, 3, 3, 5))
    bias = rng.standard_normal(7)
    for stride, pad in ((1, 1), (2, 1), (2, 0)):
        out = oracle.conv2d_nhwc(x, W, stride, pad, bias)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(W).permute(0, 3, 1, 2),
                                         torch.from_numpy(bias), stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
        assert np.allclose(out, ref, rtol=1e-11, atol=1e-11)
    relu = Table.secant(oracle.RELU, 2, -8.0, 8.0)
    res = rng.standard_normal((2, 9, 11, 7))
    out = oracle.conv2d_nhwc(x, W, 1, 1, bias, res, relu)
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).permute(0, 3, 1, 2), torch.from_numpy(W).permute(0, 3, 1, 2),
                                     torch.from_numpy(bias), padding=1).permute(0, 2, 3, 1).numpy()
    assert np.allclose(out, np.maximum(ref, 0) + res, rtol=1e-11, atol=1e-11)
    mp = oracle.maxpool_nhwc(x, 3, 2, 1)
    ref = torch.nn.functional.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(mp, ref)
    assert np.allclose(oracle.avgpool_nhwc(x), x.mean(axis=(1, 2)), rtol=1e-13)


# ---------------------------------------------------------------- Algorithms 2, 3 -

def test_alg2_worked_example_merges_minus2_to_minus1():
    """Section 3.2.2 / Fig. 3(a): with threshold 0.1 and primary length 0.5 the two primary
    segments on [-2,-1] of GELU merge into one."""
    fx = paper_facts()
    xs = oracle.hsize_startpoints(oracle.GELU, fx["alg2_example_dLx"], fx["alg2_example_dK_th"], -4.0, 4.0)
    a, b = fx["alg2_example_merged_from"], fx["alg2_example_merged_to"]
    assert a in xs and b in xs and (a + b) / 2 not in xs
    assert xs[0] == -4.0 and len(xs) < 16          # fewer than the 16 primary segments
    # a straight line never opens a new segment; a parabola opens one at every primary step
    assert len(oracle.hsize_startpoints(oracle.IDENTITY, 0.5, 0.1, -4.0, 4.0)) == 1


def test_alg3_bias_correction():
    """dE is the mean of f minus the mean of the secant; for a convex f it is negative; it removes
    ~5/6 of the squared error (closed form for small segments), the paper reporting 74-83 %."""
    fx = paper_facts()
    paper = {oracle.EXP: fx["alg3_mse_reduction_exp"], oracle.SQRT: fx["alg3_mse_reduction_sqrt"],
             oracle.RECIP: fx["alg3_mse_reduction_recip"], oracle.GELU: fx["alg3_mse_reduction_gelu"]}
    for func, (lo, hi) in ((oracle.EXP, (-8.0, 0.0)), (oracle.SQRT, (0.25, 4.0)), (oracle.RECIP, (1.0, 8.0)),
                           (oracle.GELU, (-4.0, 4.0))):
        n = 16
        xs = np.linspace(lo, hi, n + 1)
        k, b = oracle.secant_points(func, xs)
        b2, dE = oracle.bias_correct(func, xs, b)
        x = np.linspace(lo, hi, 160001)[:-1]
        seg = np.minimum(((x - lo) / (hi - lo) * n).astype(int), n - 1)
        f = np_f(func)(x)
        # dE against a numerical mean of (f - secant) per segment
        num = np.array([(f[seg == i] - (k[i] * x[seg == i] + b[i])).mean() for i in range(n)])
        assert np.allclose(dE, num, rtol=2e-3, atol=1e-7)
        if func in (oracle.EXP, oracle.RECIP):
            assert np.all(dE < 0)
        if func == oracle.SQRT:
            assert np.all(dE > 0)
        mse0 = ((k[seg] * x + b[seg] - f) ** 2).mean()
        mse1 = ((k[seg] * x + b2[seg] - f) ** 2).mean()
        red = 100 * (1 - mse1 / mse0)
        assert 70.0 < red < 84.0
        assert abs(red - paper[func]) < 12.0
    # Fig. 3(b): the GELU secant on [-1, 0] is biased (curve below the chord: convex there)
    k, b = oracle.secant_points(oracle.GELU, np.array([fx["alg3_biased_segment_from"], fx["alg3_biased_segment_to"]]))
    _, dE = oracle.bias_correct(oracle.GELU, np.array([-1.0, 0.0]), b)
    assert dE[0] < -0.02


def test_int8_storage_model_layer_against_library_routines():
    """The bf16-storage model of the int8 layer (not the definition: see the next test), rebuilt from
    library routines only (numpy rint/clip for the quantiser, numpy matmul, torch attention / layer_norm /
    gelu in fp64, torch bf16 casts) with exact nonlinearities: must agree with the oracle's composition
    in exact mode."""
    cfg = nm_inputs.with_(nm_inputs.C4, B=2, L=24, H=64, heads=4, F=128, layers=1)
    x, layers = nm_inputs.encoder_inputs(cfg, seed=5, random_affine=True)
    w = layers[0]
    q = nm_inputs.int8_encoder_inputs(cfg, layers)[0]
    got = oracle.encoder_layer_i8_storage(x, w, q, cfg.B, cfg.L, cfg.heads, _exact_tables())

    def bf(t):
        return torch.from_numpy(np.asarray(t, np.float32)).to(torch.bfloat16).to(torch.float64).numpy()

    def quant(t, s):
        s32 = np.float32(s)
        inv = np.float32(1.0) / s32
        return np.clip(np.rint(np.asarray(t, np.float32) * inv), -127, 127).astype(np.float64) * float(s32)

    def wdq(name):
        return q[name + "_q"].astype(np.float64) * q[name + "_s"].astype(np.float64)[:, None]

    H, h, d = cfg.H, cfg.heads, cfg.d
    qkv = bf(quant(x, q["a_x"]) @ wdq("Wqkv").T + w["bqkv"])
    a = bf(_torch_attention(qkv, cfg.B, cfg.L, h, d))
    z = bf(quant(a, q["a_attn"]) @ wdq("Wo").T + w["bo"] + x)
    ln = lambda t, g, b: torch.nn.functional.layer_norm(torch.from_numpy(t), (H,), torch.from_numpy(g.astype(np.float64)),
                                                        torch.from_numpy(b.astype(np.float64)), 1e-5).numpy()
    x1 = bf(ln(z, w["g1"], w["be1"]))
    g = torch.nn.functional.gelu(torch.from_numpy(quant(x1, q["a_x1"]) @ wdq("W1").T + w["b1"])).numpy()
    z2 = bf(quant(g, q["a_g"]) @ wdq("W2").T + w["b2"] + x1)
    ref = ln(z2, w["g2"], w["be2"])
    # a code on a rounding boundary may differ between two fp64 summation orders: allow a few elements
    err = np.abs(got - ref)
    assert (err > 1e-9).mean() < 0.02 and np.median(err) < 1e-12


# ---------------------------------------------------------------- int8, definition level ----------

def test_fake_quant_is_round_half_even_clamped_and_within_half_a_step():
    """code = clamp(rint(x / s), -127, 127) in fp64 against numpy, the tie and clamp cases written out,
    and the defining property |fq(x) - x| <= s / 2 inside the representable range."""
    s = 0.25
    x = np.array([0.125, 0.375, 0.625, -0.125, -0.375, 100.0, -100.0, 31.70, 31.80, 0.0])
    y, codes = oracle.fake_quant(x, s, want_codes=True)
    assert codes.tolist() == [0, 2, 2, 0, -2, 127, -127, 127, 127, 0]
    assert np.array_equal(y, codes.astype(np.float64) * s)
    rng = np.random.default_rng(31)
    t = rng.standard_normal(5000) * 2.0
    s = 5.5 / 127.0
    y, codes = oracle.fake_quant(t, s, want_codes=True)
    assert np.array_equal(codes, np.clip(np.rint(t / s), -127, 127).astype(np.int8))
    inside = np.abs(t) <= 127 * s
    assert np.abs(y - t)[inside].max() <= s / 2 * (1 + 1e-12)
    assert np.abs(y - t)[inside].max() > s / 2 * 0.98          # the bound is reached: rint, not floor or trunc
    assert np.all(np.abs(y[~inside]) == 127 * s)


def _int8_case(seed=5):
    cfg = nm_inputs.with_(nm_inputs.C4, B=2, L=24, H=64, heads=4, F=128, layers=1)
    x, layers = nm_inputs.encoder_inputs(cfg, seed=seed, random_affine=True)
    q = nm_inputs.int8_encoder_inputs(cfg, layers)[0]
    return cfg, x.astype(np.float64), layers[0], q


def test_int8_layer_definition_against_library_routines():
    """The definition-level int8 layer (fake-quantise the operand of each of the four GEMMs, round nothing
    else) rebuilt from library routines only: numpy rint/clip, numpy matmul, torch attention, layer_norm
    and gelu in fp64, exact nonlinearities.  No bf16 cast anywhere."""
    cfg, x, w, q = _int8_case()
    got, st = oracle.encoder_layer_i8(x, w, q, cfg.B, cfg.L, cfg.heads, _exact_tables(), want_stages=True)

    def fq(t, s):
        return np.clip(np.rint(t / float(s)), -127, 127) * float(s)

    def wdq(name):
        return q[name + "_q"].astype(np.float64) * q[name + "_s"].astype(np.float64)[:, None]

    H, h, d = cfg.H, cfg.heads, cfg.d
    ln = lambda t, g, b: torch.nn.functional.layer_norm(torch.from_numpy(t), (H,), torch.from_numpy(g.astype(np.float64)),
                                                        torch.from_numpy(b.astype(np.float64)), 1e-5).numpy()
    qkv = fq(x, q["a_x"]) @ wdq("Wqkv").T + w["bqkv"]
    a = _torch_attention(qkv, cfg.B, cfg.L, h, d)
    z = fq(a, q["a_attn"]) @ wdq("Wo").T + w["bo"] + x
    x1 = ln(z, w["g1"], w["be1"])
    g = torch.nn.functional.gelu(torch.from_numpy(fq(x1, q["a_x1"]) @ wdq("W1").T + w["b1"])).numpy()
    z2 = fq(g, q["a_g"]) @ wdq("W2").T + w["b2"] + x1
    ref = ln(z2, w["g2"], w["be2"])
    assert np.allclose(st["qkv"], qkv, rtol=1e-11, atol=1e-12)
    # a code that sits on a rounding boundary may fall either way between two fp64 summation orders
    for name, r in (("a", a), ("z", z), ("x1", x1), ("g", g), ("z2", z2)):
        e = np.abs(st[name] - r)
        assert (e > 1e-9).mean() < 0.01 and np.median(e) < 1e-12, name
    err = np.abs(got - ref)
    assert (err > 1e-9).mean() < 0.02 and np.median(err) < 1e-12


def test_int8_layer_definition_stays_within_the_quantisation_step_of_the_unquantised_layer():
    """Replacing an operand t by fq(t) moves every entry by at most s/2 (no clamping on these inputs), so a
    GEMM output moves by at most s/2 * sum_k |W[j,k]|: checked for the first GEMM against the plain fp64
    linear operator on the same dequantised weights; and the whole layer stays close to the unquantised
    layer on those weights (int8 with per-tensor scales of ~5 sigma / 127 is a ~1 % perturbation)."""
    cfg, x, w, q = _int8_case(seed=9)
    tabs = _exact_tables()
    y, st = oracle.encoder_layer_i8(x, w, q, cfg.B, cfg.L, cfg.heads, tabs, want_stages=True)
    wd = {n: q[n + "_q"].astype(np.float64) * q[n + "_s"].astype(np.float64)[:, None] for n in ("Wqkv", "Wo", "W1", "W2")}
    assert np.abs(x).max() <= 127 * q["a_x"]
    plain = oracle.linear(x, wd["Wqkv"], w["bqkv"])
    bound = q["a_x"] / 2 * np.abs(wd["Wqkv"]).sum(axis=1)
    assert np.all(np.abs(st["qkv"] - plain) <= bound[None, :] * (1 + 1e-9))
    assert np.abs(st["qkv"] - plain).max() > bound.max() / 50          # and the operand really was quantised
    w_plain = dict(w)
    w_plain.update(wd)
    ref = oracle.encoder_layer(x, w_plain, cfg.B, cfg.L, cfg.heads, tabs)
    rel = np.sqrt(((y - ref) ** 2).mean()) / np.sqrt((ref ** 2).mean())
    assert 1e-4 < rel < 3e-2


def test_int8_storage_model_differs_from_the_definition_only_by_storage_rounding():
    """The storage model re-rounds six tensors to bf16 (relative 2^-9 each): its distance from the
    definition is of that order, not zero and not large."""
    cfg, x, w, q = _int8_case(seed=11)
    tabs = _pwl_tables(cfg, 64)
    xb = nm_inputs.round_to(x.astype(np.float32), "bf16").astype(np.float64)
    a = oracle.encoder_layer_i8(xb, w, q, cfg.B, cfg.L, cfg.heads, tabs)
    b = oracle.encoder_layer_i8_storage(xb, w, q, cfg.B, cfg.L, cfg.heads, tabs)
    rel = np.sqrt(((a - b) ** 2).mean()) / np.sqrt((a ** 2).mean())
    assert 1e-4 < rel < 2e-2


def test_int8_linear_residual_branch_is_one_fp32_add():
    """y = fl32(fl32(fma(acc, sc, bias)) + residual): the residual branch of the strict fp32 epilogue,
    against exact rational arithmetic; the integer outputs are untouched by it."""
    M, N, K = 11, 13, 64
    Aq = nm_inputs.int8_matrix((M, K), 21)
    Wq = nm_inputs.int8_matrix((N, K), 22)
    rng = np.random.default_rng(23)
    ws = rng.uniform(1e-4, 3e-4, N).astype(np.float32)
    bias = (0.1 * rng.standard_normal(N)).astype(np.float32)
    res = rng.standard_normal((M, N)).astype(np.float32)
    a_scale = np.float32(0.027)
    t = Table.secant(oracle.GELU, 64, -4.0, 4.0)
    base = oracle.linear_i8(Aq, Wq, a_scale, ws, bias, None, t)
    r = oracle.linear_i8(Aq, Wq, a_scale, ws, bias, res, t, out_scale=0.05)
    assert np.array_equal(r["acc"], base["acc"]) and np.array_equal(r["idx"], base["idx"])
    inv = np.float32(1.0) / np.float32(0.05)
    for m in range(M):
        for j in range(N):
            ex = Fraction(float(base["y"][m, j])) + Fraction(float(res[m, j]))
            y = r["y"][m, j]
            for nb in (np.nextafter(y, np.float32(np.inf)), np.nextafter(y, np.float32(-np.inf))):
                assert abs(Fraction(float(y)) - ex) <= abs(Fraction(float(nb)) - ex)
            assert r["q"][m, j] == float(np.clip(np.rint(np.float32(y * inv)), -127, 127))
    assert np.abs(r["y"] - base["y"]).max() > 0.5           # the residual really was added


# ---------------------------------------------------------------- Algorithm 3's integrals ----------

@pytest.mark.parametrize("func,lo,hi", [(oracle.GELU, -4.0, 4.0), (oracle.EXP, -8.0, 0.0), (oracle.RECIP, 0.5, 8.0),
                                        (oracle.RSQRT, 0.25, 4.0), (oracle.RELU, -1.3, 2.1), (oracle.SQRT, 0.25, 4.0),
                                        (oracle.IDENTITY, -1.5, 2.5)])
def test_alg3_antiderivative_against_numerical_quadrature(func, lo, hi):
    """Every closed-form integral the segment mean of Algorithm 3 is taken from, against adaptive
    quadrature of the function itself (scipy), on sub-intervals of the range."""
    import scipy.integrate
    f = np_f(func)
    xs = np.linspace(lo, hi, 9)
    F = oracle.antiderivative(func, xs)
    for i in range(8):
        pts = [0.0] if xs[i] < 0.0 < xs[i + 1] else None
        want, _ = scipy.integrate.quad(lambda v: float(f(np.float64(v))), xs[i], xs[i + 1], points=pts, epsabs=1e-13,
                                       epsrel=1e-13)
        assert abs((F[i + 1] - F[i]) - want) <= 1e-11 * max(1.0, abs(want)), (func, i)


@pytest.mark.parametrize("func,xs", [(oracle.RSQRT, np.linspace(0.25, 4.0, 9)), (oracle.RELU, np.linspace(-1.2, 1.8, 7)),
                                     (oracle.IDENTITY, np.linspace(-2.0, 3.0, 6))])
def test_alg3_bias_correction_rsqrt_relu_identity(func, xs):
    """dE = mean of f over the segment minus the mean of its secant, against a numerical mean, for the
    three functions the four-function check above does not cover.  A straight line needs no correction;
    ReLU only on the segment that straddles 0; a convex function is corrected downwards."""
    k, b = oracle.secant_points(func, xs)
    b2, dE = oracle.bias_correct(func, xs, b)
    n = xs.size - 1
    f = np_f(func)
    for i in range(n):
        x = xs[i] + (xs[i + 1] - xs[i]) * (np.arange(200000) + 0.5) / 200000      # midpoint rule
        num = (f(x) - (k[i] * x + b[i])).mean()
        assert abs(dE[i] - num) <= 1e-8 + 1e-6 * abs(num), (func, i)
    assert np.allclose(b2 - b, dE, rtol=0, atol=1e-15)
    if func == oracle.IDENTITY:
        assert np.abs(dE).max() < 1e-15
    if func == oracle.RELU:
        straddle = (xs[:-1] < 0) & (xs[1:] > 0)
        assert straddle.sum() == 1 and dE[straddle][0] < -0.01 and np.abs(dE[~straddle]).max() < 1e-15
    if func == oracle.RSQRT:
        assert np.all(dE < 0)


def test_maxpool_relu_form_is_the_library_max_pool():
    """max(a, b) = b + ReLU(a - b): with the 2-segment ReLU table (exact everywhere) and fp16-representable
    inputs every difference and sum is exact in fp64, so the fold reproduces torch's max pooling exactly,
    padding and stride included."""
    rng = np.random.default_rng(21)
    x = nm_inputs.round_to(rng.standard_normal((2, 9, 11, 5)).astype(np.float32) * 3, "f16").astype(np.float64)
    relu = Table.secant(oracle.RELU, 2, -8.0, 8.0)
    for ks, st, pad in ((3, 2, 1), (2, 2, 0), (3, 1, 1)):
        got = oracle.maxpool_nhwc_relu(x, ks, st, pad, relu)
        ref = torch.nn.functional.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), ks, st, pad).permute(0, 2, 3, 1)
        assert np.array_equal(got, ref.numpy())
        assert np.array_equal(got, oracle.maxpool_nhwc(x, ks, st, pad))


def test_maxpool_relu_form_uses_the_table():
    """With a table that is not ReLU the fold is no longer a maximum: b + t(a - b) on a 1 x 2 window."""
    half = Table(2, -8.0, 8.0, np.array([0.0, 0.5], np.float32), np.array([0.0, 0.0], np.float32))   # 0.5 * ReLU
    y = oracle.maxpool_nhwc_relu(np.array([[[[1.0], [3.0]], [[0.0], [0.0]]]]), 2, 1, 0, half)
    # fold order: (0,0)=1 -> (0,1)=3: 1 + 0.5*2 = 2 -> (1,0)=0: 2 + 0 -> (1,1)=0: 2
    assert y.shape == (1, 1, 1, 1) and y[0, 0, 0, 0] == 2.0


def test_resnet50_composition_against_torch():
    """The oracle's ResNet-50-shaped network (a composition of its own conv / pool / linear routines)
    against torch.nn.functional in fp64 on a reduced image: pins the block wiring (projection shortcut
    only in a stage's first block, stride in the 3x3, ReLU after the add) and the folded-BatchNorm inputs."""
    import nm_inputs_cnn
    import oracle.cnn
    F = torch.nn.functional
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(1, seed=3, random_bn=True, image=64, num_classes=16)
    relu = Table.secant(oracle.RELU, 2, -8.0, 8.0)
    got = oracle.cnn.resnet50(x, convs, fc_w, fc_b, relu)

    def conv(inp, c):
        _, _, _, s, p = c["spec"]
        return F.conv2d(inp, torch.from_numpy(c["w"].astype(np.float64)).permute(0, 3, 1, 2),
                        torch.from_numpy(c["b"].astype(np.float64)), stride=s, padding=p)

    it = iter(convs)
    y = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    y = F.max_pool2d(F.relu(conv(y, next(it))), 3, 2, 1)
    for nb in (3, 4, 6, 3):
        for b in range(nb):
            ca, cb, cc = next(it), next(it), next(it)
            t = F.relu(conv(F.relu(conv(y, ca)), cb))
            sc = conv(y, next(it)) if b == 0 else y
            y = F.relu(conv(t, cc) + sc)
    ref = (y.mean(dim=(2, 3)) @ torch.from_numpy(fc_w.astype(np.float64)).T + torch.from_numpy(fc_b.astype(np.float64))).numpy()
    assert np.allclose(got, ref, rtol=1e-10, atol=1e-9)
    assert len(convs) == 53 and sum(c["w"].size for c in convs) + fc_w.size > 23e6   # ResNet-50's ~23.5 M conv weights


@pytest.mark.parametrize("blocks,base", [((1, 2, 1, 1), 32), ((2, 1, 1, 2), 16)])
def test_resnet_variant_composition_against_torch(blocks, base):
    """The depth / width variants (Section 5 compares ResNet-50 "and its variant models"): the same
    composition with other block counts per stage and another first-stage width, against
    torch.nn.functional in fp64; the convolution count and channel widths follow the generator's rule."""
    import nm_inputs_cnn
    import oracle.cnn
    F = torch.nn.functional
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(1, seed=5, random_bn=True, image=64, num_classes=8,
                                                         blocks=blocks, base_width=base)
    assert len(convs) == 1 + sum(3 * b + 1 for b in blocks)
    assert convs[0]["w"].shape == (base, 7, 7, 3) and fc_w.shape == (8, 32 * base)
    assert convs[-1]["w"].shape[0] == 32 * base                      # last block's conv_c: 4 * (base << 3)
    relu = Table.secant(oracle.RELU, 2, -8.0, 8.0)
    got = oracle.cnn.resnet50(x, convs, fc_w, fc_b, relu, blocks=blocks)

    def conv(inp, c):
        _, _, _, s, p = c["spec"]
        return F.conv2d(inp, torch.from_numpy(c["w"].astype(np.float64)).permute(0, 3, 1, 2),
                        torch.from_numpy(c["b"].astype(np.float64)), stride=s, padding=p)

    it = iter(convs)
    y = torch.from_numpy(x.astype(np.float64)).permute(0, 3, 1, 2)
    y = F.max_pool2d(F.relu(conv(y, next(it))), 3, 2, 1)
    for nb in blocks:
        for b in range(nb):
            ca, cb, cc = next(it), next(it), next(it)
            t = F.relu(conv(F.relu(conv(y, ca)), cb))
            sc = conv(y, next(it)) if b == 0 else y
            y = F.relu(conv(t, cc) + sc)
    ref = (y.mean(dim=(2, 3)) @ torch.from_numpy(fc_w.astype(np.float64)).T + torch.from_numpy(fc_b.astype(np.float64))).numpy()
    assert np.allclose(got, ref, rtol=1e-10, atol=1e-9)
    with pytest.raises((AssertionError, StopIteration)):   # block counts that do not match the convolutions
        oracle.cnn.resnet50(x, convs, fc_w, fc_b, relu, blocks=(1, 1, 1, 1))


# ---------------------------------------------------------------- int8 attention ----------

def _i8_attn_case(B=2, L=24, h=2, d=16, seed=41):
    rng = np.random.default_rng(seed)
    qkv = rng.standard_normal((B * L, 3 * h * d)).astype(np.float32)
    s = np.float32(4.0 / 127.0)
    codes = np.clip(np.rint(qkv / s), -127, 127).astype(np.int8)
    return codes, s


def test_int8_attention_integer_parts_are_exact_and_fp32_steps_are_single_roundings():
    """Scores and P.V against int64 matmuls; every fp32 step against exact rational arithmetic; the codes
    against numpy rint/clip; the row sum is the integer sum of the codes."""
    B, L, h, d = 2, 24, 2, 16
    codes, s = _i8_attn_case(B, L, h, d)
    H = h * d
    te = Table.secant(oracle.EXP, 64, -8.0, 0.0)
    tr = Table.secant(oracle.RECIP, 64, 1.0, float(L))
    r = oracle.attention_i8(codes, B, L, h, d, s, s, s, te, tr, want_dumps=True)
    scale = np.float32(1.0 / np.sqrt(d))
    sc = np.float32(np.float32(s * s) * scale)
    inv127 = np.float32(1.0) / np.float32(127.0)
    c1 = np.float32(s * inv127)
    def near(y, ex):       # y is the float nearest to the exact rational ex
        for nb in (np.nextafter(y, np.float32(np.inf)), np.nextafter(y, np.float32(-np.inf))):
            assert abs(Fraction(float(y)) - ex) <= abs(Fraction(float(nb)) - ex)
    for b in range(B):
        for g in range(h):
            q = codes[b * L:(b + 1) * L, g * d:(g + 1) * d].astype(np.int64)
            k = codes[b * L:(b + 1) * L, H + g * d:H + (g + 1) * d].astype(np.int64)
            v = codes[b * L:(b + 1) * L, 2 * H + g * d:2 * H + (g + 1) * d].astype(np.int64)
            acc = q @ k.T
            assert np.array_equal(r["acc"][b, g], acc.astype(np.int32))
            p = r["p"][b, g].astype(np.int64)
            assert np.array_equal(r["oacc"][b * L:(b + 1) * L, g * d:(g + 1) * d], (p @ v).astype(np.int32))
            for i in range(0, L, 5):
                m = int(acc[i].max())
                neg = np.float32(-(np.float32(m) * sc))
                near(neg, -(Fraction(m) * Fraction(float(sc))))
                for j in range(0, L, 3):
                    x = np.float32(float(Fraction(int(acc[i, j])) * Fraction(float(sc)) + Fraction(float(neg))))
                    ex = Fraction(int(acc[i, j])) * Fraction(float(sc)) + Fraction(float(neg))
                    for nb in (np.nextafter(x, np.float32(np.inf)), np.nextafter(x, np.float32(-np.inf))):
                        if abs(Fraction(float(nb)) - ex) < abs(Fraction(float(x)) - ex):
                            x = nb
                    e, _ = oracle.pwl_eval_f32(te, np.array([x], np.float32))
                    assert p[i, j] == int(np.clip(np.rint(np.float32(e[0] * np.float32(127.0))), -127, 127))
                sigma = np.float32(np.float32(int(p[i].sum())) * inv127)
                rr, _ = oracle.pwl_eval_f32(tr, np.array([sigma], np.float32))
                for c in range(0, d, 4):
                    oa = int((p[i] * v[:, c]).sum())
                    want = np.float32(np.float32(np.float32(oa) * c1) * rr[0])
                    assert r["out"][b * L + i, g * d + c] == want


def test_int8_attention_approaches_float_attention():
    """With fine tables (256 segments: table error ~1e-3), int8 attention equals textbook attention on the
    dequantised operands up to the quantisation of the probabilities (step 1/127, at most 1/254 off per key):
    the output moves by at most sum_j |v_j| / 254 per row before normalisation; and the rows of codes are
    normalised by their own sum, so a row of identical scores returns the mean of V as float attention does."""
    B, L, h, d = 1, 32, 2, 16
    codes, s = _i8_attn_case(B, L, h, d, seed=43)
    te, tr = Table.secant(oracle.EXP, 256, -16.0, 0.0), Table.secant(oracle.RECIP, 256, 0.5, 33.0)
    out = oracle.attention_i8(codes, B, L, h, d, s, s, s, te, tr).astype(np.float64)
    deq = codes.astype(np.float64) * float(s)
    ref = _torch_attention(deq, B, L, h, d)
    H = h * d
    vabs = np.abs(deq[:, 2 * H:]).reshape(L, h, d).sum(axis=0)          # sum_j |v_j| per (head, channel)
    # normalised by sigma >= 1 (the maximum element has code 127); a loose but rigorous envelope
    bound = (vabs / 254.0 + np.abs(ref).reshape(L, h, d).max(axis=0) * L / 254.0).reshape(1, H)
    assert np.all(np.abs(out - ref) <= bound + 5e-3 * np.abs(ref).max())
    assert np.abs(out - ref).max() < 0.05 and np.abs(out - ref).max() > 1e-5      # close, and really quantised
    z = codes.copy()
    z[:, :2 * H] = 0                                                            # all scores equal
    out = oracle.attention_i8(z, B, L, h, d, s, s, s, te, tr).astype(np.float64)
    want = (z[:, 2 * H:].astype(np.float64) * float(s)).mean(axis=0, keepdims=True)
    assert np.allclose(out, np.repeat(want, L, axis=0), rtol=2e-3, atol=1e-4)     # the 1/x table's own error
