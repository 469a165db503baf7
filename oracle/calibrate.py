"""Calibrated table ranges (TEST INFRASTRUCTURE, part of the oracle): Section 3.2.1, step 1 -- the input range
of every nonlinear function is obtained by running the model.  The model run here is the oracle's encoder with
the EXACT nonlinearities (Table.exact), stage by stage with the oracle's own operators, on sampled sequences;
what is recorded is the smallest and largest input each of the four functions sees:

    gelu   input: x1 W1^T + b1
    exp    input: score minus the row maximum (at most 0)
    recip  input: the row sum of the exponentials
    rsqrt  input: variance + eps of both LayerNorms

Run as a script it writes tests/golden/calibrated_ranges.json for the named configurations:

    python -m oracle.calibrate

Only the oracle and the seeded input generators are used."""
from __future__ import annotations

import json
import os

import numpy as np

from . import EXP, GELU, RECIP, RSQRT, Table, attention, exact, layernorm, linear

GOLDEN = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "tests", "golden",
                      "calibrated_ranges.json")


def encoder_input_ranges(x, layers, B, L, h, eps=1e-5):
    """Runs the exact-nonlinearity encoder over x [B*L, H] and returns {'gelu': (lo, hi), 'exp': (lo, 0.0),
    'recip': (lo, hi), 'rsqrt': (lo, hi)}: the observed input range of each function."""
    ex = {"gelu": Table.exact(GELU), "exp": Table.exact(EXP), "recip": Table.exact(RECIP), "rsqrt": Table.exact(RSQRT)}
    lo = {k: np.inf for k in ex}
    hi = {k: -np.inf for k in ex}

    def see(name, a):
        lo[name] = min(lo[name], float(np.min(a)))
        hi[name] = max(hi[name], float(np.max(a)))

    y = np.asarray(x, dtype=np.float64)
    H = y.shape[1]
    d = H // h
    scale = 1.0 / np.sqrt(d)
    for w in layers:
        qkv = linear(y, w["Wqkv"], w["bqkv"])
        for b in range(B):
            blk = qkv[b * L:(b + 1) * L]
            for g in range(h):
                q = blk[:, g * d:(g + 1) * d]
                k = blk[:, H + g * d:H + (g + 1) * d]
                s = scale * (q @ k.T)
                s = s - s.max(axis=1, keepdims=True)
                see("exp", s)
                see("recip", np.exp(s).sum(axis=1))
        a = attention(qkv, B, L, h, d, ex["exp"], ex["recip"])
        z1 = linear(a, w["Wo"], w["bo"], residual=y)
        see("rsqrt", z1.var(axis=1) + eps)
        x1 = layernorm(z1, w["g1"], w["be1"], eps, ex["rsqrt"])
        pre = linear(x1, w["W1"], w["b1"])
        see("gelu", pre)
        z2 = linear(exact(GELU, pre), w["W2"], w["b2"], residual=x1)
        see("rsqrt", z2.var(axis=1) + eps)
        y = layernorm(z2, w["g2"], w["be2"], eps, ex["rsqrt"])
    out = {k: (lo[k], hi[k]) for k in ex}
    out["exp"] = (lo["exp"], 0.0)
    return out


def widen(ranges, margin=0.05):
    """The table ranges taken from observed ones: each end moved outward by `margin` of the width (the sample is
    not the whole workload), the exp range kept ending at 0, positive-input functions kept positive."""
    out = {}
    for k, (a, b) in ranges.items():
        w = (b - a) * margin
        a2, b2 = a - w, b + w
        if k == "exp":
            b2 = 0.0
        if k in ("recip", "rsqrt"):
            a2 = max(a2, a * 0.5)
        out[k] = (float(np.float32(a2)), float(np.float32(b2)))
    return out


def calibrate_config(name, n_seq=2, seed=0):
    import nm_inputs
    cfg = nm_inputs.CONFIGS[name]
    x, layers = nm_inputs.encoder_inputs(cfg, seed=seed)
    n_seq = min(n_seq, cfg.B)
    obs = encoder_input_ranges(x[: n_seq * cfg.L], layers, n_seq, cfg.L, cfg.heads)
    return {"observed": {k: list(v) for k, v in obs.items()}, "table": {k: list(v) for k, v in widen(obs).items()},
            "sample": "%d of %d sequences, all %d layers, seed %d, exact nonlinearities" % (n_seq, cfg.B, len(layers), seed)}


def main():
    out = {}
    for name in ("c1", "c2", "c3"):
        out[name] = calibrate_config(name)
        print(name, out[name]["table"])
    os.makedirs(os.path.dirname(GOLDEN), exist_ok=True)
    with open(GOLDEN, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    print("wrote", GOLDEN)


if __name__ == "__main__":
    main()
