"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds NO arithmetic of the method: it only draws random tensors of
the shapes the workloads name, rounds them to the storage dtype, and records
the table ranges each workload uses.  Both the CPU oracle and the CUDA library
are fed from here so that they see identical numbers.

Workloads are synthetic stand-ins for the GLUE / ImageNet-class inputs the
paper evaluates on (those datasets are not available and are not reproduced);
only the BERT-base / BERT-large / ResNet-50 *shapes* are used.

Draw order for an encoder workload (numpy ``default_rng(seed)``, fp32 values):
x, then for each layer Wqkv, Wo, W1, W2, then (only when ``random_affine``)
bqkv, bo, b1, b2, g1, be1, g2, be2.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch


@dataclass(frozen=True)
class EncoderConfig:
    name: str
    dtype: str          # "f32" | "bf16" | "i8" (int8 GEMMs, bf16 activations)
    B: int
    L: int
    H: int
    heads: int
    F: int
    layers: int = 1
    segments: int = 64
    eps: float = 1e-5

    @property
    def T(self):
        return self.B * self.L

    @property
    def d(self):
        return self.H // self.heads

    def ranges(self, calibrated=False):
        """[x_min, x_max] of each PWL table: GELU input, exp input (score minus row max),
        reciprocal input (row sum, at most L), rsqrt input (variance + eps).  The default is fixed per
        workload; calibrated=True returns the ranges observed by running the exact model on sampled
        sequences (Section 3.2.1, step 1), as stored by `python -m oracle.calibrate` in
        tests/golden/calibrated_ranges.json (this module only reads the file)."""
        if calibrated:
            import json
            import os
            path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "tests", "golden", "calibrated_ranges.json")
            with open(path) as f:
                stored = json.load(f)
            key = self.name.split("_")[0]
            if key not in stored:
                raise KeyError("no calibrated ranges stored for %s" % self.name)
            return {k: tuple(v) for k, v in stored[key]["table"].items()}
        return {"gelu": (-4.0, 4.0), "exp": (-8.0, 0.0), "recip": (self.L / 16.0, float(self.L)),
                "rsqrt": (0.25, 4.0)}

    def flops_per_layer(self):
        T, H, F, L = self.T, self.H, self.F, self.L
        gemm = 2 * T * H * (3 * H) + 2 * T * H * H + 2 * 2 * T * H * F
        attn = 4 * T * L * H
        return gemm + attn


C1 = EncoderConfig("c1_tiny_f32", "f32", B=1, L=128, H=256, heads=4, F=1024)
C2 = EncoderConfig("c2_bert_base_layer_bf16", "bf16", B=8, L=128, H=768, heads=12, F=3072)
C3 = EncoderConfig("c3_bert_base_12l_bf16", "bf16", B=32, L=512, H=768, heads=12, F=3072, layers=12)
C4 = EncoderConfig("c4_bert_large_24l_i8", "i8", B=16, L=512, H=1024, heads=16, F=4096, layers=24)
CONFIGS = {"c1": C1, "c2": C2, "c3": C3, "c4": C4}


def with_(cfg: EncoderConfig, **kw) -> EncoderConfig:
    d = dict(cfg.__dict__)
    d.update(kw)
    return EncoderConfig(**d)


def round_to(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round fp32 values to the storage dtype (round-to-nearest-even) and return them as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype in ("f32",):
        return a
    t = torch.from_numpy(a)
    if dtype in ("bf16", "i8"):
        return t.to(torch.bfloat16).to(torch.float32).numpy()
    if dtype == "f16":
        return t.to(torch.float16).to(torch.float32).numpy()
    raise ValueError(dtype)


def torch_dtype(dtype: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16, "i8": torch.bfloat16, "f16": torch.float16}[dtype]


def encoder_inputs(cfg: EncoderConfig, seed: int = 0, random_affine: bool = False, layers: int | None = None):
    """Returns (x [T,H] fp32 array holding dtype-rounded values, list of per-layer weight dicts).

    Weights ~N(0, 0.02), inputs ~N(0, 1); biases 0, gamma 1, beta 0 unless ``random_affine``
    (then biases ~N(0,0.02), gamma ~N(1,0.1), beta ~N(0,0.1)) to exercise those paths."""
    rng = np.random.default_rng(seed)
    nl = cfg.layers if layers is None else layers
    H, F = cfg.H, cfg.F
    x = round_to(rng.standard_normal((cfg.T, H), dtype=np.float32), cfg.dtype)
    out = []
    for _ in range(nl):
        w = {}
        w["Wqkv"] = round_to(0.02 * rng.standard_normal((3 * H, H), dtype=np.float32), cfg.dtype)
        w["Wo"] = round_to(0.02 * rng.standard_normal((H, H), dtype=np.float32), cfg.dtype)
        w["W1"] = round_to(0.02 * rng.standard_normal((F, H), dtype=np.float32), cfg.dtype)
        w["W2"] = round_to(0.02 * rng.standard_normal((H, F), dtype=np.float32), cfg.dtype)
        if random_affine:
            w["bqkv"] = (0.02 * rng.standard_normal(3 * H)).astype(np.float32)
            w["bo"] = (0.02 * rng.standard_normal(H)).astype(np.float32)
            w["b1"] = (0.02 * rng.standard_normal(F)).astype(np.float32)
            w["b2"] = (0.02 * rng.standard_normal(H)).astype(np.float32)
            w["g1"] = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
            w["be1"] = (0.1 * rng.standard_normal(H)).astype(np.float32)
            w["g2"] = (1.0 + 0.1 * rng.standard_normal(H)).astype(np.float32)
            w["be2"] = (0.1 * rng.standard_normal(H)).astype(np.float32)
        else:
            w["bqkv"] = np.zeros(3 * H, np.float32)
            w["bo"] = np.zeros(H, np.float32)
            w["b1"] = np.zeros(F, np.float32)
            w["b2"] = np.zeros(H, np.float32)
            w["g1"] = np.ones(H, np.float32)
            w["be1"] = np.zeros(H, np.float32)
            w["g2"] = np.ones(H, np.float32)
            w["be2"] = np.zeros(H, np.float32)
        out.append(w)
    return x, out


def matrix(shape, seed, dtype="f32", scale=1.0):
    """A seeded N(0, scale) matrix rounded to ``dtype`` (returned as fp32)."""
    rng = np.random.default_rng(seed)
    return round_to(scale * rng.standard_normal(shape, dtype=np.float32), dtype)


def int8_matrix(shape, seed, lo=-127, hi=127):
    rng = np.random.default_rng(seed)
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int8)


def pwl_probe_points(x_min, x_max, n, count, seed):
    """fp32 points for table-evaluation tests: uniform over a range 25% wider than the table's,
    plus every breakpoint, its fp32 neighbours, and the special values 0, +-inf."""
    rng = np.random.default_rng(seed)
    span = x_max - x_min
    u = rng.uniform(x_min - 0.25 * span, x_max + 0.25 * span, size=count).astype(np.float32)
    bp = (x_min + (x_max - x_min) * np.arange(n + 1, dtype=np.float64) / n).astype(np.float32)
    near = np.concatenate([bp, np.nextafter(bp, np.float32(np.inf)), np.nextafter(bp, np.float32(-np.inf))])
    special = np.array([0.0, -0.0, np.inf, -np.inf, 1e30, -1e30], np.float32)
    return np.concatenate([u, near, special]).astype(np.float32)


def quantize_weights_per_channel(W: np.ndarray):
    """Symmetric int8 per output channel (row): scale_j = max|W[j,:]| / 127, code = rint(W / scale) in
    [-127, 127] (ties to even).  The int8 codes and fp32 scales ARE the inputs both sides receive."""
    W = np.asarray(W, np.float32)
    s = (np.abs(W).max(axis=1) / np.float32(127.0)).astype(np.float32)
    s = np.maximum(s, np.float32(1e-12))
    q = np.clip(np.rint(W / s[:, None]), -127, 127).astype(np.int8)
    return q, s


def int8_encoder_inputs(cfg: EncoderConfig, layers):
    """Per-layer int8 weights, weight scales and static per-tensor activation scales for the int8 path.
    Activation scales are fixed from the synthetic distributions (inputs and LayerNorm outputs ~N(0,1),
    attention output ~N(0, 0.02^2 H / L), GELU output of N(0, 0.02^2 H)): the same numbers go to both sides."""
    sig_v = 0.02 * np.sqrt(cfg.H)
    scales = {"a_x": 5.5 / 127.0, "a_attn": 6.0 * sig_v / np.sqrt(cfg.L) / 127.0, "a_x1": 5.5 / 127.0,
              "a_g": 4.5 * sig_v / 127.0}
    out = []
    for w in layers:
        d = {k: float(np.float32(v)) for k, v in scales.items()}
        for name in ("Wqkv", "Wo", "W1", "W2"):
            q, s = quantize_weights_per_channel(w[name])
            d[name + "_q"] = q
            d[name + "_s"] = s
        out.append(d)
    return out
