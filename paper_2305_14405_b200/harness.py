"""Device-side set-up shared by the tests, the benchmark and the smoke check: moves seeded
host arrays into device tensors of the workload's dtype and fills the C structs.  No
arithmetic of the forward pass lives here."""
from __future__ import annotations

import numpy as np
import torch

from . import BF16, F32, I8, Context, layer_array

_TORCH = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16, "i8": torch.bfloat16}
_NM = {"f32": F32, "bf16": BF16, "i8": I8}


def to_device(a: np.ndarray, dtype: str, device="cuda:0"):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device=device, dtype=_TORCH[dtype])


def f32_device(a: np.ndarray, device="cuda:0"):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


class EncoderModel:
    """Weights of an encoder stack resident on the device plus the workspace the library needs."""

    def __init__(self, ctx: Context, cfg, layers_np, device="cuda:0", algo=0, quant=None):
        self.ctx = ctx
        self.cfg = cfg
        self.device = device
        self.ccfg = Context.encoder_cfg(cfg.B, cfg.L, cfg.H, cfg.heads, cfg.F, _NM[cfg.dtype], cfg.eps, algo)
        self.tensors = []  # keeps device memory alive
        structs = []
        for li, w in enumerate(layers_np):
            d = {}
            for name in ("Wqkv", "Wo", "W1", "W2"):
                if cfg.dtype == "i8":
                    d[name] = torch.from_numpy(np.ascontiguousarray(quant[li][name + "_q"])).to(device)
                    d["s_w" + name[1:].lower()] = f32_device(quant[li][name + "_s"], device)
                else:
                    d[name] = to_device(w[name], cfg.dtype, device)
            for name in ("bqkv", "bo", "b1", "b2", "g1", "be1", "g2", "be2"):
                d[name] = f32_device(w[name], device)
            if cfg.dtype == "i8":
                for name in ("a_x", "a_attn", "a_x1", "a_g"):
                    d[name] = float(quant[li][name])
            self.tensors.append(d)
            structs.append(Context.encoder_weights(d))
        self.structs = structs
        self.array = layer_array(structs)
        self.n_layers = len(structs)
        ws = ctx.encoder_workspace_bytes(self.ccfg)
        assert ws > 0, "bad encoder configuration"
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=device)

    def act_dtype(self):
        return _TORCH[self.cfg.dtype]

    def forward(self, x, y=None):
        if y is None:
            y = torch.empty_like(x)
        self.ctx.encoder_stack(self.array, self.n_layers, self.ccfg, x, y, self.workspace)
        return y

    def forward_layer(self, li, x, y=None):
        if y is None:
            y = torch.empty_like(x)
        self.ctx.encoder_layer(self.structs[li], self.ccfg, x, y, self.workspace)
        return y
