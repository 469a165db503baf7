"""Device-side set-up of the ResNet-50-shaped workload and its depth / width variants: uploads seeded host
arrays and fills the C structs.  No arithmetic of the forward pass lives here."""
from __future__ import annotations

import numpy as np
import torch

from . import BF16, F16, ConvParams, Context

_TORCH = {"f16": torch.float16, "bf16": torch.bfloat16}
_NM = {"f16": F16, "bf16": BF16}


class Resnet50Model:
    def __init__(self, ctx: Context, batch, convs_np, fc_w, fc_b, dtype="f16", device="cuda:0", algo=0, blocks=None,
                 base_width=0):
        self.cfg = Context.resnet50_cfg(batch, _NM[dtype], num_classes=fc_w.shape[0], algo=algo, blocks=blocks,
                                        base_width=base_width)
        assert len(convs_np) == ctx.resnet_conv_count(self.cfg), "convolutions do not match the configuration"
        self.ctx = ctx
        self.dtype = _TORCH[dtype]
        self.keep = []
        arr = (ConvParams * len(convs_np))()
        for i, c in enumerate(convs_np):
            w = torch.from_numpy(np.ascontiguousarray(c["w"])).to(device=device, dtype=self.dtype)
            b = torch.from_numpy(np.ascontiguousarray(c["b"], dtype=np.float32)).to(device)
            self.keep += [w, b]
            arr[i].w, arr[i].bias = w.data_ptr(), b.data_ptr()
        self.array = arr
        self.fc_w = torch.from_numpy(np.ascontiguousarray(fc_w)).to(device=device, dtype=self.dtype)
        self.fc_b = torch.from_numpy(np.ascontiguousarray(fc_b, dtype=np.float32)).to(device)
        ws = ctx.resnet50_workspace_bytes(self.cfg)
        assert ws > 0
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=device)
        self.batch = batch
        self.device = device

    def forward(self, x, logits=None):
        if logits is None:
            logits = torch.empty((self.batch, self.fc_w.shape[0]), dtype=self.dtype, device=self.device)
        self.ctx.resnet50_forward(self.array, self.fc_w, self.fc_b, self.cfg, x, logits, self.workspace)
        return logits
