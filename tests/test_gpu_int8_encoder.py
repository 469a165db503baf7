"""GPU parity, int8 encoder layers (config 4 shapes: hidden 1024, 16 heads, FFN 4096, seq 512): the
four weight GEMMs run as int8 x int8 -> int32 on the tensor cores with an fp32 epilogue; checked per
layer against the oracle's int8 evaluation on the same int8 weights, scales and bf16 layer input."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import assert_close_bf16, load_tables_both, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def test_c4_int8_layers_sampled(nm, ctx):
    from paper_2305_14405_b200.harness import EncoderModel
    cfg = nm_inputs.with_(nm_inputs.C4, B=4, layers=3)
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0, random_affine=True)
    quant = nm_inputs.int8_encoder_inputs(cfg, layers)
    m = EncoderModel(ctx, cfg, layers, quant=quant)
    L = cfg.L
    cur = torch.from_numpy(x).cuda().bfloat16()
    for li in range(cfg.layers):
        nxt = m.forward_layer(li, cur)
        ctx.check_device_status()
        b = (li + 1) % cfg.B
        xin = to_np(cur[b * L:(b + 1) * L])
        ref = oracle.encoder_layer_i8(xin, layers[li], quant[li], 1, L, cfg.heads, tabs, cfg.eps)
        got = to_np(nxt[b * L:(b + 1) * L])
        # Quantised codes are integer decisions taken from floating-point activations.  The oracle takes
        # them in the workload's storage precision (bf16), yet ~30 % of the attention outputs still differ
        # from the GPU's by one bf16 ulp (the GPU sums bf16 probabilities in fp32), a few per cent of the
        # int8 codes downstream move to the neighbouring code, and FFN2 sums 4096 of them: the layer
        # output carries an error of std ~6e-3 on top of the usual bf16 rounding.  So the per-element
        # bf16 bound is asserted for 99 % of the elements, with rms and maximum bounds for the rest;
        # exactness of the int8 arithmetic itself is asserted per GEMM in test_gpu_linear.py.
        err = np.abs(got - ref)
        bad = err > 1e-2 + 1e-2 * np.abs(ref)
        rms = np.sqrt((err ** 2).mean())
        print("int8 layer %d: max err %.4f, rms %.5f, outside bound %d / %d" % (li, err.max(), rms, bad.sum(), bad.size))
        assert bad.mean() < 1e-2 and rms < 1e-2 and err.max() < 0.1
        cur = nxt
    y = m.forward(torch.from_numpy(x).cuda().bfloat16())
    assert torch.equal(y, cur)


def test_c4_full_size_launch_configuration(nm, ctx):
    """The 24-layer, batch-16 stack in one call: every launch at its full size; output finite and equal
    to the layer-by-layer run."""
    from paper_2305_14405_b200.harness import EncoderModel
    cfg = nm_inputs.C4
    load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=1, layers=2)
    layers = [layers[i % 2] for i in range(cfg.layers)]          # 24 layers cycling two weight sets
    quant2 = nm_inputs.int8_encoder_inputs(cfg, layers[:2])
    quant = [quant2[i % 2] for i in range(cfg.layers)]
    m = EncoderModel(ctx, cfg, layers, quant=quant)
    xd = torch.from_numpy(x).cuda().bfloat16()
    y = m.forward(xd)
    ctx.check_device_status()
    assert torch.isfinite(y.float()).all()
    cur = xd
    for li in range(cfg.layers):
        cur = m.forward_layer(li, cur)
    assert torch.equal(y, cur)
