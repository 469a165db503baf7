"""GPU parity, int8 encoder (config 4 shapes: hidden 1024, 16 heads, FFN 4096, seq 512): the four weight
GEMMs run as int8 x int8 -> int32 on the tensor cores with an fp32 epilogue.

What is asserted, and against what:
 * stage by stage with the integer decisions shared (every int8 code the GPU feeds a GEMM is handed to the
   oracle as that GEMM's operand): int32 accumulators, segment numbers and int8 codes bit-exact, every
   floating-point output within |gpu - oracle| <= 1e-2 + 1e-2*|oracle| on EVERY element;
 * free-running (the oracle takes its own integer decisions from its own fp64 activations): the share of
   int8 codes that differ and by how much, and the deviation of a layer / of the whole 24-layer stack from the
   definition-level oracle (which rounds nothing) and from its bf16-storage model, reported and bounded.
"""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import assert_close_bf16, load_tables_both, rms_rel, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def _bf16_round(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).bfloat16().float().numpy()


def _inv(scale):
    return float(np.float32(1.0) / np.float32(scale))


def test_c4_layer_stage_by_stage_with_shared_integer_decisions(nm, ctx):
    """One config-4 layer (two sequences) driven stage by stage through the C ABI, so that every tensor
    exists on the device; each stage is compared with the oracle run on the GPU's own operands of that
    stage.  The fused layer call must reproduce the staged result bit for bit (its kernels emit the int8
    codes themselves instead of running the separate quantisation pass)."""
    from paper_2305_14405_b200.harness import EncoderModel
    cfg = nm_inputs.with_(nm_inputs.C4, B=2, layers=1)
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x_np, layers = nm_inputs.encoder_inputs(cfg, seed=4, random_affine=True)
    w = layers[0]
    q = nm_inputs.int8_encoder_inputs(cfg, layers)[0]
    m = EncoderModel(ctx, cfg, layers, quant=[q])
    d = m.tensors[0]
    T, H, F, h = cfg.T, cfg.H, cfg.F, cfg.heads
    dev = "cuda"
    x = torch.from_numpy(x_np).to(dev).bfloat16()

    def i8(shape):
        return torch.empty(shape, dtype=torch.int8, device=dev)

    def bf(shape):
        return torch.full(shape, float("nan"), dtype=torch.bfloat16, device=dev)

    def i32(shape):
        return torch.full(shape, -12345, dtype=torch.int32, device=dev)

    # ---- the GPU, stage by stage
    xq = i8((T, H)); ctx.quantize_i8(x, _inv(q["a_x"]), xq)
    qkv, acc_qkv = bf((T, 3 * H)), i32((T, 3 * H))
    ctx.linear_pwl(xq, d["Wqkv"], qkv, bias=d["bqkv"], a_scale=q["a_x"], w_scale=d["s_wqkv"], acc_dump=acc_qkv)
    attn = bf((T, H)); ctx.attention_pwl(qkv, attn, cfg.B, cfg.L, h, cfg.d)
    aq = i8((T, H)); ctx.quantize_i8(attn, _inv(q["a_attn"]), aq)
    z, acc_o = bf((T, H)), i32((T, H))
    ctx.linear_pwl(aq, d["Wo"], z, bias=d["bo"], residual=x, a_scale=q["a_attn"], w_scale=d["s_wo"], acc_dump=acc_o)
    x1 = bf((T, H)); ctx.layernorm_pwl(z, d["g1"], d["be1"], x1, eps=cfg.eps)
    x1q = i8((T, H)); ctx.quantize_i8(x1, _inv(q["a_x1"]), x1q)
    gq, acc_1, idx_1 = i8((T, F)), i32((T, F)), i32((T, F))
    ctx.linear_pwl(x1q, d["W1"], gq, bias=d["b1"], slot=nm.SLOT_GELU, a_scale=q["a_x1"], w_scale=d["s_w1"],
                   inv_out_scale=_inv(q["a_g"]), acc_dump=acc_1, idx_dump=idx_1)
    z2, acc_2 = bf((T, H)), i32((T, H))
    ctx.linear_pwl(gq, d["W2"], z2, bias=d["b2"], residual=x1, a_scale=q["a_g"], w_scale=d["s_w2"], acc_dump=acc_2)
    y = bf((T, H)); ctx.layernorm_pwl(z2, d["g2"], d["be2"], y, eps=cfg.eps)
    ctx.check_device_status()
    y_fused = m.forward_layer(0, x)
    ctx.check_device_status()
    assert torch.equal(y_fused, y), "the fused layer differs from its stages"

    # ---- the oracle, each stage from the GPU's operands of that stage
    c = lambda t: t.cpu().numpy()
    f = lambda t: t.float().cpu().numpy()
    assert np.array_equal(c(xq), oracle.quantize_i8(x_np, q["a_x"]))
    r = oracle.linear_i8(c(xq), q["Wqkv_q"], q["a_x"], q["Wqkv_s"], w["bqkv"])
    assert np.array_equal(c(acc_qkv), r["acc"]), "QKV accumulators"
    assert np.array_equal(f(qkv), _bf16_round(r["y"])), "QKV output (bf16 of the fp32 epilogue value)"
    assert_close_bf16(f(qkv), r["y"], "C4 stage qkv")

    ref = oracle.attention(f(qkv), cfg.B, cfg.L, h, cfg.d, tabs["exp"], tabs["recip"])
    assert_close_bf16(f(attn), ref, "C4 stage attention")
    assert np.array_equal(c(aq), oracle.quantize_i8(f(attn), q["a_attn"]))

    r = oracle.linear_i8(c(aq), q["Wo_q"], q["a_attn"], q["Wo_s"], w["bo"], residual=x_np)
    assert np.array_equal(c(acc_o), r["acc"]), "out-projection accumulators"
    assert np.array_equal(f(z), _bf16_round(r["y"]))
    assert_close_bf16(f(z), r["y"], "C4 stage out-projection + residual")

    ref = oracle.layernorm(f(z), w["g1"], w["be1"], cfg.eps, tabs["rsqrt"])
    assert_close_bf16(f(x1), ref, "C4 stage LayerNorm 1")
    assert np.array_equal(c(x1q), oracle.quantize_i8(f(x1), q["a_x1"]))

    r = oracle.linear_i8(c(x1q), q["W1_q"], q["a_x1"], q["W1_s"], w["b1"], table=tabs["gelu"], out_scale=q["a_g"])
    assert np.array_equal(c(acc_1), r["acc"]), "FFN1 accumulators"
    assert np.array_equal(c(idx_1), r["idx"]), "FFN1 segment numbers"
    assert np.array_equal(c(gq), r["q"]), "FFN1 int8 output codes"

    r = oracle.linear_i8(c(gq), q["W2_q"], q["a_g"], q["W2_s"], w["b2"], residual=f(x1))
    assert np.array_equal(c(acc_2), r["acc"]), "FFN2 accumulators"
    assert np.array_equal(f(z2), _bf16_round(r["y"]))
    assert_close_bf16(f(z2), r["y"], "C4 stage FFN2 + residual")

    ref = oracle.layernorm(f(z2), w["g2"], w["be2"], cfg.eps, tabs["rsqrt"])
    assert_close_bf16(f(y), ref, "C4 stage LayerNorm 2")

    # ---- free-running: the definition-level oracle decides its own codes from its own activations
    yd, st = oracle.encoder_layer_i8(x_np, w, q, cfg.B, cfg.L, h, tabs, cfg.eps, want_stages=True)
    for name, gpu_codes, act, scale in (("attention output", aq, st["a"], q["a_attn"]), ("LN1 output", x1q, st["x1"], q["a_x1"]),
                                        ("GELU output", gq, st["g"], q["a_g"])):
        _, oc = oracle.fake_quant(act, scale, want_codes=True)
        diff = np.abs(c(gpu_codes).astype(np.int32) - oc.astype(np.int32))
        print("free-running codes, %s: %.3f %% differ, max difference %d" % (name, 100 * (diff > 0).mean(), diff.max()))
        # neighbouring codes, except after the GELU: its input codes already differ here and there, which moves
        # an FFN1 accumulator, and with it the output, by more than one step of the output scale
        assert (diff > 0).mean() < 0.15 and diff.max() <= (2 if name == "GELU output" else 1), name
    ys = oracle.encoder_layer_i8_storage(x_np, w, q, cfg.B, cfg.L, h, tabs, cfg.eps)
    _check_free_running(f(y), yd, ys, "staged layer")


# Free-running comparison of one int8 layer (both sides start from the same bf16 layer input and take
# their own integer decisions).  Against the bf16-storage model >= 99 % of the elements hold the
# per-element bound; against the definition, which rounds no activation, the bf16 roundings of the
# workload's stored activations move 4-9 % of the int8 codes to a neighbour and ~6 % of the outputs
# leave the bound, with rms(err)/rms(ref) below 1 %: the stated per-element bound is NOT met for every
# element in this mode (it is, for every element, with the integer decisions shared: the staged test).
def _check_free_running(got, ref_def, ref_storage, what):
    for name, ref, frac_max, rr_max in (("definition", ref_def, 0.10, 1.5e-2), ("bf16-storage model", ref_storage, 1e-2, 1e-2)):
        err = np.abs(got - ref)
        bad = err > 1e-2 + 1e-2 * np.abs(ref)
        rr = rms_rel(got, ref)
        print("free-running %s vs %s: outside bound %d / %d (%.3f %%), max err %.4f, rms(err)/rms(ref) %.5f"
              % (what, name, bad.sum(), bad.size, 100 * bad.mean(), err.max(), rr))
        assert np.all(np.isfinite(got))
        assert bad.mean() < frac_max and rr < rr_max and err.max() < 0.1, (what, name)


def test_c4_int8_layers_sampled(nm, ctx):
    """Three layers at batch 4, each compared with the oracle started from the GPU's own bf16 layer input,
    free-running inside the layer (see _check_free_running for what holds in this mode)."""
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
        got = to_np(nxt[b * L:(b + 1) * L])
        args = (xin, layers[li], quant[li], 1, L, cfg.heads, tabs, cfg.eps)
        _check_free_running(got, oracle.encoder_layer_i8(*args), oracle.encoder_layer_i8_storage(*args), "layer %d" % li)
        cur = nxt
    y = m.forward(torch.from_numpy(x).cuda().bfloat16())
    assert torch.equal(y, cur)


def test_c4_full_stack_against_oracle(nm, ctx):
    """Config 4 as a config: 24 layers with 24 independent weight sets, batch 16, one call, every launch at
    its full size.  One whole sequence is compared end to end with the definition-level oracle (and with
    its bf16-storage model); three layers are compared per layer from the GPU's own layer input; the
    one-call stack equals the layer-by-layer run bit for bit."""
    from paper_2305_14405_b200.harness import EncoderModel
    cfg = nm_inputs.C4
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=1)
    assert len(layers) == 24 and not np.array_equal(layers[0]["Wqkv"], layers[1]["Wqkv"])
    quant = nm_inputs.int8_encoder_inputs(cfg, layers)
    m = EncoderModel(ctx, cfg, layers, quant=quant)
    xd = torch.from_numpy(x).cuda().bfloat16()
    y = m.forward(xd)
    ctx.check_device_status()
    assert torch.isfinite(y.float()).all()
    L = cfg.L
    cur = xd
    for li in range(cfg.layers):
        nxt = m.forward_layer(li, cur)
        if li in (0, 11, 23):
            b = (5 * li + 2) % cfg.B
            xin = to_np(cur[b * L:(b + 1) * L])
            got = to_np(nxt[b * L:(b + 1) * L])
            args = (xin, layers[li], quant[li], 1, L, cfg.heads, tabs, cfg.eps)
            _check_free_running(got, oracle.encoder_layer_i8(*args), oracle.encoder_layer_i8_storage(*args),
                                "C4 layer %d, sequence %d" % (li, b))
        cur = nxt
    assert torch.equal(y, cur)
    # end to end: sequence 9 through all 24 layers
    b = 9
    got = to_np(y[b * L:(b + 1) * L])
    xin = x[b * L:(b + 1) * L]
    refs = {}
    for name, fn in (("definition", oracle.encoder_layer_i8), ("bf16-storage model", oracle.encoder_layer_i8_storage)):
        ref = xin
        for li in range(cfg.layers):
            ref = fn(ref, layers[li], quant[li], 1, L, cfg.heads, tabs, cfg.eps)
        refs[name] = ref
    # the yardstick: how far the int8 evaluation itself is from the same network without activation
    # quantisation (same dequantised weights, fp64): the method's own quantisation noise after 24 layers
    ref = xin
    for li in range(cfg.layers):
        wd = dict(layers[li])
        for n_ in ("Wqkv", "Wo", "W1", "W2"):
            wd[n_] = quant[li][n_ + "_q"].astype(np.float64) * quant[li][n_ + "_s"].astype(np.float64)[:, None]
        ref = oracle.encoder_layer(ref, wd, 1, L, cfg.heads, tabs, cfg.eps)
    noise = rms_rel(refs["definition"], ref)
    print("C4 end to end: int8 definition vs the unquantised-activation network: rms(diff)/rms %.5f" % noise)
    for name, ref in refs.items():
        err = np.abs(got - ref)
        bound = 1e-2 + 1e-2 * np.abs(ref)
        k = np.sqrt(cfg.layers)
        print("C4 end to end (24 layers) vs %s: outside 1x bound %.4f, outside sqrt(24)x bound %.5f, max err %.4f, "
              "rms err %.5f, rms(err)/rms(ref) %.5f"
              % (name, (err > bound).mean(), (err > k * bound).mean(), err.max(), np.sqrt((err ** 2).mean()), rms_rel(got, ref)))
    # Per layer the GPU is 0.85 % (rms) from the definition and 0.5 % from the storage model (checked above);
    # over 24 layers these add up roughly in quadrature with some gain.  The per-element bound is not met end
    # to end (it is not claimed); asserted: the deviation stays below the int8 evaluation's own quantisation
    # noise over the same 24 layers, and below 10 % in rms.
    rr = rms_rel(got, refs["definition"])
    assert rr < 0.10 and rr < noise and np.abs(got - refs["definition"]).max() < 0.6
    assert rms_rel(got, refs["bf16-storage model"]) < 0.10
