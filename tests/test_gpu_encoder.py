"""GPU parity, whole encoder layers and stacks against the oracle on the seeded workloads."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import assert_close_bf16, assert_close_f32, load_tables_both, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def build(nm, ctx, cfg, layers_np, algo=0):
    from paper_2305_14405_b200.harness import EncoderModel
    return EncoderModel(ctx, cfg, layers_np, algo=algo)


@pytest.mark.parametrize("random_affine", [False, True])
def test_c1_tiny_fp32_layer(nm, ctx, random_affine):
    """Config 1: batch 1, seq 128, hidden 256, 4 heads, FFN 1024, fp32, seed 0, 64-segment tables."""
    cfg = nm_inputs.C1
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0, random_affine=random_affine)
    m = build(nm, ctx, cfg, layers)
    y = m.forward(torch.from_numpy(x).cuda())
    ctx.check_device_status()
    ref = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, tabs, cfg.eps)
    assert_close_f32(to_np(y), ref, "C1 encoder layer")


@pytest.mark.parametrize("algo", [0, 1])
@pytest.mark.parametrize("random_affine", [False, True])
def test_c2_bert_base_layer_bf16(nm, ctx, algo, random_affine):
    """Config 2: batch 8, seq 128, hidden 768, 12 heads, FFN 3072, bf16 with fp32 accumulate."""
    cfg = nm_inputs.C2
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0, random_affine=random_affine)
    m = build(nm, ctx, cfg, layers, algo=algo)
    y = m.forward(torch.from_numpy(x).cuda().bfloat16())
    ctx.check_device_status()
    ref = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, tabs, cfg.eps)
    assert_close_bf16(to_np(y), ref, "C2 encoder layer algo %d" % algo)


def test_c2_layer_with_calibrated_table_ranges(nm, ctx):
    """The table ranges observed by running the exact model (Section 3.2.1 step 1; tests/golden/
    calibrated_ranges.json) instead of the fixed ones: same bound against the oracle with the same tables, and
    the result is closer to the exact-nonlinearity layer than with the fixed ranges."""
    cfg = nm_inputs.C2
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0)
    m = build(nm, ctx, cfg, layers)
    exact = {"gelu": oracle.Table.exact(oracle.GELU), "exp": oracle.Table.exact(oracle.EXP),
             "recip": oracle.Table.exact(oracle.RECIP), "rsqrt": oracle.Table.exact(oracle.RSQRT)}
    ref_exact = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, exact, cfg.eps)
    dist = {}
    for mode in (False, True):
        tabs = load_tables_both(ctx, cfg.segments, cfg.ranges(calibrated=mode))
        y = m.forward(torch.from_numpy(x).cuda().bfloat16())
        ctx.check_device_status()
        ref = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, tabs, cfg.eps)
        assert_close_bf16(to_np(y), ref, "C2 layer, %s ranges" % ("calibrated" if mode else "fixed"))
        dist[mode] = float(np.sqrt(((ref - ref_exact) ** 2).mean()))
    print("C2 layer, rms |PWL oracle - exact oracle|: fixed %.3e, calibrated %.3e" % (dist[False], dist[True]))
    assert dist[True] < dist[False]
    load_tables_both(ctx, cfg.segments, cfg.ranges())


@pytest.mark.parametrize("H,L", [(512, 256), (1024, 128), (1536, 128)])
def test_width_sweep_layer_bf16(nm, ctx, H, L):
    """Widths of the width/depth sweep (heads of 64, FFN 4H): one layer, two sequences, random biases and
    LayerNorm parameters."""
    cfg = nm_inputs.with_(nm_inputs.C2, B=2, L=L, H=H, heads=H // 64, F=4 * H, name="sweep_H%d" % H)
    tabs = load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=H, random_affine=True)
    m = build(nm, ctx, cfg, layers)
    y = m.forward(torch.from_numpy(x).cuda().bfloat16())
    ctx.check_device_status()
    ref = oracle.encoder_layer(x, layers[0], cfg.B, cfg.L, cfg.heads, tabs, cfg.eps)
    if H <= 1024:   # the widths of the stated configurations: the stated per-element bound
        assert_close_bf16(to_np(y), ref, "encoder layer H=%d" % H)
    else:
        # Beyond them the rounding noise of a K-term sum of bf16 operands keeps growing like sqrt(K)
        # (FFN2 has K = 4H) while the bound stays put: at H = 1536 about 5 elements per million of
        # near-zero reference value cross it.  Asserted: < 1e-4 of the elements outside the bound,
        # none outside twice the bound.
        got = np.asarray(to_np(y), np.float64)
        err = np.abs(got - ref)
        bound = 1e-2 + 1e-2 * np.abs(ref)
        assert np.all(np.isfinite(got))
        assert (err > bound).mean() < 1e-4, (err > bound).mean()
        assert not (err > 2 * bound).any(), err.max()


@pytest.mark.parametrize("n", [16, 64, 256])
def test_c3_stack_sampled_sequences(nm, ctx, n):
    """Config 3 in the benchmark's launch configuration (12 layers, batch 32, seq 512, bf16).
    Sequences are independent, so the oracle runs whole sampled sequences: per layer from the
    GPU's own bf16 layer input, and end to end through all 12 layers."""
    cfg = nm_inputs.with_(nm_inputs.C3, segments=n)
    tabs = load_tables_both(ctx, n, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=0)
    m = build(nm, ctx, cfg, layers)
    xd = torch.from_numpy(x).cuda().bfloat16()
    L = cfg.L
    # per layer: feed each layer the previous GPU output, compare one sequence per layer
    cur = xd
    for li in range(cfg.layers):
        nxt = m.forward_layer(li, cur)
        if li in (0, 5, 11):
            b = (7 * li + 3) % cfg.B
            xin = to_np(cur[b * L:(b + 1) * L])
            ref = oracle.encoder_layer(xin, layers[li], 1, L, cfg.heads, tabs, cfg.eps)
            assert_close_bf16(to_np(nxt[b * L:(b + 1) * L]), ref, "C3 layer %d, sequence %d, n=%d" % (li, b, n))
        cur = nxt
    ctx.check_device_status()
    # end to end in one call; must equal the layer-by-layer result bit for bit
    y = m.forward(xd)
    ctx.check_device_status()
    assert torch.equal(y, cur)
    if n == 64:
        b = 17
        ref = oracle.encoder_stack(x[b * L:(b + 1) * L], layers, 1, L, cfg.heads, tabs, cfg.eps)
        got = to_np(y[b * L:(b + 1) * L])
        err = np.abs(got - ref)
        bound = 1e-2 + 1e-2 * np.abs(ref)
        frac1 = float((err > bound).mean())
        # Each layer meets the per-element bound from the same bf16 input (checked above).  Over 12
        # layers the bf16 rounding of the stored activations is re-injected at every layer while the
        # fp64 oracle rounds nothing; LayerNorm keeps the perturbation gain near one, so independent
        # per-layer errors add in quadrature: the end-to-end bound is sqrt(layers) times the per-layer one.
        k = np.sqrt(cfg.layers)
        frac = float((err > k * bound).mean())
        print("C3 end-to-end: max err %.4f, rms err %.5f, outside 1x bound %.5f, outside sqrt(12)x bound %.6f"
              % (err.max(), np.sqrt((err ** 2).mean()), frac1, frac))
        # the quadrature bound is a ~3.5 sigma statement, so a handful of elements in 393216 may pass it
        assert frac < 1e-3 and err.max() < 0.15 and np.sqrt((err ** 2).mean()) < 0.02


def test_encoder_host_entry_point(nm, ctx):
    cfg = nm_inputs.with_(nm_inputs.C2, B=2)
    load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=1, layers=2)
    m = build(nm, ctx, cfg, layers)
    xh = torch.from_numpy(x).bfloat16().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    xd = torch.empty(xh.shape, dtype=torch.bfloat16, device="cuda")
    yd = torch.empty_like(xd)
    ctx.encoder_stack_host(m.array, m.n_layers, m.ccfg, xh, yh, xd, yd, m.workspace)
    y = m.forward(xh.cuda())
    torch.cuda.synchronize()
    assert torch.equal(yh, y.cpu())


def test_encoder_host_entry_point_async_two_streams(nm, ctx):
    """Six asynchronous host-buffer calls alternating between two streams, each with its own device buffers and
    workspace, different inputs per call: every result equals the blocking call's."""
    cfg = nm_inputs.with_(nm_inputs.C2, B=2)
    load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=1, layers=2)
    m = build(nm, ctx, cfg, layers)
    base = torch.from_numpy(x).bfloat16()
    xs = [(base * (1.0 + 0.05 * i)).pin_memory() for i in range(6)]
    want = []
    xd = torch.empty(base.shape, dtype=torch.bfloat16, device="cuda")
    yd = torch.empty_like(xd)
    for xh in xs:
        yh = torch.empty_like(xh).pin_memory()
        ctx.encoder_stack_host(m.array, m.n_layers, m.ccfg, xh, yh, xd, yd, m.workspace)
        want.append(yh.clone())
    slots = [(torch.empty_like(xd), torch.empty_like(yd), torch.empty_like(m.workspace), torch.cuda.Stream())
             for _ in range(2)]
    outs = [torch.empty_like(xs[0]).pin_memory() for _ in range(6)]
    torch.cuda.synchronize()
    for i, xh in enumerate(xs):
        sx, sy, ws, st = slots[i % 2]
        ctx.encoder_stack_host(m.array, m.n_layers, m.ccfg, xh, outs[i], sx, sy, ws, stream=st, wait=False)
    torch.cuda.synchronize()
    ctx.check_device_status()
    for i in range(6):
        assert torch.equal(outs[i], want[i]), i
    assert not torch.equal(want[0], want[1])


def test_encoder_workspace_errors(nm, ctx):
    cfg = nm_inputs.with_(nm_inputs.C2, B=1)
    load_tables_both(ctx, cfg.segments, cfg.ranges())
    x, layers = nm_inputs.encoder_inputs(cfg, seed=1)
    m = build(nm, ctx, cfg, layers)
    xd = torch.from_numpy(x).cuda().bfloat16()
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.encoder_layer(m.structs[0], m.ccfg, xd, torch.empty_like(xd), small)
    assert ei.value.code == 8
    with pytest.raises(nm.NmError) as ei:
        ctx.encoder_layer(m.structs[0], m.ccfg, xd, xd, m.workspace)
    assert ei.value.code == 1
