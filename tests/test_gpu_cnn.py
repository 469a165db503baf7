"""GPU parity, CNN path: convolution as GEMM with PWL (ReLU) epilogue, pooling, and the
ResNet-50-shaped network against the oracle on seeded inputs."""
import numpy as np
import pytest
import torch

import nm_inputs
import nm_inputs_cnn
import oracle
import oracle.cnn
from util import assert_close_bf16, load_tables_both, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def relu_tables(ctx):
    return load_tables_both(ctx, 2, {"relu": (-8.0, 8.0)})["relu"]


@pytest.mark.parametrize("N,H,W,Cin,Cout,k,stride,pad", [
    (2, 14, 14, 64, 128, 1, 1, 0),      # 1x1: activation used as the GEMM operand directly
    (2, 14, 14, 64, 64, 3, 1, 1),       # 3x3, Cin = 64: implicit GEMM
    (3, 15, 13, 32, 72, 3, 2, 1),       # odd sizes, stride 2, Cin = 32: explicit gather
    (2, 28, 28, 256, 512, 1, 2, 0),     # strided 1x1 (projection shortcut)
    (2, 40, 40, 3, 64, 7, 2, 3),        # first layer: Cin = 3, padded 8-channel copy, one K-block per filter row
    (1, 9, 9, 16, 8, 5, 1, 2),
])
@pytest.mark.parametrize("epi", ["relu", "relu_res", "res_then_relu", "plain"])
def test_conv2d_parity(nm, ctx, N, H, W, Cin, Cout, k, stride, pad, epi):
    _conv_case(nm, ctx, N, H, W, Cin, Cout, k, stride, pad, epi, nm.ALGO_AUTO)


@pytest.mark.parametrize("N,H,W,Cin,Cout,k,stride,pad", [
    (2, 56, 56, 64, 64, 3, 1, 1),       # stage-1 3x3: 8 x 8 pixel patches of two images, 64-column tile
    (3, 28, 28, 128, 128, 3, 2, 1),     # strided 3x3 (element-strided boxes), odd image count, 128-column tile
    (4, 7, 7, 512, 512, 3, 1, 1),       # 7 x 7 images: a patch spans many images
    (1, 13, 11, 64, 24, 3, 2, 1),       # odd sizes, ragged patches, fewer output channels than a tile
    (5, 9, 9, 128, 320, 3, 1, 1),       # two column tiles, the second ragged
    (2, 17, 17, 192, 64, 5, 1, 2),      # 5x5 taps, three channel blocks
    (2, 33, 29, 3, 32, 7, 2, 3),        # few-channel first layer, odd sizes
    (2, 20, 20, 3, 16, 3, 1, 1),        # few-channel 3x3, stride 1
    (1, 12, 12, 8, 64, 5, 1, 0),        # 8 channels, no padding
])
@pytest.mark.parametrize("algo", ["pairs", "one_cta"])
@pytest.mark.parametrize("epi", ["relu_res", "res_then_relu", "plain"])
def test_conv2d_implicit_gemm_parity(nm, ctx, N, H, W, Cin, Cout, k, stride, pad, epi, algo):
    """Shapes that take the implicit-GEMM forms (one TMA box of the activation per filter tap; the padded
    8-channel copy for a few-channel first layer), with CTA pairs and with one CTA per tile."""
    _conv_case(nm, ctx, N, H, W, Cin, Cout, k, stride, pad, epi, nm.ALGO_TC if algo == "pairs" else nm.ALGO_TC_1CTA)


def test_conv2d_gather_path_still_agrees(nm, ctx):
    """algo = 1 keeps the explicit gather and the CUDA-core GEMM: same answer within the tolerance."""
    _conv_case(nm, ctx, 2, 14, 14, 64, 64, 3, 1, 1, "relu_res", nm.ALGO_SIMT)
    _conv_case(nm, ctx, 2, 20, 20, 3, 16, 3, 1, 1, "relu", nm.ALGO_SIMT)


def _conv_case(nm, ctx, N, H, W, Cin, Cout, k, stride, pad, epi, algo):
    relu = relu_tables(ctx)
    rng = np.random.default_rng(N * 1000 + H + Cin + k)
    x = nm_inputs.round_to(rng.standard_normal((N, H, W, Cin)).astype(np.float32), "f16")
    w = nm_inputs.round_to((np.sqrt(2.0 / (Cin * k * k)) * rng.standard_normal((Cout, k, k, Cin))).astype(np.float32), "f16")
    b = (0.1 * rng.standard_normal(Cout)).astype(np.float32)
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    res = nm_inputs.round_to(rng.standard_normal((N, Ho, Wo, Cout)).astype(np.float32), "f16") if "res" in epi else None
    xd = torch.from_numpy(x).cuda().half()
    wd = torch.from_numpy(w).cuda().half()
    out = torch.full((N, Ho, Wo, Cout), float("nan"), dtype=torch.float16, device="cuda")
    bd = torch.from_numpy(b).cuda()                      # the descriptor holds raw pointers: keep the tensors alive
    rd = torch.from_numpy(res).cuda().half() if res is not None else None
    d = nm.Context.conv_desc(xd, wd, out, stride, pad, bias=bd, residual=rd,
                             slot=nm.SLOT_NONE if epi == "plain" else nm.SLOT_RELU, res_first=(epi == "res_then_relu"),
                             algo=algo)
    ws_bytes = ctx.conv2d_workspace_bytes(d)
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device="cuda")
    ctx.conv2d_pwl(d, ws)
    ctx.check_device_status()
    if epi == "res_then_relu":
        ref = oracle.pwl_eval(relu, oracle.conv2d_nhwc(x, w, stride, pad, b, res, None))[0]
    else:
        ref = oracle.conv2d_nhwc(x, w, stride, pad, b, res, None if epi == "plain" else relu)
    assert_close_bf16(to_np(out), ref, "conv %s" % epi)


@pytest.mark.parametrize("N,H,W,C,dtype", [(128, 7, 7, 2048, "f16"), (5, 7, 7, 200, "f16"), (300, 3, 5, 64, "bf16"),
                                           (2, 1, 300, 72, "f16")])
def test_avgpool_as_gemm(nm, ctx, N, H, W, C, dtype):
    """Global average pool as a tensor-core GEMM with the constant matrix (1/HW) * identity (ragged channel
    blocks, more images than one tile, CTA pairs), and the CUDA-core kernel for a 300-wide image."""
    rng = np.random.default_rng(N + C)
    x = nm_inputs.round_to(rng.standard_normal((N, H, W, C)).astype(np.float32) + 0.5, dtype)
    td = nm_inputs.torch_dtype(dtype)
    xd = torch.from_numpy(x).cuda().to(td)
    a = torch.full((N, C), float("nan"), dtype=td, device="cuda")
    ctx.avgpool_global(xd, a)
    ctx.check_device_status()
    assert_close_bf16(to_np(a), oracle.avgpool_nhwc(x), "avgpool %dx%dx%dx%d %s" % (N, H, W, C, dtype))


def test_pools_parity(nm, ctx):
    rng = np.random.default_rng(5)
    x = nm_inputs.round_to(rng.standard_normal((3, 23, 17, 64)).astype(np.float32), "f16")
    xd = torch.from_numpy(x).cuda().half()
    y = torch.empty((3, 12, 9, 64), dtype=torch.float16, device="cuda")
    ctx.maxpool2d(xd, y, 3, 2, 1)
    assert np.array_equal(to_np(y), oracle.maxpool_nhwc(x, 3, 2, 1))          # a maximum of fp16 values: exact
    a = torch.empty((3, 64), dtype=torch.float16, device="cuda")
    ctx.avgpool_global(xd, a)
    assert_close_bf16(to_np(a), oracle.avgpool_nhwc(x), "avgpool")
    with pytest.raises(nm.NmError) as ei:
        ctx.maxpool2d(xd[..., :12].contiguous(), y, 3, 2, 1)                  # channels not a multiple of 8
    assert ei.value.code == 2


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("ks,stride,pad", [(3, 2, 1), (2, 2, 0), (3, 1, 1)])
def test_maxpool_relu_form(nm, ctx, dtype, ks, stride, pad):
    """max(a, b) = b + PWL_relu(a - b) folded over the window: equals the oracle's fold (and, with the
    2-segment ReLU table, the plain maximum) exactly once rounded to the storage type."""
    rng = np.random.default_rng(31 + ks)
    x = nm_inputs.round_to(3 * rng.standard_normal((2, 21, 19, 32)).astype(np.float32), dtype)
    k, b = ctx.load_function_table(nm.SLOT_RELU, nm.FUNC_RELU, 2, -8.0, 8.0)
    relu = oracle.Table.secant(oracle.RELU, 2, -8.0, 8.0)
    assert np.array_equal(np.asarray(k, np.float32), relu.k) and np.array_equal(np.asarray(b, np.float32), relu.b)
    ref = oracle.maxpool_nhwc_relu(x, ks, stride, pad, relu)
    td = nm_inputs.torch_dtype(dtype)
    xd = torch.from_numpy(x).cuda().to(td)
    y = torch.empty(ref.shape, dtype=td, device="cuda")
    ctx.maxpool2d_pwl(xd, y, ks, stride, pad, nm.SLOT_RELU)
    assert np.array_equal(to_np(y), ref)
    assert np.array_equal(to_np(y), oracle.maxpool_nhwc(x, ks, stride, pad))
    with pytest.raises(nm.NmError) as ei:
        ctx.maxpool2d_pwl(xd, y, ks, stride, pad, 13)      # a slot that was never loaded
    assert ei.value.code == 4


@pytest.mark.parametrize("random_bn", [False, True])
def test_resnet50_two_images(nm, ctx, random_bn):
    """The whole ResNet-50-shaped network (53 convolutions, pools, classifier) on two 224x224 images,
    fp16 NHWC, BatchNorm folded into the convolutions, against the fp64 oracle."""
    from paper_2305_14405_b200.harness_cnn import Resnet50Model
    relu = relu_tables(ctx)
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(2, seed=0, random_bn=random_bn)
    m = Resnet50Model(ctx, 2, convs, fc_w, fc_b)
    logits = m.forward(torch.from_numpy(x).cuda().half())
    ctx.check_device_status()
    ref = oracle.cnn.resnet50(x, convs, fc_w, fc_b, relu)
    got = to_np(logits)
    err = np.abs(got - ref)
    rms = np.sqrt((ref ** 2).mean())
    print("resnet50 logits: max |ref| %.3f, rms ref %.3f, max err %.4f, rms err %.5f"
          % (np.abs(ref).max(), rms, err.max(), np.sqrt((err ** 2).mean())))
    # A logit is a sum of 2048 products of magnitude up to ~1e3 that largely cancel: its rounding error
    # scales with the typical logit magnitude, not with its own value, so elements near zero are held to
    # the bound of an rms-sized element (the same rule as for the fp32 path, at the fp16 tolerance).
    bound = 1e-2 + 1e-2 * np.maximum(np.abs(ref), rms)
    assert np.all(np.isfinite(got)) and not (err > bound).any(), "%d outside" % (err > bound).sum()


@pytest.mark.parametrize("blocks,base", [((1, 1, 1, 1), 64), ((2, 1, 2, 1), 128), ((1, 2, 1, 1), 32)])
def test_resnet_variants(nm, ctx, blocks, base):
    """Depth and width variants of the network (other block counts per stage, first-stage width 128 and 32 --
    the latter takes the gather path for its 32-channel 3x3 convolution) on one image against the oracle."""
    from paper_2305_14405_b200.harness_cnn import Resnet50Model
    relu = relu_tables(ctx)
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(1, seed=2, random_bn=True, num_classes=64, blocks=blocks,
                                                         base_width=base)
    m = Resnet50Model(ctx, 1, convs, fc_w, fc_b, blocks=blocks, base_width=base)
    logits = m.forward(torch.from_numpy(x).cuda().half())
    ctx.check_device_status()
    ref = oracle.cnn.resnet50(x, convs, fc_w, fc_b, relu, blocks=blocks)
    got = to_np(logits)
    err = np.abs(got - ref)
    rms = np.sqrt((ref ** 2).mean())
    bound = 1e-2 + 1e-2 * np.maximum(np.abs(ref), rms)
    assert np.all(np.isfinite(got)) and not (err > bound).any(), "%d outside, max err %.4f" % ((err > bound).sum(), err.max())


def test_resnet_variant_argument_errors(nm, ctx):
    from paper_2305_14405_b200.harness_cnn import Resnet50Model
    cfg = nm.Context.resnet50_cfg(1, nm.F16, blocks=(3, 4, 6, 3), base_width=64)
    assert ctx.resnet_conv_count(cfg) == 53 and ctx.resnet_conv_count(nm.Context.resnet50_cfg(1, nm.F16)) == 53
    assert ctx.resnet_conv_count(nm.Context.resnet50_cfg(1, nm.F16, blocks=(3, 4, 23, 3))) == 104
    for bad in (dict(blocks=(3, 0, 6, 3)), dict(base_width=20), dict(base_width=512), dict(blocks=(1, 1, 1, 99))):
        c = nm.Context.resnet50_cfg(1, nm.F16, **bad)
        assert ctx.resnet_conv_count(c) == 0 and ctx.resnet50_workspace_bytes(c) == 0


def test_resnet50_host_entry_points_two_streams(nm, ctx):
    """The host-buffer forms: the blocking call equals the device-resident forward bit for bit, and four
    asynchronous calls alternating between two streams (own device buffers and workspaces, different images
    per call) equal the blocking call's results."""
    from paper_2305_14405_b200.harness_cnn import Resnet50Model
    relu_tables(ctx)
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(2, seed=3, random_bn=True)
    m = Resnet50Model(ctx, 2, convs, fc_w, fc_b)
    base = torch.from_numpy(x).half()
    xs = [(base * (1.0 - 0.1 * i)).pin_memory() for i in range(4)]
    xd = torch.empty(base.shape, dtype=torch.float16, device="cuda")
    ld = torch.empty((2, fc_w.shape[0]), dtype=torch.float16, device="cuda")
    want = []
    for xh in xs:
        lh = torch.empty((2, fc_w.shape[0]), dtype=torch.float16).pin_memory()
        ctx.resnet50_forward_host(m.array, m.fc_w, m.fc_b, m.cfg, xh, lh, xd, ld, m.workspace)
        want.append(lh.clone())
    assert torch.equal(want[0], m.forward(xs[0].cuda()).cpu())
    slots = [(torch.empty_like(xd), torch.empty_like(ld), torch.empty_like(m.workspace), torch.cuda.Stream())
             for _ in range(2)]
    outs = [torch.empty_like(want[0]).pin_memory() for _ in range(4)]
    torch.cuda.synchronize()
    for i, xh in enumerate(xs):
        sx, sl, ws, st = slots[i % 2]
        ctx.resnet50_forward_host(m.array, m.fc_w, m.fc_b, m.cfg, xh, outs[i], sx, sl, ws, stream=st, wait=False)
    torch.cuda.synchronize()
    ctx.check_device_status()
    for i in range(4):
        assert torch.equal(outs[i], want[i]), i
    assert not torch.equal(want[0], want[1])


def test_resnet50_full_batch_sampled_images(nm, ctx):
    """Config 5 in the benchmark's launch configuration (batch 128, fp16 NHWC, random folded BatchNorm):
    images are independent, so the oracle runs two sampled images through the whole network."""
    from paper_2305_14405_b200.harness_cnn import Resnet50Model
    relu = relu_tables(ctx)
    x, convs, fc_w, fc_b = nm_inputs_cnn.resnet50_inputs(128, seed=0, random_bn=True)
    m = Resnet50Model(ctx, 128, convs, fc_w, fc_b)
    logits = m.forward(torch.from_numpy(x).cuda().half())
    ctx.check_device_status()
    got_all = to_np(logits)
    assert np.all(np.isfinite(got_all))
    for i in (5, 127):
        ref = oracle.cnn.resnet50(x[i:i + 1], convs, fc_w, fc_b, relu)
        rms = np.sqrt((ref ** 2).mean())
        err = np.abs(got_all[i:i + 1] - ref)
        assert not (err > 1e-2 + 1e-2 * np.maximum(np.abs(ref), rms)).any(), "image %d: max err %.3f" % (i, err.max())
