"""GPU parity, HBM-bound row kernels: table evaluation, LayerNorm, int8 quantisation."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import FUNCS, assert_close_bf16, assert_close_f32, load_tables_both, to_np

pytestmark = pytest.mark.gpu

RANGES = {"gelu": (-4.0, 4.0), "exp": (-8.0, 0.0), "recip": (8.0, 128.0), "rsqrt": (0.25, 4.0), "relu": (-3.0, 3.0)}


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("name", list(RANGES))
@pytest.mark.parametrize("n", [2, 16, 64, 256])
def test_pwl_apply_f32_bit_exact(nm, ctx, name, n):
    """Segment numbers and fp32 values are bit-exact: both sides take the index with one fp32
    fused multiply-add and evaluate fma(k, x, b)."""
    lo, hi = RANGES[name]
    tabs = load_tables_both(ctx, n, {name: (lo, hi)})
    x = nm_inputs.pwl_probe_points(lo, hi, n, 100003, seed=n)   # ragged count
    xd = torch.from_numpy(x).cuda()
    yd = torch.empty_like(xd)
    idx = torch.empty(x.size, dtype=torch.int32, device="cuda")
    from util import SLOTS
    ctx.pwl_apply(SLOTS[name], xd, yd, idx)
    ctx.check_device_status()
    y_ref, idx_ref = oracle.pwl_eval_f32(tabs[name], x)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)
    got = yd.cpu().numpy()
    nan = np.isnan(y_ref)                     # e.g. 0 * inf; the payload of a NaN is not compared
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), y_ref[~nan].view(np.uint32))


def test_pwl_apply_nan_and_empty(nm, ctx):
    load_tables_both(ctx, 64, {"gelu": RANGES["gelu"]})
    x = torch.tensor([float("nan"), 1.0, float("nan"), -2.0, 0.5, 0.25, 8.0, -8.0], device="cuda")
    y = torch.empty_like(x)
    idx = torch.empty(8, dtype=torch.int32, device="cuda")
    ctx.pwl_apply(nm.SLOT_GELU, x, y, idx)
    assert idx[0].item() == 0 and torch.isnan(y[0]) and idx[2].item() == 0
    e = torch.empty(0, device="cuda")
    ctx.pwl_apply(nm.SLOT_GELU, e, e)          # zero elements: a no-op, not an error
    with pytest.raises(nm.NmError) as ei:
        ctx.pwl_apply(9, x, y)                 # slot never loaded
    assert ei.value.code == 4


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_pwl_apply_half_types(nm, ctx, dtype):
    tabs = load_tables_both(ctx, 64, {"gelu": RANGES["gelu"]})
    x = nm_inputs.round_to(nm_inputs.matrix((1 << 16) + 24, 3, "f32", 2.0), dtype)
    td = nm_inputs.torch_dtype(dtype)
    xd = torch.from_numpy(x).cuda().to(td)
    yd = torch.empty_like(xd)
    idx = torch.empty(x.size, dtype=torch.int32, device="cuda")
    ctx.pwl_apply(nm.SLOT_GELU, xd, yd, idx)
    y_ref, idx_ref = oracle.pwl_eval_f32(tabs["gelu"], x)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)
    want = torch.from_numpy(y_ref).to(td)       # the same fp32 value, rounded to the storage type
    assert torch.equal(yd.cpu(), want)
    assert torch.isfinite(want.float()).all()


@pytest.mark.parametrize("dtype,rows,H", [("f32", 128, 256), ("f32", 77, 1000), ("bf16", 1024, 768), ("bf16", 333, 1024),
                                          ("bf16", 64, 4096), ("f16", 100, 768), ("bf16", 5, 8)])
def test_layernorm_parity(nm, ctx, dtype, rows, H):
    tabs = load_tables_both(ctx, 64, {"rsqrt": RANGES["rsqrt"]})
    rng = np.random.default_rng(rows + H)
    z = nm_inputs.round_to((rng.standard_normal((rows, H)) * rng.uniform(0.6, 1.8, (rows, 1)) + 0.3).astype(np.float32), dtype)
    g = (1 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    b = (0.1 * rng.standard_normal(H)).astype(np.float32)
    td = nm_inputs.torch_dtype(dtype)
    zd = torch.from_numpy(z).cuda().to(td)
    yd = torch.empty_like(zd)
    ctx.layernorm_pwl(zd, torch.from_numpy(g).cuda(), torch.from_numpy(b).cuda(), yd, eps=1e-5)
    ref = oracle.layernorm(z, g, b, 1e-5, tabs["rsqrt"])
    if dtype == "f32":
        assert_close_f32(to_np(yd), ref, "layernorm f32")
    else:
        assert_close_bf16(to_np(yd), ref, "layernorm " + dtype)


@pytest.mark.parametrize("dtype,rows,H,n", [("f32", 96, 256, 64), ("bf16", 1024, 768, 64), ("bf16", 333, 1024, 16),
                                            ("f16", 100, 768, 256), ("bf16", 5, 8, 64)])
def test_layernorm_sqrt_recip_parity(nm, ctx, dtype, rows, H, n):
    """LayerNorm in the paper's two-function form: sqrt table on v + eps, 1/x table on its result."""
    import oracle as orc
    rng = np.random.default_rng(rows * 3 + H)
    z = nm_inputs.round_to((rng.standard_normal((rows, H)) * rng.uniform(0.6, 1.8, (rows, 1)) + 0.3).astype(np.float32), dtype)
    g = (1 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    b = (0.1 * rng.standard_normal(H)).astype(np.float32)
    r_sqrt, r_recip = (0.0625, 9.0), (0.2, 3.2)
    tabs = {}
    for slot, func, (lo, hi) in ((nm.SLOT_USER0, nm.FUNC_SQRT, r_sqrt), (nm.SLOT_USER0 + 1, nm.FUNC_RECIP, r_recip)):
        k, bb = ctx.load_function_table(slot, func, n, lo, hi)
        t = orc.Table.secant(func, n, lo, hi)
        assert np.array_equal(np.asarray(k, np.float32), t.k) and np.array_equal(np.asarray(bb, np.float32), t.b)
        tabs[func] = t
    td = nm_inputs.torch_dtype(dtype)
    zd = torch.from_numpy(z).cuda().to(td)
    yd = torch.empty_like(zd)
    ctx.layernorm_pwl_sqrt_recip(zd, torch.from_numpy(g).cuda(), torch.from_numpy(b).cuda(), yd, nm.SLOT_USER0,
                                 nm.SLOT_USER0 + 1, eps=1e-5)
    ref = orc.layernorm_sqrt_recip(z, g, b, 1e-5, tabs[nm.FUNC_SQRT], tabs[nm.FUNC_RECIP])
    if dtype == "f32":
        assert_close_f32(to_np(yd), ref, "layernorm sqrt+recip f32")
    else:
        assert_close_bf16(to_np(yd), ref, "layernorm sqrt+recip " + dtype)
    # an empty slot is an error, not a silent fallback
    with pytest.raises(nm.NmError) as ei:
        ctx.layernorm_pwl_sqrt_recip(zd, torch.from_numpy(g).cuda(), torch.from_numpy(b).cuda(), yd, nm.SLOT_USER0,
                                     13, eps=1e-5)   # slot 13 is never loaded in this module
    assert ei.value.code == 4


def test_layernorm_rejects_bad_shapes(nm, ctx):
    load_tables_both(ctx, 64, {"rsqrt": RANGES["rsqrt"]})
    z = torch.zeros(4, 12, device="cuda")
    g = torch.ones(12, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.layernorm_pwl(z, g, g, torch.empty_like(z))
    assert ei.value.code == 2
    z0 = torch.zeros(0, 16, device="cuda")
    g16 = torch.ones(16, device="cuda")
    ctx.layernorm_pwl(z0, g16, g16, torch.empty_like(z0))    # zero rows: no-op


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_quantize_bit_exact(nm, ctx, dtype):
    x = nm_inputs.round_to(nm_inputs.matrix(70001, 11, "f32", 1.0), dtype)
    x[:8] = [0.5, 1.5, 2.5, -0.5, -1.5, 1e6, -1e6, 0.0]
    x = nm_inputs.round_to(x, dtype)
    scale = np.float32(0.03)
    inv = float(np.float32(1.0) / scale)
    xd = torch.from_numpy(x).cuda().to(nm_inputs.torch_dtype(dtype))
    q = torch.empty(x.size, dtype=torch.int8, device="cuda")
    ctx.quantize_i8(xd, inv, q)
    assert np.array_equal(q.cpu().numpy(), oracle.quantize_i8(x, scale))


@pytest.mark.parametrize("func,lo,hi,dLx,dK", [("gelu", -4.0, 4.0, 0.125, 0.02), ("exp", -8.0, 0.0, 0.125, 0.01),
                                               ("recip", 1.0, 33.0, 0.25, 0.002)])
def test_elastic_tables_evaluate_bit_exact(nm, ctx, func, lo, hi, dLx, dK):
    """Tables with Algorithm 2's merged segments and Algorithm 3's bias correction (not continuous any
    more: the fp32 index contract decides which side of a jump an input lands on) evaluate bit for bit."""
    from util import FUNCS, oracle_elastic_table
    n, k, b, nseg = nm.pwl_table_build_elastic(FUNCS[func], lo, hi, dLx, dK, bias_correct=True)
    t, _ = oracle_elastic_table(FUNCS[func], lo, hi, dLx, dK, bias_correct=True)
    assert nseg < n
    ctx.pwl_table_load(nm.SLOT_USER0, n, lo, hi, k, b)
    x = nm_inputs.pwl_probe_points(lo, hi, n, 50021, seed=7)
    x = x[np.isfinite(x)]
    xd = torch.from_numpy(x).cuda()
    yd = torch.empty_like(xd)
    idx = torch.empty(x.size, dtype=torch.int32, device="cuda")
    ctx.pwl_apply(nm.SLOT_USER0, xd, yd, idx)
    y_ref, idx_ref = oracle.pwl_eval_f32(t, x)
    assert np.array_equal(idx.cpu().numpy(), idx_ref)
    assert np.array_equal(yd.cpu().numpy().view(np.uint32), y_ref.view(np.uint32))
    # and the elastic table approximates the function at least as well (in mean square) as its secants
    xx = np.linspace(lo, hi, 20001)[1:-1]
    exact = oracle.exact(FUNCS[func], xx)
    t0, _ = oracle_elastic_table(FUNCS[func], lo, hi, dLx, dK, bias_correct=False)
    assert ((t(xx) - exact) ** 2).mean() < ((t0(xx) - exact) ** 2).mean()


def test_bounded_wait_times_out_and_context_survives(nm, ctx):
    """Failure detection without a GPU fault: a wait that can never be satisfied gives up after its
    limit, the kernel returns normally, the status word carries NM_ERR_TIMEOUT, and the context keeps
    working."""
    assert ctx.poll_status() == 0
    ctx.selftest_bounded_wait(100_000_000)              # ~50 ms of SM clock
    assert ctx.poll_status() == 7                       # NM_ERR_TIMEOUT, and the word is cleared by the poll
    assert ctx.poll_status() == 0
    load_tables_both(ctx, 64, {"gelu": RANGES["gelu"]})
    x = torch.linspace(-3, 3, 64, device="cuda")
    y = torch.empty_like(x)
    ctx.pwl_apply(nm.SLOT_GELU, x, y)                   # the context is still usable
    torch.cuda.synchronize()
    assert torch.isfinite(y).all() and ctx.poll_status() == 0
