"""GPU parity, linear operator with PWL epilogue: CUDA-core fp32 path, tcgen05 bf16 / fp16 /
int8 paths, ragged edges, full-size sampled rows."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import assert_close_bf16, assert_close_f32, load_tables_both, to_np

pytestmark = pytest.mark.gpu

RANGES = {"gelu": (-4.0, 4.0), "relu": (-3.0, 3.0)}


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def run_float(nm, ctx, dtype, M, N, K, bias, residual, slot_name, algo, seed=0, w_scale=0.05):
    tabs = load_tables_both(ctx, 64, RANGES)
    A = nm_inputs.matrix((M, K), seed, dtype, 1.0)
    W = nm_inputs.matrix((N, K), seed + 1, dtype, w_scale)
    rng = np.random.default_rng(seed + 2)
    bv = (0.1 * rng.standard_normal(N)).astype(np.float32) if bias else None
    rv = nm_inputs.round_to(rng.standard_normal((M, N)).astype(np.float32), dtype) if residual else None
    td = nm_inputs.torch_dtype(dtype)
    Ad, Wd = torch.from_numpy(A).cuda().to(td), torch.from_numpy(W).cuda().to(td)
    out = torch.full((M, N), float("nan"), dtype=td, device="cuda")
    slot = {"gelu": nm.SLOT_GELU, "relu": nm.SLOT_RELU, None: nm.SLOT_NONE}[slot_name]
    ctx.linear_pwl(Ad, Wd, out, bias=torch.from_numpy(bv).cuda() if bias else None,
                   residual=torch.from_numpy(rv).cuda().to(td) if residual else None, slot=slot, algo=algo)
    ctx.check_device_status()
    ref = oracle.linear(A, W, bv, rv, tabs[slot_name] if slot_name else None)
    return to_np(out), ref


@pytest.mark.parametrize("M,N,K", [(128, 768, 256), (128, 1024, 256), (128, 256, 1024), (37, 29, 53), (1, 8, 8)])
@pytest.mark.parametrize("epi", ["plain", "gelu_bias", "bias_res"])
def test_linear_f32_simt(nm, ctx, M, N, K, epi):
    Kp = (K + 3) // 4 * 4
    Np = (N + 3) // 4 * 4
    got, ref = run_float(nm, ctx, "f32", M, Np, Kp, epi != "plain", epi == "bias_res",
                         "gelu" if epi == "gelu_bias" else None, nm.ALGO_AUTO)
    assert_close_f32(got, ref, "linear f32 %s" % epi)


@pytest.mark.parametrize("algo", ["tc", "tc_1cta"])
@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (256, 256, 128), (384, 768, 768), (128, 128, 256),
                                   (200, 328, 72), (130, 136, 1032), (1024, 2304, 768), (600, 520, 200)])
def test_linear_tc_plain(nm, ctx, algo, dtype, M, N, K):
    """Several tiles, ragged rows / columns / K, both tile widths; "tc" uses CTA pairs
    (cta_group::2, 256-row tiles) once M and N reach 256, "tc_1cta" forces one CTA per tile."""
    a = nm.ALGO_TC if algo == "tc" else nm.ALGO_TC_1CTA
    got, ref = run_float(nm, ctx, dtype, M, N, K, False, False, None, a)
    assert_close_bf16(got, ref, "linear %s %s %dx%dx%d" % (algo, dtype, M, N, K))


@pytest.mark.parametrize("algo", ["tc", "tc_1cta"])
@pytest.mark.parametrize("epi", ["gelu_bias", "bias_res", "relu_bias_res"])
@pytest.mark.parametrize("M,N,K", [(256, 512, 192), (200, 328, 72), (512, 3072, 768), (700, 776, 136)])
def test_linear_tc_epilogues(nm, ctx, algo, epi, M, N, K):
    slot = "gelu" if epi == "gelu_bias" else ("relu" if epi == "relu_bias_res" else None)
    a = nm.ALGO_TC if algo == "tc" else nm.ALGO_TC_1CTA
    got, ref = run_float(nm, ctx, "bf16", M, N, K, True, "res" in epi, slot, a, seed=5)
    assert_close_bf16(got, ref, "linear tc %s" % epi)


def test_linear_tc_matches_simt_path_choice(nm, ctx):
    """algo=auto must pick a kernel and give the same answer within tolerance as either forced one."""
    for algo in (nm.ALGO_AUTO, nm.ALGO_SIMT, nm.ALGO_TC):
        got, ref = run_float(nm, ctx, "bf16", 256, 256, 256, True, True, "gelu", algo, seed=9)
        assert_close_bf16(got, ref, "algo %d" % algo)


@pytest.mark.parametrize("algo", ["simt", "tc", "tc_1cta"])
@pytest.mark.parametrize("M,N,K,out", [(256, 256, 256, "bf16"), (200, 328, 144, "bf16"), (384, 1024, 1024, "i8"),
                                       (128, 512, 4096, "f32"), (512, 512, 512, "f32")])
def test_linear_int8_bit_exact(nm, ctx, algo, M, N, K, out):
    """int32 accumulators and segment numbers must match the oracle bit for bit; so must the
    fp32 epilogue value and the requantised int8 output."""
    tabs = load_tables_both(ctx, 64, RANGES)
    Aq = nm_inputs.int8_matrix((M, K), 21)
    Wq = nm_inputs.int8_matrix((N, K), 22)
    rng = np.random.default_rng(23)
    a_scale = np.float32(4.0 / 127)
    ws = (rng.uniform(0.5, 1.5, N) * 0.08 / 127).astype(np.float32)
    bias = (0.1 * rng.standard_normal(N)).astype(np.float32)
    out_scale = np.float32(0.02)
    inv = float(np.float32(1.0) / out_scale)
    td = {"bf16": torch.bfloat16, "i8": torch.int8, "f32": torch.float32}[out]
    Ad, Wd = torch.from_numpy(Aq).cuda(), torch.from_numpy(Wq).cuda()
    o = torch.zeros((M, N), dtype=td, device="cuda")
    acc = torch.full((M, N), -1, dtype=torch.int32, device="cuda")
    idx = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    ctx.linear_pwl(Ad, Wd, o, bias=torch.from_numpy(bias).cuda(), slot=nm.SLOT_GELU, a_scale=float(a_scale),
                   w_scale=torch.from_numpy(ws).cuda(), inv_out_scale=inv, acc_dump=acc, idx_dump=idx,
                   algo={"simt": nm.ALGO_SIMT, "tc": nm.ALGO_TC, "tc_1cta": nm.ALGO_TC_1CTA}[algo])
    ctx.check_device_status()
    r = oracle.linear_i8(Aq, Wq, a_scale, ws, bias, None, tabs["gelu"], out_scale=out_scale)
    assert np.array_equal(acc.cpu().numpy(), r["acc"])
    assert np.array_equal(idx.cpu().numpy(), r["idx"])
    if out == "i8":
        assert np.array_equal(o.cpu().numpy(), r["q"])
    elif out == "f32":
        assert np.array_equal(o.cpu().numpy().view(np.uint32), r["y"].view(np.uint32))
    else:
        assert torch.equal(o.cpu(), torch.from_numpy(r["y"]).to(torch.bfloat16))


def test_linear_full_size_sampled_rows(nm, ctx):
    """FFN1 of the 12-layer BERT-base workload (16384 x 3072 x 768, GELU table): the launch is the
    one the benchmark times; 48 sampled rows are checked against the oracle."""
    tabs = load_tables_both(ctx, 64, RANGES)
    M, N, K = 16384, 3072, 768
    A = nm_inputs.matrix((M, K), 31, "bf16", 1.0)
    W = nm_inputs.matrix((N, K), 32, "bf16", 0.02)
    bias = (0.02 * np.random.default_rng(33).standard_normal(N)).astype(np.float32)
    Ad, Wd = torch.from_numpy(A).cuda().bfloat16(), torch.from_numpy(W).cuda().bfloat16()
    out = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ctx.linear_pwl(Ad, Wd, out, bias=torch.from_numpy(bias).cuda(), slot=nm.SLOT_GELU)
    ctx.check_device_status()
    rows = np.unique(np.concatenate([[0, 127, 128, M - 1], np.random.default_rng(34).integers(0, M, 44)]))
    ref = oracle.linear(A[rows], W, bias, None, tabs["gelu"])
    assert_close_bf16(to_np(out[torch.from_numpy(rows).cuda()]), ref, "FFN1 full size")


def test_linear_argument_errors(nm, ctx):
    A = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.linear_pwl(A, A, o, slot=11)                       # table never loaded
    assert ei.value.code == 4
    with pytest.raises(nm.NmError) as ei:
        ctx.linear_pwl(A, A, torch.zeros(64, 64, device="cuda"))   # bf16 in, fp32 out
    assert ei.value.code == 5
    with pytest.raises(nm.NmError) as ei:
        ctx.linear_pwl(A[:, 1:], A[:, 1:], o)                  # misaligned operand
    assert ei.value.code == 3
    e = torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda")
    ctx.linear_pwl(e, A, torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda"))   # empty: no-op
