"""GPU parity, elastic tables (Algorithm 2's merged segments, Algorithm 3's bias-corrected intercepts) INSIDE
the fused kernels: the softmax reciprocal of nm_attention_pwl on [1, L] with peaked rows, where a uniform
1/x table of the same parameter count is unusable (Section 3.2.3 on rapidly changing functions), and a
bias-corrected GELU table in the epilogue of nm_linear_pwl, where the table is no longer continuous and the
fp32 index contract decides on which side of a jump an accumulator lands."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import FUNCS, assert_close_bf16, oracle_elastic_table, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def _load_elastic(nm, ctx, slot, func, lo, hi, dLx, dK):
    """The library's elastic table into `slot`; returns the oracle's own construction of the same table."""
    n, k, b, nseg = nm.pwl_table_build_elastic(FUNCS[func], lo, hi, dLx, dK, bias_correct=True)
    t, nseg_ref = oracle_elastic_table(FUNCS[func], lo, hi, dLx, dK, bias_correct=True)
    assert n == t.n and nseg == nseg_ref
    assert np.array_equal(np.asarray(k, np.float32), t.k) and np.array_equal(np.asarray(b, np.float32), t.b)
    ctx.pwl_table_load(slot, n, lo, hi, k, b)
    return t, nseg


@pytest.mark.parametrize("algo", ["simt", "tc"])
@pytest.mark.parametrize("L", [128, 512])
def test_attention_with_elastic_reciprocal_on_peaked_rows(nm, ctx, algo, L):
    """Queries and keys scaled up so that rows are dominated by a few keys (row sums of a few units, below
    L/16): the reciprocal table must cover [1, L]."""
    B, h, d = 2, 3, 64
    H = h * d
    lo = 1.0
    dLx = 0.5 if L == 128 else 2.0                    # at most 256 primary cells
    hi = lo + dLx * round((L - lo) / dLx + 0.49)      # a whole number of primary cells covering [1, L]
    t_rcp, nseg = _load_elastic(nm, ctx, nm.SLOT_USER0 + 4, "recip", lo, hi, dLx, 2e-4 if L == 128 else 2e-5)
    # peaked rows reach far below the row maximum: the exp table spans [-16, 0] here
    k, b = ctx.load_function_table(nm.SLOT_EXP, nm.FUNC_EXP, 64, -16.0, 0.0)
    t_exp = oracle.Table.secant(oracle.EXP, 64, -16.0, 0.0)
    assert np.array_equal(np.asarray(k, np.float32), t_exp.k) and np.array_equal(np.asarray(b, np.float32), t_exp.b)
    qkv = nm_inputs.matrix((B * L, 3 * H), 100 + L, "bf16", 1.0)
    qkv[:, :2 * H] *= 1.5
    qkv = nm_inputs.round_to(qkv, "bf16")
    qd = torch.from_numpy(qkv).cuda().bfloat16()
    out = torch.full((B * L, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.attention_pwl(qd, out, B, L, h, d, recip_slot=nm.SLOT_USER0 + 4, algo=nm.ALGO_SIMT if algo == "simt" else nm.ALGO_TC)
    ctx.check_device_status()
    ref = oracle.attention(qkv, B, L, h, d, t_exp, t_rcp)
    assert_close_bf16(to_np(out), ref, "attention, elastic 1/x on [1, %g], %s" % (hi, algo))
    # the rows really are peaked, and the elastic table is what makes them usable: against the exact
    # reciprocal, it beats the uniform table with as many parameters by a wide margin
    exact = oracle.attention(qkv, B, L, h, d, t_exp, oracle.Table.exact(oracle.RECIP))
    uniform = oracle.attention(qkv, B, L, h, d, t_exp, oracle.Table.secant(oracle.RECIP, nseg, lo, hi))
    e_el = np.sqrt(((ref - exact) ** 2).mean()) / np.sqrt((exact ** 2).mean())
    e_un = np.sqrt(((uniform - exact) ** 2).mean()) / np.sqrt((exact ** 2).mean())
    print("L=%d: %d kept segments on %d primary cells; rms deviation from the exact reciprocal: elastic %.3e, "
          "uniform table of %d segments %.3e" % (L, nseg, t_rcp.n, e_el, nseg, e_un))
    # (at L = 512 the 256-cell limit makes the first primary cell [1, 3], hence the looser figure)
    assert e_el < (0.01 if L == 128 else 0.1) and e_un > 5 * e_el


@pytest.mark.parametrize("algo", ["simt", "tc", "tc_1cta"])
def test_linear_int8_with_bias_corrected_gelu_is_bit_exact(nm, ctx, algo):
    """int8 GEMM whose epilogue evaluates a bias-corrected (discontinuous) GELU table: accumulators,
    segment numbers and the fp32 value bit for bit, jumps included."""
    t, nseg = _load_elastic(nm, ctx, nm.SLOT_USER0 + 5, "gelu", -4.0, 4.0, 0.125, 0.02)
    assert nseg < t.n and np.abs(np.diff(t.k * (-4.0 + 0.125 * np.arange(1, t.n + 1)) + t.b)).max() > 0   # not trivial
    M, N, K = 384, 520, 256
    Aq = nm_inputs.int8_matrix((M, K), 41)
    Wq = nm_inputs.int8_matrix((N, K), 42)
    rng = np.random.default_rng(43)
    ws = rng.uniform(3e-4, 8e-4, N).astype(np.float32)
    bias = (0.2 * rng.standard_normal(N)).astype(np.float32)
    a_scale = float(np.float32(0.031))
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    idx = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    a = {"simt": nm.ALGO_SIMT, "tc": nm.ALGO_TC, "tc_1cta": nm.ALGO_TC_1CTA}[algo]
    ctx.linear_pwl(torch.from_numpy(Aq).cuda(), torch.from_numpy(Wq).cuda(), out, bias=torch.from_numpy(bias).cuda(),
                   slot=nm.SLOT_USER0 + 5, a_scale=a_scale, w_scale=torch.from_numpy(ws).cuda(), acc_dump=acc,
                   idx_dump=idx, algo=a)
    ctx.check_device_status()
    r = oracle.linear_i8(Aq, Wq, a_scale, ws, bias, None, t)
    assert np.array_equal(acc.cpu().numpy(), r["acc"])
    assert np.array_equal(idx.cpu().numpy(), r["idx"])
    assert np.array_equal(out.cpu().numpy().view(np.uint32), r["y"].view(np.uint32))
    assert len(np.unique(r["idx"])) > t.n // 2           # the inputs spread over the table


def test_linear_bf16_with_bias_corrected_gelu(nm, ctx):
    t, _ = _load_elastic(nm, ctx, nm.SLOT_USER0 + 5, "gelu", -4.0, 4.0, 0.125, 0.02)
    M, N, K = 512, 776, 192
    A = nm_inputs.matrix((M, K), 51, "bf16", 1.0)
    W = nm_inputs.matrix((N, K), 52, "bf16", 0.08)
    bias = (0.1 * np.random.default_rng(53).standard_normal(N)).astype(np.float32)
    out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.linear_pwl(torch.from_numpy(A).cuda().bfloat16(), torch.from_numpy(W).cuda().bfloat16(), out,
                   bias=torch.from_numpy(bias).cuda(), slot=nm.SLOT_USER0 + 5, algo=nm.ALGO_TC)
    ctx.check_device_status()
    ref = oracle.linear(A, W, bias, None, t)
    assert_close_bf16(to_np(out), ref, "linear bf16, bias-corrected GELU table")
