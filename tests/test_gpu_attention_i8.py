"""GPU parity, INT8 attention: Q K^T and P V on the int8 tensor-core path.  Every integer the kernel produces
(scores, probability codes, integer P.V) and the fp32 output are compared with the oracle bit for bit; the bf16
output within the bf16 bound."""
import numpy as np
import pytest
import torch

import nm_inputs
import oracle
from util import assert_close_bf16, load_tables_both

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx(nm):
    c = nm.Context(0)
    yield c
    c.close()


def _codes(B, L, h, d, seed, qk_scale):
    """int8 codes of a seeded N(0,1) packed projection with a per-tensor scale of 4.5 sigma / 127."""
    x = nm_inputs.matrix((B * L, 3 * h * d), seed, "f32", 1.0)
    s = np.float32(4.5 / 127.0)
    c = np.clip(np.rint(x / s), -127, 127).astype(np.int8)
    return c, float(s) * qk_scale, float(s)


@pytest.mark.parametrize("B,L,h,qk", [(1, 128, 2, 0.6), (2, 256, 3, 0.6), (1, 512, 4, 0.5), (2, 128, 1, 1.2), (1, 384, 5, 0.8)])
def test_int8_attention_bit_exact(nm, ctx, B, L, h, qk):
    d = 64
    tabs = load_tables_both(ctx, 64, {"exp": (-8.0, 0.0), "recip": (L / 16.0, float(L))})
    codes, s_qk, s_v = _codes(B, L, h, d, 7 + L + h, qk)
    H = h * d
    qd = torch.from_numpy(codes).cuda()
    out = torch.full((B * L, H), float("nan"), dtype=torch.float32, device="cuda")
    acc = torch.full((B, h, L, L), -7, dtype=torch.int32, device="cuda")
    pc = torch.full((B, h, L, L), -7, dtype=torch.int8, device="cuda")
    oacc = torch.full((B * L, H), -7, dtype=torch.int32, device="cuda")
    ctx.attention_pwl_i8(qd, out, B, L, h, d, s_qk, s_qk, s_v, acc_dump=acc, p_dump=pc, oacc_dump=oacc)
    ctx.check_device_status()
    r = oracle.attention_i8(codes, B, L, h, d, s_qk, s_qk, s_v, tabs["exp"], tabs["recip"], want_dumps=True)
    assert np.array_equal(acc.cpu().numpy(), r["acc"]), "integer scores"
    assert np.array_equal(pc.cpu().numpy(), r["p"]), "probability codes"
    assert np.array_equal(oacc.cpu().numpy(), r["oacc"]), "integer P.V"
    assert np.array_equal(out.cpu().numpy().view(np.uint32), r["out"].view(np.uint32)), "fp32 output"
    # the same launch without dumps and with bf16 output
    ob = torch.full((B * L, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.attention_pwl_i8(qd, ob, B, L, h, d, s_qk, s_qk, s_v)
    ctx.check_device_status()
    assert_close_bf16(ob.float().cpu().numpy(), r["out"], "int8 attention, bf16 output")
    want = torch.from_numpy(r["out"]).bfloat16()
    assert torch.equal(ob.cpu(), want), "bf16 output = the fp32 value rounded once"


def test_int8_attention_full_size_sampled(nm, ctx):
    """The config-3 launch shape (B 32, L 512, 12 heads): three batch entries checked in full, bit for bit."""
    B, L, h, d = 32, 512, 12, 64
    tabs = load_tables_both(ctx, 64, {"exp": (-8.0, 0.0), "recip": (L / 16.0, float(L))})
    codes, s_qk, s_v = _codes(B, L, h, d, 99, 0.6)
    out = torch.full((B * L, h * d), float("nan"), dtype=torch.float32, device="cuda")
    ctx.attention_pwl_i8(torch.from_numpy(codes).cuda(), out, B, L, h, d, s_qk, s_qk, s_v)
    ctx.check_device_status()
    got = out.cpu().numpy()
    for b in (0, 17, 31):
        ref = oracle.attention_i8(codes[b * L:(b + 1) * L], 1, L, h, d, s_qk, s_qk, s_v, tabs["exp"], tabs["recip"])
        assert np.array_equal(got[b * L:(b + 1) * L].view(np.uint32), ref.view(np.uint32)), "batch %d" % b


@pytest.mark.parametrize("B,L,h", [(10, 128, 50), (4, 384, 40)])
def test_int8_attention_several_tiles_per_cta(nm, ctx, B, L, h):
    """More tiles than resident CTAs (3 per SM), lengths with an odd number of barrier phases per tile (3 and 9
    score products): the persistent CTAs carry their phase counts from tile to tile.  fp32 output bit for bit."""
    d = 64
    assert B * h * (L // 128) > 3 * torch.cuda.get_device_properties(0).multi_processor_count
    tabs = load_tables_both(ctx, 64, {"exp": (-8.0, 0.0), "recip": (L / 16.0, float(L))})
    codes, s_qk, s_v = _codes(B, L, h, d, 41 + L, 0.7)
    out = torch.full((B * L, h * d), float("nan"), dtype=torch.float32, device="cuda")
    ctx.attention_pwl_i8(torch.from_numpy(codes).cuda(), out, B, L, h, d, s_qk, s_qk, s_v)
    ctx.check_device_status()
    ref = oracle.attention_i8(codes, B, L, h, d, s_qk, s_qk, s_v, tabs["exp"], tabs["recip"])
    assert np.array_equal(out.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def test_int8_attention_argument_errors(nm, ctx):
    load_tables_both(ctx, 64, {"exp": (-8.0, 0.0), "recip": (8.0, 128.0)})
    q = torch.zeros(128, 192, dtype=torch.int8, device="cuda")
    o = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.attention_pwl_i8(q, o, 1, 128, 1, 64, 0.03, 0.03, 0.03, exp_slot=12)
    assert ei.value.code == 4
    with pytest.raises(nm.NmError) as ei:
        ctx.attention_pwl_i8(q, o, 1, 128, 1, 64, 0.03, 0.0, 0.03)
    assert ei.value.code == 1
    q2 = torch.zeros(96, 192, dtype=torch.int8, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.attention_pwl_i8(q2, o, 1, 96, 1, 64, 0.03, 0.03, 0.03)     # L not a multiple of 128
    assert ei.value.code == 5
    ctx.attention_pwl_i8(q, o, 0, 128, 1, 64, 0.03, 0.03, 0.03)       # empty batch: no-op
