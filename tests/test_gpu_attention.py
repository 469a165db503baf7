"""GPU parity, attention with PWL softmax (final row maximum, PWL exp, PWL reciprocal)."""
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


def ranges(L):
    return {"exp": (-8.0, 0.0), "recip": (L / 16.0, float(L))}


def run(nm, ctx, dtype, B, L, h, d, algo, seed=0, n=64, qk_scale=1.0):
    tabs = load_tables_both(ctx, n, ranges(L))
    H = h * d
    qkv = nm_inputs.matrix((B * L, 3 * H), seed, dtype, 1.0)
    qkv[:, :2 * H] *= qk_scale
    qkv = nm_inputs.round_to(qkv, dtype)
    td = nm_inputs.torch_dtype(dtype)
    qd = torch.from_numpy(qkv).cuda().to(td)
    out = torch.full((B * L, H), float("nan"), dtype=td, device="cuda")
    ctx.attention_pwl(qd, out, B, L, h, d, algo=algo)
    ctx.check_device_status()
    ref = oracle.attention(qkv, B, L, h, d, tabs["exp"], tabs["recip"])
    return to_np(out), ref


@pytest.mark.parametrize("B,L,h,d", [(1, 128, 4, 64), (2, 40, 3, 16), (1, 7, 1, 8)])
def test_attention_f32_simt(nm, ctx, B, L, h, d):
    got, ref = run(nm, ctx, "f32", B, L, h, d, nm.ALGO_AUTO)
    assert_close_f32(got, ref, "attention f32")


@pytest.mark.parametrize("algo", ["simt", "tc", "tc_resident"])
@pytest.mark.parametrize("B,L,h,d,qk", [(2, 128, 12, 64, 0.6), (1, 512, 3, 64, 0.6), (3, 128, 2, 64, 1.5), (1, 256, 2, 64, 1.0),
                                        (1, 384, 1, 64, 0.8), (1, 1024, 2, 64, 0.7)])
def test_attention_bf16(nm, ctx, algo, B, L, h, d, qk):
    """Scores of different spread: near-uniform rows (the synthetic BERT workload) and peaked ones
    that reach the clamped end segments of the exp table."""
    a = {"simt": nm.ALGO_SIMT, "tc": nm.ALGO_TC, "tc_resident": nm.ALGO_ATTN_RESIDENT}[algo]
    try:
        got, ref = run(nm, ctx, "bf16", B, L, h, d, a, seed=L + h, qk_scale=qk)
    except nm.NmError as e:
        if algo == "tc_resident" and e.code == 5 and L > 512:
            pytest.skip("the resident-score kernel takes L up to 512 only")
        raise
    assert_close_bf16(got, ref, "attention bf16 %s" % algo)


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("B,L,h", [(2, 128, 3), (1, 384, 2), (1, 640, 1)])
def test_attention_stream_lengths(nm, ctx, dtype, B, L, h):
    """The streaming kernel at lengths with an odd and an even number of 128-key chunks."""
    got, ref = run(nm, ctx, dtype, B, L, h, 64, nm.ALGO_TC, seed=17 + L, qk_scale=0.8)
    assert_close_bf16(got, ref, "attention %s, L=%d" % (dtype, L))


@pytest.mark.parametrize("B,L,h", [(10, 128, 50), (4, 384, 40), (3, 640, 31)])
def test_attention_stream_several_tiles_per_cta(nm, ctx, B, L, h):
    """More (batch, head, query block) tiles than resident CTAs (3 per SM), so that every CTA walks over
    several tiles; the lengths give an odd number of barrier phases per tile (3, 9 and 15 score products),
    which the running phase counters must carry from tile to tile."""
    assert B * h * (L // 128) > 3 * torch.cuda.get_device_properties(0).multi_processor_count
    got, ref = run(nm, ctx, "bf16", B, L, h, 64, nm.ALGO_TC, seed=5 + L, qk_scale=0.8)
    assert_close_bf16(got, ref, "attention, %d tiles, L=%d" % (B * h * (L // 128), L))


@pytest.mark.parametrize("n", [16, 256])
def test_attention_bf16_segment_counts(nm, ctx, n):
    got, ref = run(nm, ctx, "bf16", 1, 128, 2, 64, nm.ALGO_AUTO, seed=3, n=n, qk_scale=0.6)
    assert_close_bf16(got, ref, "attention n=%d" % n)


def test_attention_full_size_sampled(nm, ctx):
    """B=32, L=512, 12 heads of 64: the launch the benchmark times; three sampled batch entries
    are checked in full against the oracle."""
    B, L, h, d = 32, 512, 12, 64
    tabs = load_tables_both(ctx, 64, ranges(L))
    H = h * d
    qkv = nm_inputs.matrix((B * L, 3 * H), 77, "bf16", 0.6)
    qd = torch.from_numpy(qkv).cuda().bfloat16()
    out = torch.empty((B * L, H), dtype=torch.bfloat16, device="cuda")
    ctx.attention_pwl(qd, out, B, L, h, d)
    ctx.check_device_status()
    for b in (0, 13, 31):
        ref = oracle.attention(qkv[b * L:(b + 1) * L], 1, L, h, d, tabs["exp"], tabs["recip"])
        assert_close_bf16(to_np(out[b * L:(b + 1) * L]), ref, "attention full size, batch %d" % b)


def test_attention_argument_errors(nm, ctx):
    load_tables_both(ctx, 64, ranges(128))
    q = torch.zeros(128, 192, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(nm.NmError) as ei:
        ctx.attention_pwl(q, o, 1, 128, 1, 64, exp_slot=12)
    assert ei.value.code == 4
    for bad_scale in (0.0, -0.125, float("nan"), float("inf")):   # the row maximum is taken before scaling
        with pytest.raises(nm.NmError) as ei:
            ctx.attention_pwl(q, o, 1, 128, 1, 64, scale=bad_scale)
        assert ei.value.code == 1
    ctx.attention_pwl(q, o, 0, 128, 1, 64)     # empty batch: no-op
