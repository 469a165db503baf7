"""Shared checks for the GPU parity tests."""
import numpy as np
import torch

# bf16 / fp16 paths: |gpu - oracle| <= 1e-2 + 1e-2*|oracle| per element
BF16_ATOL, BF16_RTOL = 1e-2, 1e-2
# ... and, because the absolute term is a large share of a small output (attention outputs have an rms of
# 0.03-0.09 at L = 512), a ceiling on rms(gpu - oracle) / rms(oracle): storing a result in bf16 alone costs
# 2^-9 / sqrt(3) = 1.1e-3, a bf16 probability tile about as much again; a few-percent error in one PWL
# factor (the reciprocal of the row sum, the rsqrt of the variance) would show here at its full size.
BF16_RMS_REL = 1e-2
# fp32 path: |gpu - oracle| <= 1e-4 * max(|oracle|, rms(oracle))
F32_RTOL = 1e-4


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy() if t.dtype != torch.int8 and t.dtype != torch.int32 \
        else t.detach().to("cpu").numpy()


def rms_rel(gpu, ref):
    """rms(gpu - ref) / rms(ref)."""
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.sqrt(np.mean(ref * ref))
    return float(np.sqrt(np.mean((gpu - ref) ** 2)) / den) if den > 0 else 0.0


def assert_close_bf16(gpu, ref, what="", rms_rel_max=BF16_RMS_REL):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    assert gpu.shape == ref.shape, (gpu.shape, ref.shape)
    assert np.all(np.isfinite(gpu)), what + ": non-finite GPU output"
    err = np.abs(gpu - ref)
    bound = BF16_ATOL + BF16_RTOL * np.abs(ref)
    bad = err > bound
    rr = rms_rel(gpu, ref)
    print("%s: max err %.3e, rms(err)/rms(ref) %.3e" % (what, err.max() if err.size else 0.0, rr))
    assert not bad.any(), "%s: %d / %d elements outside 1e-2 + 1e-2*|ref| (max err %.3e at ref %.3e)" % (
        what, bad.sum(), bad.size, err.max(), ref.ravel()[err.argmax()])
    assert rr <= rms_rel_max, "%s: rms(err)/rms(ref) = %.3e above the ceiling %.1e" % (what, rr, rms_rel_max)


def assert_close_f32(gpu, ref, what="", rtol=F32_RTOL):
    gpu = np.asarray(gpu, np.float64)
    ref = np.asarray(ref, np.float64)
    assert gpu.shape == ref.shape
    assert np.all(np.isfinite(gpu)), what + ": non-finite GPU output"
    rms = np.sqrt(np.mean(ref * ref))
    bound = rtol * np.maximum(np.abs(ref), rms)
    err = np.abs(gpu - ref)
    bad = err > bound
    assert not bad.any(), "%s: %d / %d elements outside %.0e*max(|ref|, rms) (max err %.3e, rms %.3e)" % (
        what, bad.sum(), bad.size, rtol, err.max(), rms)


FUNCS = {"gelu": 0, "exp": 1, "recip": 2, "rsqrt": 3, "relu": 4, "sqrt": 5, "identity": 6}
SLOTS = {"gelu": 0, "exp": 1, "recip": 2, "rsqrt": 3, "relu": 4}


def load_tables_both(ctx, n, ranges):
    """Builds each table twice -- by the library's builder and by the oracle's -- checks they
    agree bit for bit, loads the library's into the context and returns the oracle's."""
    import oracle
    out = {}
    for name, (lo, hi) in ranges.items():
        k, b = ctx.load_function_table(SLOTS[name], FUNCS[name], n, lo, hi)
        t = oracle.Table.secant(FUNCS[name], n, lo, hi)
        assert np.array_equal(np.asarray(k, np.float32), t.k), name
        assert np.array_equal(np.asarray(b, np.float32), t.b), name
        out[name] = t
    return out


def oracle_elastic_table(func, r_min, r_max, dLx, dK_th, bias_correct=True, e_th=0.0):
    """The elastic table (Algorithm 2 start points, Algorithm 3 parameters) built from the oracle's own
    routines and laid on the primary grid: returns (oracle.Table on n_cells equal cells, n_segments)."""
    import oracle
    starts = oracle.hsize_startpoints(func, dLx, dK_th, r_min, r_max)
    xs = np.concatenate([starts, [r_max]])
    k, b = oracle.secant_points(func, xs)
    if bias_correct:
        b, _ = oracle.bias_correct(func, xs, b, e_th)
    n_cells = int(round((r_max - r_min) / dLx))
    cell_x = r_min + dLx * np.arange(n_cells)
    seg = np.searchsorted(starts, cell_x + 1e-9 * dLx, side="right") - 1
    return oracle.Table(n_cells, r_min, r_max, k[seg].astype(np.float32), b[seg].astype(np.float32)), len(starts)
