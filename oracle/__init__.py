"""CPU oracle of the NeuralMatrix PWL forward pass -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` /
``--impl reference`` legs of ``bench.py`` may import this package.  It shares
nothing with the CUDA library: the arithmetic lives in ``nm_oracle.c`` (plain
fp64 loops written from the paper), this module only compiles that file with
gcc and marshals numpy arrays into it.

Every wrapper takes and returns numpy arrays; floating inputs are promoted to
fp64 exactly (a bf16 / fp16 / int8 value is representable in fp64), so the
oracle sees precisely the numbers the GPU sees.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nm_oracle.c")
_SO = os.path.join(_HERE, "libnm_oracle.so")
_lock = threading.Lock()
_lib = None

GELU, EXP, RECIP, RSQRT, RELU, SQRT, IDENTITY = range(7)
FUNC_NAMES = {GELU: "gelu", EXP: "exp", RECIP: "recip", RSQRT: "rsqrt", RELU: "relu", SQRT: "sqrt",
              IDENTITY: "identity"}


def build(force: bool = False) -> str:
    """Compile nm_oracle.c into libnm_oracle.so next to it (gcc, OpenMP, no fp contraction)."""
    with _lock:
        if (not force and os.path.exists(_SO)
                and os.path.getmtime(_SO) >= os.path.getmtime(_SRC)):
            return _SO
        tmp = _SO + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _SO)
        return _SO


class _Pwl(C.Structure):
    _fields_ = [("n", C.c_int32), ("x_min", C.c_float), ("x_max", C.c_float),
                ("k", C.POINTER(C.c_float)), ("b", C.POINTER(C.c_float)), ("exact_func", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.nmo_exact.restype = C.c_double
        _lib.nmo_exact.argtypes = [C.c_int, C.c_double]
        _lib.nmo_segment_index.restype = C.c_int32
        _lib.nmo_segment_index.argtypes = [C.POINTER(_Pwl), C.c_float]
        _lib.nmo_num_threads.restype = C.c_int
        _lib.nmo_antiderivative.restype = C.c_double
        _lib.nmo_antiderivative.argtypes = [C.c_int, C.c_double]
    return _lib


def num_threads() -> int:
    return int(lib().nmo_num_threads())


def _dp(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _fp(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _ip(a):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _bp(a):
    return a.ctypes.data_as(C.POINTER(C.c_int8))


def _f64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _f32(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float32)


class Table:
    """A PWL operator: ``n`` equal segments on ``[x_min, x_max]`` with fp32 ``k`` and ``b``.

    ``Table.exact(func)`` is the exact nonlinearity in the same slot, used only to measure the
    approximation error of a whole layer."""

    def __init__(self, n, x_min, x_max, k, b, exact_func=-1, func=None):
        self.n = int(n)
        self.x_min = float(np.float32(x_min))
        self.x_max = float(np.float32(x_max))
        self.k = _f32(k)
        self.b = _f32(b)
        self.exact_func = int(exact_func)
        self.func = func
        self._c = _Pwl(self.n, self.x_min, self.x_max, _fp(self.k), _fp(self.b), self.exact_func)

    @classmethod
    def secant(cls, func, n, x_min, x_max):
        """Section 3.2.1 + Algorithm 3 line 1: equal segments, secant lines."""
        x_min = float(np.float32(x_min))
        x_max = float(np.float32(x_max))
        k = np.zeros(n, np.float32)
        b = np.zeros(n, np.float32)
        rc = lib().nmo_table_secant(C.c_int(func), C.c_int(n), C.c_double(x_min), C.c_double(x_max),
                                    _fp(k), _fp(b))
        if rc != 0:
            raise ValueError("bad table request")
        return cls(n, x_min, x_max, k, b, func=func)

    @classmethod
    def exact(cls, func):
        z = np.zeros(1, np.float32)
        return cls(1, 0.0, 1.0, z, z.copy(), exact_func=func, func=func)

    @property
    def ref(self):
        return C.byref(self._c)

    def index(self, x):
        x = _f32(x)
        out = np.empty(x.shape, np.int32)
        f = lib().nmo_segment_index
        flat = x.ravel()
        o = out.ravel()
        for i in range(flat.size):
            o[i] = f(self.ref, C.c_float(float(flat[i])))
        return out

    def __call__(self, x):
        return pwl_eval(self, x)[0]


def exact(func, x):
    x = _f64(x)
    f = lib().nmo_exact
    return np.array([f(func, float(v)) for v in x.ravel()], np.float64).reshape(x.shape)


def secant_points(func, xs):
    """Secant k, b (fp64) on arbitrary start points ``xs[0..n]``."""
    xs = _f64(xs)
    n = xs.size - 1
    k = np.zeros(n)
    b = np.zeros(n)
    lib().nmo_table_secant_points(C.c_int(func), C.c_int(n), _dp(xs), _dp(k), _dp(b))
    return k, b


def bias_correct(func, xs, b, e_th=0.0):
    """Algorithm 3 lines 2-3 on segments ``xs``; returns (corrected b, dE per segment)."""
    xs = _f64(xs)
    b = _f64(b).copy()
    dE = np.zeros(xs.size - 1)
    lib().nmo_table_bias_correct(C.c_int(func), C.c_int(xs.size - 1), _dp(xs), C.c_double(e_th), _dp(b), _dp(dE))
    return b, dE


def hsize_startpoints(func, dLx, dK_th, r_min, r_max, max_pts=4096):
    """Algorithm 2: start-point set (first entry r_min)."""
    xs = np.zeros(max_pts)
    n = lib().nmo_hsize_startpoints(C.c_int(func), C.c_double(dLx), C.c_double(dK_th), C.c_double(r_min),
                                    C.c_double(r_max), _dp(xs), C.c_int(max_pts))
    if n < 0:
        raise ValueError("too many start points")
    return xs[:n].copy()


def pwl_eval(t: Table, x):
    """(y fp64, idx int32) with the fp32 index contract."""
    x = _f64(x)
    y = np.empty_like(x)
    idx = np.empty(x.shape, np.int32)
    lib().nmo_pwl_eval(t.ref, _dp(x), C.c_int64(x.size), _dp(y), _ip(idx))
    return y, idx


def pwl_eval_f32(t: Table, x):
    """Strict fp32 evaluation (y = fmaf(k, x, b)); returns (y fp32, idx int32)."""
    x = _f32(x)
    y = np.empty_like(x)
    idx = np.empty(x.shape, np.int32)
    lib().nmo_pwl_eval_f32(t.ref, _fp(x), C.c_int64(x.size), _fp(y), _ip(idx))
    return y, idx


def linear(A, W, bias=None, residual=None, table: Table | None = None, want_idx=False):
    """out = PWL(A @ W.T + bias) + residual; A [M,K], W [N,K]."""
    A = _f64(A)
    W = _f64(W)
    M, K = A.shape
    N = W.shape[0]
    assert W.shape[1] == K
    bias_ = _f64(bias) if bias is not None else None
    res_ = _f64(residual) if residual is not None else None
    out = np.empty((M, N))
    idx = np.empty((M, N), np.int32) if want_idx else None
    lib().nmo_linear(_dp(A), C.c_int64(K), _dp(W), C.c_int64(K),
                     _dp(bias_) if bias_ is not None else None,
                     _dp(res_) if res_ is not None else None, C.c_int64(N),
                     C.c_int64(M), C.c_int64(N), C.c_int64(K),
                     table.ref if table is not None else None,
                     _dp(out), C.c_int64(N), _ip(idx) if want_idx else None)
    return (out, idx) if want_idx else out


def attention(qkv, B, L, h, d, t_exp: Table, t_recip: Table, scale=None):
    """qkv is the packed [B*L, 3*h*d] projection (Q | K | V); returns [B*L, h*d]."""
    qkv = _f64(qkv)
    H = h * d
    assert qkv.shape == (B * L, 3 * H)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty((B * L, H))
    base = qkv.ctypes.data
    q = C.cast(base, C.POINTER(C.c_double))
    k = C.cast(base + 8 * H, C.POINTER(C.c_double))
    v = C.cast(base + 16 * H, C.POINTER(C.c_double))
    lib().nmo_attention(q, k, v, C.c_int64(L * 3 * H), C.c_int64(3 * H), C.c_int32(B), C.c_int32(L),
                        C.c_int32(h), C.c_int32(d), C.c_double(scale), t_exp.ref, t_recip.ref, _dp(out))
    return out


def layernorm(z, gamma, beta, eps, t_rsqrt: Table):
    z = _f64(z)
    rows, H = z.shape
    g = _f64(gamma)
    be = _f64(beta)
    y = np.empty_like(z)
    lib().nmo_layernorm(_dp(z), _dp(g), _dp(be), C.c_int64(rows), C.c_int32(H), C.c_double(eps),
                        t_rsqrt.ref, _dp(y))
    return y


def layernorm_sqrt_recip(z, gamma, beta, eps, t_sqrt: Table, t_recip: Table):
    """LayerNorm with r = PWLrecip(PWLsqrt(v + eps)): Section 3.2.2's sqrt(x) and 1/x tables."""
    z = _f64(z)
    rows, H = z.shape
    g = _f64(gamma)
    be = _f64(beta)
    y = np.empty_like(z)
    lib().nmo_layernorm_sqrt_recip(_dp(z), _dp(g), _dp(be), C.c_int64(rows), C.c_int32(H), C.c_double(eps),
                                   t_sqrt.ref, t_recip.ref, _dp(y))
    return y


WEIGHT_NAMES = ("Wqkv", "bqkv", "Wo", "bo", "g1", "be1", "W1", "b1", "W2", "b2", "g2", "be2")


def encoder_layer(x, w: dict, B, L, h, tables: dict, eps=1e-5):
    """One post-LN encoder layer; ``w`` maps WEIGHT_NAMES to arrays; ``tables`` maps
    'gelu','exp','recip','rsqrt' to Table objects. x is [B*L, H]."""
    x = _f64(x)
    T, H = x.shape
    assert T == B * L
    ww = {n: _f64(w[n]) for n in WEIGHT_NAMES}
    F = ww["W1"].shape[0]
    y = np.empty_like(x)
    rc = lib().nmo_encoder_layer(
        _dp(x), C.c_int32(B), C.c_int32(L), C.c_int32(H), C.c_int32(h), C.c_int32(F),
        _dp(ww["Wqkv"]), _dp(ww["bqkv"]), _dp(ww["Wo"]), _dp(ww["bo"]), _dp(ww["g1"]), _dp(ww["be1"]),
        _dp(ww["W1"]), _dp(ww["b1"]), _dp(ww["W2"]), _dp(ww["b2"]), _dp(ww["g2"]), _dp(ww["be2"]),
        C.c_double(eps), tables["gelu"].ref, tables["exp"].ref, tables["recip"].ref, tables["rsqrt"].ref,
        _dp(y))
    if rc != 0:
        raise MemoryError("oracle encoder layer: allocation failed")
    return y


def encoder_stack(x, layers: list, B, L, h, tables: dict, eps=1e-5):
    """Layers applied in order; the output of one is the input of the next."""
    y = _f64(x)
    for w in layers:
        y = encoder_layer(y, w, B, L, h, tables, eps)
    return y


def linear_i8(Aq, Wq, a_scale, w_scale, bias=None, residual=None, table: Table | None = None,
              out_scale=None):
    """INT8 linear with the strict fp32 epilogue. Returns dict(acc, idx, y, q)."""
    Aq = np.ascontiguousarray(Aq, dtype=np.int8)
    Wq = np.ascontiguousarray(Wq, dtype=np.int8)
    M, K = Aq.shape
    N = Wq.shape[0]
    ws = _f32(w_scale)
    bias_ = _f32(bias) if bias is not None else None
    res_ = _f32(residual) if residual is not None else None
    acc = np.empty((M, N), np.int32)
    idx = np.empty((M, N), np.int32)
    y = np.empty((M, N), np.float32)
    q = np.empty((M, N), np.int8) if out_scale is not None else None
    inv = np.float32(1.0) / np.float32(out_scale) if out_scale is not None else np.float32(0)
    lib().nmo_linear_i8(_bp(Aq), _bp(Wq), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                        C.c_float(float(np.float32(a_scale))), _fp(ws),
                        _fp(bias_) if bias_ is not None else None,
                        _fp(res_) if res_ is not None else None,
                        table.ref if table is not None else None, C.c_float(float(inv)),
                        _ip(acc), _ip(idx), _fp(y), _bp(q) if q is not None else None)
    return {"acc": acc, "idx": idx, "y": y, "q": q}


def attention_i8(qkv_q, B, L, h, d, s_q, s_k, s_v, t_exp: Table, t_recip: Table, scale=None, want_dumps=False):
    """INT8 attention (both matrix products on integers, strict fp32 in between; see nm_oracle.c).
    qkv_q: packed int8 [B*L, 3*h*d] codes (Q | K | V).  Returns out fp32 [B*L, h*d], or with want_dumps a
    dict(out, acc int32 [B,h,L,L], p int8 [B,h,L,L], oacc int32 [B*L, h*d])."""
    qkv_q = np.ascontiguousarray(qkv_q, dtype=np.int8)
    H = h * d
    assert qkv_q.shape == (B * L, 3 * H)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.empty((B * L, H), np.float32)
    acc = np.empty((B, h, L, L), np.int32) if want_dumps else None
    pc = np.empty((B, h, L, L), np.int8) if want_dumps else None
    oacc = np.empty((B * L, H), np.int32) if want_dumps else None
    base = qkv_q.ctypes.data
    q = C.cast(base, C.POINTER(C.c_int8))
    k = C.cast(base + H, C.POINTER(C.c_int8))
    v = C.cast(base + 2 * H, C.POINTER(C.c_int8))
    f32 = lambda x: C.c_float(float(np.float32(x)))
    lib().nmo_attention_i8(q, k, v, C.c_int64(L * 3 * H), C.c_int64(3 * H), C.c_int32(B), C.c_int32(L), C.c_int32(h),
                           C.c_int32(d), f32(s_q), f32(s_k), f32(s_v), f32(scale), t_exp.ref, t_recip.ref, _fp(out),
                           _ip(acc) if want_dumps else None, _bp(pc) if want_dumps else None,
                           _ip(oacc) if want_dumps else None)
    return {"out": out, "acc": acc, "p": pc, "oacc": oacc} if want_dumps else out


def quantize_i8(x, scale):
    x = _f32(x)
    q = np.empty(x.shape, np.int8)
    inv = np.float32(1.0) / np.float32(scale)
    lib().nmo_quantize_i8(_fp(x), C.c_int64(x.size), C.c_float(float(inv)), _bp(q))
    return q


def conv2d_nhwc(x, W, stride, pad, bias=None, residual=None, table: Table | None = None):
    """x [N,H,W,Cin], W [Cout,kh,kw,Cin] -> [N,Ho,Wo,Cout]."""
    x = _f64(x)
    W = _f64(W)
    Nb, Hin, Win, Cin = x.shape
    Cout, kh, kw, _ = W.shape
    Ho = (Hin + 2 * pad - kh) // stride + 1
    Wo = (Win + 2 * pad - kw) // stride + 1
    out = np.empty((Nb, Ho, Wo, Cout))
    bias_ = _f64(bias) if bias is not None else None
    res_ = _f64(residual) if residual is not None else None
    lib().nmo_conv2d_nhwc(_dp(x), C.c_int32(Nb), C.c_int32(Hin), C.c_int32(Win), C.c_int32(Cin), _dp(W),
                          C.c_int32(Cout), C.c_int32(kh), C.c_int32(kw), C.c_int32(stride), C.c_int32(pad),
                          _dp(bias_) if bias_ is not None else None,
                          _dp(res_) if res_ is not None else None,
                          table.ref if table is not None else None, _dp(out))
    return out


def maxpool_nhwc(x, ksz, stride, pad):
    x = _f64(x)
    Nb, Hin, Win, Cc = x.shape
    Ho = (Hin + 2 * pad - ksz) // stride + 1
    Wo = (Win + 2 * pad - ksz) // stride + 1
    out = np.empty((Nb, Ho, Wo, Cc))
    lib().nmo_maxpool_nhwc(_dp(x), C.c_int32(Nb), C.c_int32(Hin), C.c_int32(Win), C.c_int32(Cc),
                           C.c_int32(ksz), C.c_int32(stride), C.c_int32(pad), _dp(out))
    return out


def maxpool_nhwc_relu(x, ksz, stride, pad, t_relu: Table):
    """Max pooling with the maximum itself written as the paper's operator form (Section 3: a network of
    linear operators and PWL nonlinearities): max(a, b) = b + PWLrelu(a - b), folded over the window in
    raster order; the first cell inside the image starts the fold, padding cells are skipped."""
    x = _f64(x)
    Nb, Hin, Win, Cc = x.shape
    Ho = (Hin + 2 * pad - ksz) // stride + 1
    Wo = (Win + 2 * pad - ksz) // stride + 1
    out = np.empty((Nb, Ho, Wo, Cc))
    for oy in range(Ho):
        for ox in range(Wo):
            m = None
            for ky in range(ksz):
                for kx in range(ksz):
                    iy, ix = oy * stride - pad + ky, ox * stride - pad + kx
                    if iy < 0 or iy >= Hin or ix < 0 or ix >= Win:
                        continue
                    v = x[:, iy, ix, :]
                    m = v.copy() if m is None else m + pwl_eval(t_relu, v - m)[0]
            out[:, oy, ox, :] = m
    return out


def avgpool_nhwc(x):
    x = _f64(x)
    Nb, Hin, Win, Cc = x.shape
    out = np.empty((Nb, Cc))
    lib().nmo_avgpool_nhwc(_dp(x), C.c_int32(Nb), C.c_int32(Hin), C.c_int32(Win), C.c_int32(Cc), _dp(out))
    return out


def antiderivative(func, x):
    """The closed-form integral F (F' = f) that Algorithm 3's segment mean is taken from."""
    x = _f64(x)
    f = lib().nmo_antiderivative
    return np.array([f(func, float(v)) for v in x.ravel()], np.float64).reshape(x.shape)


def fake_quant(x, scale, want_codes=False):
    """Definition-level int8 quantisation in fp64: scale * clamp(rint(x / scale), -127, 127)."""
    x = _f64(x)
    y = np.empty_like(x)
    codes = np.empty(x.shape, np.int8) if want_codes else None
    lib().nmo_fake_quant(_dp(x), C.c_int64(x.size), C.c_double(float(scale)), _dp(y),
                         _bp(codes) if want_codes else None)
    return (y, codes) if want_codes else y


def _deq_weight(q, name):
    return q[name + "_q"].astype(np.float64) * q[name + "_s"].astype(np.float64)[:, None]


def encoder_layer_i8(x, w: dict, q: dict, B, L, h, tables: dict, eps=1e-5, want_stages=False):
    """The int8 evaluation of one encoder layer at DEFINITION level (Section 5 evaluates INT8 networks;
    the paper fixes no scheme, the reading taken is: weights per output channel, activations per tensor,
    symmetric).  The tensor entering each of the four weight GEMMs is replaced by the value its int8 code
    stands for, fq(t) = s * clamp(rint(t / s), -127, 127); everything else is the fp64 layer above.
    Nothing is rounded to a storage type anywhere:
        qkv = fq(x) Wqkv^T + b;  a = attention(qkv);  x1 = LN(x + fq(a) Wo^T + bo)
        g = PWLgelu(fq(x1) W1^T + b1);  y = LN(x1 + fq(g) W2^T + b2)
    W* are the dequantised int8 weights (code * per-channel scale).  With want_stages the intermediate
    tensors are returned as well (dict)."""
    x = _f64(x)
    H = x.shape[1]
    d = H // h
    qkv = linear(fake_quant(x, q["a_x"]), _deq_weight(q, "Wqkv"), w["bqkv"])
    a = attention(qkv, B, L, h, d, tables["exp"], tables["recip"])
    z = linear(fake_quant(a, q["a_attn"]), _deq_weight(q, "Wo"), w["bo"], residual=x)
    x1 = layernorm(z, w["g1"], w["be1"], eps, tables["rsqrt"])
    g = linear(fake_quant(x1, q["a_x1"]), _deq_weight(q, "W1"), w["b1"], table=tables["gelu"])
    z2 = linear(fake_quant(g, q["a_g"]), _deq_weight(q, "W2"), w["b2"], residual=x1)
    y = layernorm(z2, w["g2"], w["be2"], eps, tables["rsqrt"])
    if want_stages:
        return y, {"qkv": qkv, "a": a, "z": z, "x1": x1, "g": g, "z2": z2}
    return y


def encoder_layer_i8_storage(x, w: dict, q: dict, B, L, h, tables: dict, eps=1e-5):
    """A STORAGE MODEL of the int8 layer, not the definition (that is encoder_layer_i8): the same
    composition with every tensor a bf16 workload keeps in memory rounded to bf16 before it is quantised
    or reused, and the GELU output requantised from its fp32 value.  The paper fixes none of these
    rounding points; they describe a workload that stores activations in bf16, and this function exists
    to tell how much of a GPU-vs-definition difference is storage rounding.  The four weight
    GEMMs take int8 activations (static per-tensor scales q['a_*']) and int8 weights (per-channel scales
    q['W*_s']); everything between them is the fp64 path above.  Composition of the routines in this
    file, in the order of nmo_encoder_layer:
        qkv = deq(Q(x)) Wqkv^T + b;  a = attention(qkv);  x1 = LN(x + deq(Q(a)) Wo^T + bo)
        g = PWLgelu(deq(Q(x1)) W1^T + b1);  y = LN(x1 + deq(Q(g)) W2^T + b2)
    with Q(t) = clamp(rint(t / scale), -127, 127) and deq(c) = c * scale."""
    x = _f64(x)

    # A quantised code is an integer decided by a floating-point value; it is taken in the
    # precision the workload stores that value in: activations between operators are bf16
    # (round to nearest even), the GELU output is requantised from its fp32 epilogue value.
    def bf16(t):
        u = np.ascontiguousarray(t, dtype=np.float32).view(np.uint32)
        r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000))
        return r.view(np.float32).astype(np.float64)

    def deq_act(t, scale):
        return quantize_i8(np.asarray(t, np.float32), scale).astype(np.float64) * float(np.float32(scale))

    def deq_w(name):
        return q[name + "_q"].astype(np.float64) * q[name + "_s"].astype(np.float64)[:, None]

    H = x.shape[1]
    d = H // h
    qkv = bf16(linear(deq_act(x, q["a_x"]), deq_w("Wqkv"), w["bqkv"]))
    a = bf16(attention(qkv, B, L, h, d, tables["exp"], tables["recip"]))
    z = bf16(linear(deq_act(a, q["a_attn"]), deq_w("Wo"), w["bo"], residual=x))
    x1 = bf16(layernorm(z, w["g1"], w["be1"], eps, tables["rsqrt"]))
    g = linear(deq_act(x1, q["a_x1"]), deq_w("W1"), w["b1"], table=tables["gelu"])
    z2 = bf16(linear(deq_act(g, q["a_g"]), deq_w("W2"), w["b2"], residual=x1))
    return layernorm(z2, w["g2"], w["be2"], eps, tables["rsqrt"])
