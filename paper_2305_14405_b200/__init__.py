"""Python binding of the B200-native NeuralMatrix library (libnm_b200.so).

Argument marshalling only: every function here turns torch tensors into raw
device pointers and sizes and calls the C entry point of the same name; all
arithmetic runs in the CUDA kernels.  PyTorch supplies device memory and
streams, nothing else.  There is no CPU fallback: if the shared library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
SO_PATH = os.path.join(_HERE, "libnm_b200.so")
HEADER = os.path.join(os.path.dirname(_HERE), "include", "nm_b200.h")

NM_OK = 0
F32, BF16, F16, I8 = 0, 1, 2, 3
SLOT_NONE, SLOT_GELU, SLOT_EXP, SLOT_RECIP, SLOT_RSQRT, SLOT_RELU, SLOT_USER0 = -1, 0, 1, 2, 3, 4, 5
FUNC_GELU, FUNC_EXP, FUNC_RECIP, FUNC_RSQRT, FUNC_RELU, FUNC_SQRT, FUNC_IDENTITY = range(7)
ALGO_AUTO, ALGO_SIMT, ALGO_TC, ALGO_TC_1CTA = 0, 1, 2, 3
ALGO_ATTN_RESIDENT = 3   # attention only: the kernel that keeps the score block in tensor memory
STATIC_WS_BYTES = 32 << 20

EXPORTS = [
    "nm_status_string", "nm_ctx_create", "nm_ctx_destroy", "nm_ctx_poll_status", "nm_ctx_launch_count",
    "nm_pwl_table_build", "nm_pwl_table_load", "nm_pwl_apply", "nm_linear_pwl", "nm_attention_pwl",
    "nm_layernorm_pwl", "nm_layernorm_pwl_sqrt_recip", "nm_quantize_i8", "nm_encoder_workspace_bytes", "nm_encoder_layer", "nm_encoder_stack",
    "nm_encoder_stack_host", "nm_ctx_profile_enable", "nm_ctx_profile_read", "nm_encoder_layer_static",
    "nm_conv2d_workspace_bytes", "nm_conv2d_pwl", "nm_maxpool2d", "nm_maxpool2d_pwl", "nm_avgpool_global", "nm_resnet50_workspace_bytes",
    "nm_resnet50_forward", "nm_resnet50_forward_host", "nm_pwl_table_build_elastic",
    "nm_selftest_bounded_wait", "nm_attention_pwl_i8", "nm_encoder_stack_host_async", "nm_resnet50_forward_host_async",
    "nm_resnet_conv_count",
]
KERNEL_KINDS = ("pwl_apply", "layernorm", "quantize", "linear_simt", "linear_tc", "attention_simt", "attention_tc",
                "im2col", "pool")
RESNET50_CONVS = 53


class NmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s failed: %s" % (where, status_string(code)))


class LinearDesc(C.Structure):
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("in_dtype", C.c_int), ("out_dtype", C.c_int),
                ("A", C.c_void_p), ("lda", C.c_int64), ("W", C.c_void_p), ("ldw", C.c_int64), ("bias", C.c_void_p),
                ("residual", C.c_void_p), ("ldr", C.c_int64), ("slot", C.c_int32), ("out", C.c_void_p),
                ("ldo", C.c_int64), ("a_scale", C.c_float), ("w_scale", C.c_void_p), ("inv_out_scale", C.c_float),
                ("acc_dump", C.c_void_p), ("idx_dump", C.c_void_p), ("algo", C.c_int32),
                ("res_first", C.c_int32)]


class AttnDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("heads", C.c_int32), ("d", C.c_int32), ("dtype", C.c_int),
                ("Q", C.c_void_p), ("K", C.c_void_p), ("V", C.c_void_p), ("stride_b", C.c_int64),
                ("stride_t", C.c_int64), ("scale", C.c_float), ("exp_slot", C.c_int32), ("recip_slot", C.c_int32),
                ("out", C.c_void_p), ("algo", C.c_int32)]


class AttnI8Desc(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("heads", C.c_int32), ("d", C.c_int32), ("Q", C.c_void_p),
                ("K", C.c_void_p), ("V", C.c_void_p), ("stride_b", C.c_int64), ("stride_t", C.c_int64),
                ("s_q", C.c_float), ("s_k", C.c_float), ("s_v", C.c_float), ("scale", C.c_float),
                ("exp_slot", C.c_int32), ("recip_slot", C.c_int32), ("out", C.c_void_p), ("out_dtype", C.c_int),
                ("acc_dump", C.c_void_p), ("p_dump", C.c_void_p), ("oacc_dump", C.c_void_p)]


class EncoderWeights(C.Structure):
    _fields_ = [("Wqkv", C.c_void_p), ("bqkv", C.c_void_p), ("Wo", C.c_void_p), ("bo", C.c_void_p),
                ("g1", C.c_void_p), ("be1", C.c_void_p), ("W1", C.c_void_p), ("b1", C.c_void_p),
                ("W2", C.c_void_p), ("b2", C.c_void_p), ("g2", C.c_void_p), ("be2", C.c_void_p),
                ("s_wqkv", C.c_void_p), ("s_wo", C.c_void_p), ("s_w1", C.c_void_p), ("s_w2", C.c_void_p),
                ("a_x", C.c_float), ("a_attn", C.c_float), ("a_x1", C.c_float), ("a_g", C.c_float)]


class ConvDesc(C.Structure):
    _fields_ = [("N", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("Cin", C.c_int32), ("Cout", C.c_int32),
                ("kh", C.c_int32), ("kw", C.c_int32), ("stride", C.c_int32), ("pad", C.c_int32), ("dtype", C.c_int),
                ("x", C.c_void_p), ("w", C.c_void_p), ("bias", C.c_void_p), ("residual", C.c_void_p),
                ("slot", C.c_int32), ("res_first", C.c_int32), ("out", C.c_void_p), ("algo", C.c_int32)]


class ConvParams(C.Structure):
    _fields_ = [("w", C.c_void_p), ("bias", C.c_void_p)]


class Resnet50Cfg(C.Structure):
    _fields_ = [("batch", C.c_int32), ("dtype", C.c_int), ("relu_slot", C.c_int32), ("num_classes", C.c_int32),
                ("algo", C.c_int32), ("blocks", C.c_int32 * 4), ("base_width", C.c_int32)]


class EncoderCfg(C.Structure):
    _fields_ = [("B", C.c_int32), ("L", C.c_int32), ("H", C.c_int32), ("heads", C.c_int32), ("F", C.c_int32),
                ("dtype", C.c_int), ("eps", C.c_float), ("gelu_slot", C.c_int32), ("exp_slot", C.c_int32),
                ("recip_slot", C.c_int32), ("rsqrt_slot", C.c_int32), ("algo", C.c_int32)]


_lib = None


def load():
    """Loads libnm_b200.so (built in-tree by ``build.build()``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(SO_PATH):
        raise RuntimeError("CUDA library not built: %s is missing (run python -m paper_2305_14405_b200.build)"
                           % SO_PATH)
    lib = C.CDLL(SO_PATH)
    lib.nm_status_string.restype = C.c_char_p
    lib.nm_status_string.argtypes = [C.c_int]
    lib.nm_ctx_create.argtypes = [C.POINTER(C.c_void_p), C.c_int]
    lib.nm_ctx_destroy.argtypes = [C.c_void_p]
    lib.nm_ctx_poll_status.argtypes = [C.c_void_p, C.POINTER(C.c_int), C.c_void_p]
    lib.nm_ctx_launch_count.restype = C.c_int64
    lib.nm_ctx_launch_count.argtypes = [C.c_void_p, C.c_int]
    lib.nm_pwl_table_build.argtypes = [C.c_int, C.c_int, C.c_float, C.c_float, C.POINTER(C.c_float),
                                       C.POINTER(C.c_float)]
    lib.nm_pwl_table_build_elastic.argtypes = [C.c_int, C.c_float, C.c_float, C.c_float, C.c_float, C.c_int, C.c_float,
                                               C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_float),
                                               C.POINTER(C.c_float)]
    lib.nm_pwl_table_load.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_float, C.POINTER(C.c_float),
                                      C.POINTER(C.c_float)]
    lib.nm_pwl_apply.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_void_p,
                                 C.c_void_p]
    lib.nm_linear_pwl.argtypes = [C.c_void_p, C.POINTER(LinearDesc), C.c_void_p]
    lib.nm_attention_pwl.argtypes = [C.c_void_p, C.POINTER(AttnDesc), C.c_void_p]
    lib.nm_attention_pwl_i8.argtypes = [C.c_void_p, C.POINTER(AttnI8Desc), C.c_void_p]
    lib.nm_layernorm_pwl.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                     C.c_int32, C.c_float, C.c_int32, C.c_int, C.c_void_p]
    lib.nm_layernorm_pwl_sqrt_recip.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                                C.c_int32, C.c_float, C.c_int32, C.c_int32, C.c_int, C.c_void_p]
    lib.nm_quantize_i8.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_void_p, C.c_void_p]
    lib.nm_encoder_workspace_bytes.restype = C.c_size_t
    lib.nm_encoder_workspace_bytes.argtypes = [C.POINTER(EncoderCfg)]
    lib.nm_encoder_layer.argtypes = [C.c_void_p, C.POINTER(EncoderWeights), C.POINTER(EncoderCfg), C.c_void_p,
                                     C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.nm_encoder_stack.argtypes = [C.c_void_p, C.POINTER(EncoderWeights), C.c_int32, C.POINTER(EncoderCfg),
                                     C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.nm_encoder_stack_host.argtypes = [C.c_void_p, C.POINTER(EncoderWeights), C.c_int32, C.POINTER(EncoderCfg),
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                          C.c_void_p]
    lib.nm_encoder_stack_host_async.argtypes = lib.nm_encoder_stack_host.argtypes
    lib.nm_encoder_layer_static.argtypes = [C.c_void_p, C.POINTER(EncoderWeights), C.POINTER(EncoderCfg), C.c_void_p,
                                            C.c_void_p, C.c_void_p]
    lib.nm_conv2d_workspace_bytes.restype = C.c_size_t
    lib.nm_conv2d_workspace_bytes.argtypes = [C.POINTER(ConvDesc)]
    lib.nm_conv2d_pwl.argtypes = [C.c_void_p, C.POINTER(ConvDesc), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.nm_maxpool2d.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int] + [C.c_int32] * 7 + [C.c_void_p]
    lib.nm_maxpool2d_pwl.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int] + [C.c_int32] * 8 + [C.c_void_p]
    lib.nm_avgpool_global.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int] + [C.c_int32] * 4 + [C.c_void_p]
    lib.nm_resnet50_workspace_bytes.restype = C.c_size_t
    lib.nm_resnet50_workspace_bytes.argtypes = [C.POINTER(Resnet50Cfg)]
    lib.nm_resnet50_forward.argtypes = [C.c_void_p, C.POINTER(ConvParams), C.c_void_p, C.c_void_p,
                                        C.POINTER(Resnet50Cfg), C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                        C.c_void_p]
    lib.nm_resnet50_forward_host.argtypes = [C.c_void_p, C.POINTER(ConvParams), C.c_void_p, C.c_void_p,
                                             C.POINTER(Resnet50Cfg), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.c_size_t, C.c_void_p]
    lib.nm_resnet50_forward_host_async.argtypes = lib.nm_resnet50_forward_host.argtypes
    lib.nm_resnet_conv_count.restype = C.c_int32
    lib.nm_resnet_conv_count.argtypes = [C.POINTER(Resnet50Cfg)]
    lib.nm_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    lib.nm_ctx_profile_enable.argtypes = [C.c_void_p, C.c_int]
    lib.nm_ctx_profile_read.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int64), C.POINTER(C.c_double),
                                        C.POINTER(C.c_double)]
    _lib = lib
    return lib


def status_string(code) -> str:
    return load().nm_status_string(int(code)).decode()


def _check(code, where):
    if code != NM_OK:
        raise NmError(code, where)


def _torch():
    import torch
    return torch


def dtype_of(t) -> int:
    torch = _torch()
    return {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16, torch.int8: I8}[t.dtype]


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def pwl_table_build(func: int, n: int, x_min: float, x_max: float):
    """nm_pwl_table_build: returns (k, b) as two lists of n Python floats (fp32 values)."""
    k = (C.c_float * n)()
    b = (C.c_float * n)()
    _check(load().nm_pwl_table_build(func, n, x_min, x_max, k, b), "nm_pwl_table_build")
    return list(k), list(b)


def pwl_table_build_elastic(func, r_min, r_max, dLx, dK_th, bias_correct=True, e_th=0.0):
    """nm_pwl_table_build_elastic (Algorithms 2 and 3): returns (n_cells, k, b, n_segments) on the primary grid."""
    k = (C.c_float * 256)()
    b = (C.c_float * 256)()
    n, nseg = C.c_int(0), C.c_int(0)
    _check(load().nm_pwl_table_build_elastic(func, r_min, r_max, dLx, dK_th, 1 if bias_correct else 0, e_th,
                                             C.byref(n), C.byref(nseg), k, b), "nm_pwl_table_build_elastic")
    return n.value, list(k)[:n.value], list(b)[:n.value], nseg.value


class Context:
    """Owns an nm_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        self._lib = load()
        h = C.c_void_p()
        _check(self._lib.nm_ctx_create(C.byref(h), int(device)), "nm_ctx_create")
        self._h = h
        self.device = device

    def close(self):
        if self._h:
            self._lib.nm_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- tables -------------------------------------------------------------------
    def pwl_table_load(self, slot, n, x_min, x_max, k, b):
        ka = (C.c_float * n)(*k)
        ba = (C.c_float * n)(*b)
        _check(self._lib.nm_pwl_table_load(self._h, slot, n, x_min, x_max, ka, ba), "nm_pwl_table_load")

    def load_function_table(self, slot, func, n, x_min, x_max):
        k, b = pwl_table_build(func, n, x_min, x_max)
        self.pwl_table_load(slot, n, x_min, x_max, k, b)
        return k, b

    def load_encoder_tables(self, n, ranges):
        """Loads the four tables of an encoder layer into their standard slots."""
        self.load_function_table(SLOT_GELU, FUNC_GELU, n, *ranges["gelu"])
        self.load_function_table(SLOT_EXP, FUNC_EXP, n, *ranges["exp"])
        self.load_function_table(SLOT_RECIP, FUNC_RECIP, n, *ranges["recip"])
        self.load_function_table(SLOT_RSQRT, FUNC_RSQRT, n, *ranges["rsqrt"])

    # -- status -------------------------------------------------------------------
    def poll_status(self, stream=None) -> int:
        v = C.c_int(0)
        _check(self._lib.nm_ctx_poll_status(self._h, C.byref(v), _stream(stream)), "nm_ctx_poll_status")
        return v.value

    def check_device_status(self, stream=None):
        v = self.poll_status(stream)
        if v != NM_OK:
            raise NmError(v, "device kernel")

    def selftest_bounded_wait(self, limit_cycles, stream=None):
        _check(self._lib.nm_selftest_bounded_wait(self._h, int(limit_cycles), _stream(stream)),
               "nm_selftest_bounded_wait")

    def launch_count(self, reset=False) -> int:
        return int(self._lib.nm_ctx_launch_count(self._h, 1 if reset else 0))

    def profile_enable(self, on=True):
        _check(self._lib.nm_ctx_profile_enable(self._h, 1 if on else 0), "nm_ctx_profile_enable")

    def profile_read(self):
        """{kind name: (launches, total ms, total work)} for the launches recorded since profile_enable."""
        out = {}
        for i, name in enumerate(KERNEL_KINDS):
            n, ms, work = C.c_int64(0), C.c_double(0), C.c_double(0)
            _check(self._lib.nm_ctx_profile_read(self._h, i, C.byref(n), C.byref(ms), C.byref(work)),
                   "nm_ctx_profile_read")
            out[name] = (n.value, ms.value, work.value)
        return out

    # -- kernels ------------------------------------------------------------------
    def pwl_apply(self, slot, x, y, idx_out=None, stream=None):
        _check(self._lib.nm_pwl_apply(self._h, slot, _ptr(x), _ptr(y), x.numel(), dtype_of(x), _ptr(idx_out),
                                      _stream(stream)), "nm_pwl_apply")

    def linear_pwl(self, A, W, out, bias=None, residual=None, slot=SLOT_NONE, a_scale=0.0, w_scale=None,
                   inv_out_scale=0.0, acc_dump=None, idx_dump=None, algo=ALGO_AUTO, res_first=False, stream=None):
        d = LinearDesc()
        d.M, d.K = A.shape
        d.N = W.shape[0]
        d.in_dtype = dtype_of(A)
        d.out_dtype = dtype_of(out)
        d.A, d.lda = A.data_ptr(), A.stride(0)
        d.W, d.ldw = W.data_ptr(), W.stride(0)
        d.bias = bias.data_ptr() if bias is not None else None
        d.residual = residual.data_ptr() if residual is not None else None
        d.ldr = residual.stride(0) if residual is not None else 0
        d.slot = slot
        d.out, d.ldo = out.data_ptr(), out.stride(0)
        d.a_scale = a_scale
        d.w_scale = w_scale.data_ptr() if w_scale is not None else None
        d.inv_out_scale = inv_out_scale
        d.acc_dump = acc_dump.data_ptr() if acc_dump is not None else None
        d.idx_dump = idx_dump.data_ptr() if idx_dump is not None else None
        d.algo = algo
        d.res_first = 1 if res_first else 0
        _check(self._lib.nm_linear_pwl(self._h, C.byref(d), _stream(stream)), "nm_linear_pwl")

    def attention_pwl(self, qkv, out, B, L, heads, d, scale=None, exp_slot=SLOT_EXP, recip_slot=SLOT_RECIP,
                      algo=ALGO_AUTO, stream=None):
        """qkv: packed [B*L, 3*heads*d] projection (Q | K | V); out: [B*L, heads*d]."""
        H = heads * d
        es = qkv.element_size()
        a = AttnDesc()
        a.B, a.L, a.heads, a.d = B, L, heads, d
        a.dtype = dtype_of(qkv)
        base = qkv.data_ptr()
        a.Q, a.K, a.V = base, base + H * es, base + 2 * H * es
        a.stride_b, a.stride_t = L * qkv.stride(0), qkv.stride(0)
        a.scale = float(scale) if scale is not None else float(d) ** -0.5
        a.exp_slot, a.recip_slot = exp_slot, recip_slot
        a.out = out.data_ptr()
        a.algo = algo
        _check(self._lib.nm_attention_pwl(self._h, C.byref(a), _stream(stream)), "nm_attention_pwl")

    def attention_pwl_i8(self, qkv_q, out, B, L, heads, d, s_q, s_k, s_v, scale=None, exp_slot=SLOT_EXP,
                         recip_slot=SLOT_RECIP, acc_dump=None, p_dump=None, oacc_dump=None, stream=None):
        """qkv_q: packed int8 [B*L, 3*heads*d] codes (Q | K | V); out: [B*L, heads*d] bf16 or fp32."""
        H = heads * d
        a = AttnI8Desc()
        a.B, a.L, a.heads, a.d = B, L, heads, d
        base = qkv_q.data_ptr()
        a.Q, a.K, a.V = base, base + H, base + 2 * H
        a.stride_b, a.stride_t = L * qkv_q.stride(0), qkv_q.stride(0)
        a.s_q, a.s_k, a.s_v = float(s_q), float(s_k), float(s_v)
        a.scale = float(scale) if scale is not None else float(d) ** -0.5
        a.exp_slot, a.recip_slot = exp_slot, recip_slot
        a.out, a.out_dtype = out.data_ptr(), dtype_of(out)
        a.acc_dump = acc_dump.data_ptr() if acc_dump is not None else None
        a.p_dump = p_dump.data_ptr() if p_dump is not None else None
        a.oacc_dump = oacc_dump.data_ptr() if oacc_dump is not None else None
        _check(self._lib.nm_attention_pwl_i8(self._h, C.byref(a), _stream(stream)), "nm_attention_pwl_i8")

    def layernorm_pwl(self, x, gamma, beta, y, eps=1e-5, rsqrt_slot=SLOT_RSQRT, stream=None):
        rows, H = x.shape
        _check(self._lib.nm_layernorm_pwl(self._h, _ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), rows, H, eps,
                                          rsqrt_slot, dtype_of(x), _stream(stream)), "nm_layernorm_pwl")

    def layernorm_pwl_sqrt_recip(self, x, gamma, beta, y, sqrt_slot, recip_slot, eps=1e-5, stream=None):
        rows, H = x.shape
        _check(self._lib.nm_layernorm_pwl_sqrt_recip(self._h, _ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), rows, H,
                                                     eps, sqrt_slot, recip_slot, dtype_of(x), _stream(stream)),
               "nm_layernorm_pwl_sqrt_recip")

    def quantize_i8(self, x, inv_scale, q, stream=None):
        _check(self._lib.nm_quantize_i8(self._h, _ptr(x), dtype_of(x), x.numel(), inv_scale, _ptr(q),
                                        _stream(stream)), "nm_quantize_i8")

    # -- CNN ----------------------------------------------------------------------
    @staticmethod
    def conv_desc(x, w, out, stride, pad, bias=None, residual=None, slot=SLOT_NONE, res_first=False,
                  algo=ALGO_AUTO):
        """x [N,H,W,Cin], w [Cout,kh,kw,Cin], out [N,Ho,Wo,Cout] (contiguous device tensors)."""
        d = ConvDesc()
        d.N, d.H, d.W, d.Cin = x.shape
        d.Cout, d.kh, d.kw = w.shape[0], w.shape[1], w.shape[2]
        d.stride, d.pad = stride, pad
        d.dtype = dtype_of(x)
        d.x, d.w, d.out = x.data_ptr(), w.data_ptr(), out.data_ptr()
        d.bias = bias.data_ptr() if bias is not None else None
        d.residual = residual.data_ptr() if residual is not None else None
        d.slot = slot
        d.res_first = 1 if res_first else 0
        d.algo = algo
        return d

    def conv2d_workspace_bytes(self, desc) -> int:
        return int(self._lib.nm_conv2d_workspace_bytes(C.byref(desc)))

    def conv2d_pwl(self, desc, workspace=None, stream=None):
        ws = workspace.numel() * workspace.element_size() if workspace is not None else 0
        _check(self._lib.nm_conv2d_pwl(self._h, C.byref(desc), _ptr(workspace), ws, _stream(stream)), "nm_conv2d_pwl")

    def maxpool2d(self, x, y, ks, stride, pad, stream=None):
        N, H, W, Cc = x.shape
        _check(self._lib.nm_maxpool2d(self._h, _ptr(x), _ptr(y), dtype_of(x), N, H, W, Cc, ks, stride, pad,
                                      _stream(stream)), "nm_maxpool2d")

    def maxpool2d_pwl(self, x, y, ks, stride, pad, relu_slot=SLOT_RELU, stream=None):
        N, H, W, Cc = x.shape
        _check(self._lib.nm_maxpool2d_pwl(self._h, _ptr(x), _ptr(y), dtype_of(x), N, H, W, Cc, ks, stride, pad,
                                          relu_slot, _stream(stream)), "nm_maxpool2d_pwl")

    def avgpool_global(self, x, y, stream=None):
        N, H, W, Cc = x.shape
        _check(self._lib.nm_avgpool_global(self._h, _ptr(x), _ptr(y), dtype_of(x), N, H, W, Cc, _stream(stream)),
               "nm_avgpool_global")

    @staticmethod
    def resnet50_cfg(batch, dtype, num_classes=1000, relu_slot=SLOT_RELU, algo=ALGO_AUTO, blocks=None, base_width=0):
        """blocks: bottleneck blocks of the four stages (None: ResNet-50's 3, 4, 6, 3); base_width: width of the
        first stage (0: 64)."""
        c = Resnet50Cfg()
        c.batch, c.dtype, c.relu_slot, c.num_classes, c.algo = batch, dtype, relu_slot, num_classes, algo
        if blocks is not None:
            for i in range(4):
                c.blocks[i] = blocks[i]
        c.base_width = base_width
        return c

    def resnet_conv_count(self, cfg) -> int:
        return int(self._lib.nm_resnet_conv_count(C.byref(cfg)))

    def resnet50_workspace_bytes(self, cfg) -> int:
        return int(self._lib.nm_resnet50_workspace_bytes(C.byref(cfg)))

    def resnet50_forward(self, conv_array, fc_w, fc_b, cfg, x, logits, workspace, stream=None):
        _check(self._lib.nm_resnet50_forward(self._h, conv_array, _ptr(fc_w), _ptr(fc_b), C.byref(cfg), _ptr(x),
                                             _ptr(logits), _ptr(workspace),
                                             workspace.numel() * workspace.element_size(), _stream(stream)),
               "nm_resnet50_forward")

    def resnet50_forward_host(self, conv_array, fc_w, fc_b, cfg, x_host, logits_host, x_dev, logits_dev, workspace,
                              stream=None, wait=True):
        """wait=False: nm_resnet50_forward_host_async (the caller synchronises the stream)."""
        name = "nm_resnet50_forward_host" if wait else "nm_resnet50_forward_host_async"
        _check(getattr(self._lib, name)(self._h, conv_array, _ptr(fc_w), _ptr(fc_b), C.byref(cfg),
                                        C.c_void_p(x_host.data_ptr()), C.c_void_p(logits_host.data_ptr()),
                                        _ptr(x_dev), _ptr(logits_dev), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)), name)

    # -- encoder ------------------------------------------------------------------
    @staticmethod
    def encoder_cfg(B, L, H, heads, F, dtype, eps=1e-5, algo=ALGO_AUTO):
        c = EncoderCfg()
        c.B, c.L, c.H, c.heads, c.F = B, L, H, heads, F
        c.dtype = dtype
        c.eps = eps
        c.gelu_slot, c.exp_slot, c.recip_slot, c.rsqrt_slot = SLOT_GELU, SLOT_EXP, SLOT_RECIP, SLOT_RSQRT
        c.algo = algo
        return c

    def encoder_workspace_bytes(self, cfg) -> int:
        return int(self._lib.nm_encoder_workspace_bytes(C.byref(cfg)))

    @staticmethod
    def encoder_weights(w: dict):
        """w maps the field names of nm_encoder_weights to device tensors (or floats for a_*)."""
        s = EncoderWeights()
        for name, _ in EncoderWeights._fields_:
            v = w.get(name)
            if name.startswith("a_"):
                setattr(s, name, float(v) if v is not None else 0.0)
            else:
                setattr(s, name, v.data_ptr() if v is not None else None)
        return s

    def encoder_layer(self, weights, cfg, x, y, workspace, stream=None):
        _check(self._lib.nm_encoder_layer(self._h, C.byref(weights), C.byref(cfg), _ptr(x), _ptr(y),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)), "nm_encoder_layer")

    def encoder_layer_static(self, weights, cfg, x, y, stream=None):
        """nm_encoder_layer_static: the layer with the library's own fixed scratch array instead of a
        caller workspace, for callers that cannot allocate device memory.  Raises NmError
        (NM_ERR_WORKSPACE) when the configuration needs more than STATIC_WS_BYTES."""
        _check(self._lib.nm_encoder_layer_static(self._h, C.byref(weights), C.byref(cfg), _ptr(x), _ptr(y),
                                                 _stream(stream)), "nm_encoder_layer_static")

    def encoder_stack(self, layer_array, n_layers, cfg, x, y, workspace, stream=None):
        _check(self._lib.nm_encoder_stack(self._h, layer_array, n_layers, C.byref(cfg), _ptr(x), _ptr(y),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)), "nm_encoder_stack")

    def encoder_stack_host(self, layer_array, n_layers, cfg, x_host, y_host, x_dev, y_dev, workspace, stream=None,
                           wait=True):
        """x_host / y_host: CPU tensors (pinned for full copy speed).  wait=False: nm_encoder_stack_host_async
        (the caller synchronises the stream before reading y_host)."""
        name = "nm_encoder_stack_host" if wait else "nm_encoder_stack_host_async"
        _check(getattr(self._lib, name)(self._h, layer_array, n_layers, C.byref(cfg),
                                        C.c_void_p(x_host.data_ptr()), C.c_void_p(y_host.data_ptr()),
                                        _ptr(x_dev), _ptr(y_dev), _ptr(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)), name)


def layer_array(weight_structs):
    """A C array of nm_encoder_weights from a list of EncoderWeights."""
    arr = (EncoderWeights * len(weight_structs))()
    for i, s in enumerate(weight_structs):
        arr[i] = s
    return arr
