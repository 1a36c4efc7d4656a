"""ctypes binding of the operator-level entry points (include/fax_ops.h)."""
from __future__ import annotations

import ctypes as C

FAX_EPI_NONE, FAX_EPI_BIAS, FAX_EPI_BIAS_GELU, FAX_EPI_BIAS_RESID, FAX_EPI_DGELU = range(5)

_P = C.c_void_p


class GemmDesc(C.Structure):
    _fields_ = [("M", C.c_int32), ("N", C.c_int32), ("K", C.c_int32),
                ("A", _P), ("lda", C.c_int64), ("a_mn_major", C.c_int32),
                ("B", _P), ("ldb", C.c_int64), ("b_mn_major", C.c_int32),
                ("C", _P), ("ldc", C.c_int64), ("c_f32", C.c_int32), ("accumulate", C.c_int32),
                ("epilogue", C.c_int32), ("bias", _P), ("resid", _P), ("ldr", C.c_int64),
                ("aux", _P), ("ldaux", C.c_int64), ("alpha", C.c_float), ("force_simt", C.c_int32)]


_SIGNATURES = {
    "fax_op_gemm": (C.c_int32, [_P, C.c_int32, C.POINTER(GemmDesc)]),
    "fax_op_layernorm_forward": (C.c_int32, [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, C.c_float,
                                             _P, _P, _P]),
    "fax_op_layernorm_backward_scratch_bytes": (C.c_int32, [C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]),
    "fax_op_layernorm_backward": (C.c_int32, [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, _P, _P, _P,
                                              _P, _P, _P, _P, C.c_size_t]),
    "fax_op_layernorm_backward_static": (C.c_int32, [_P, C.c_int32, C.c_int32, C.c_int32, _P, _P, _P, _P, _P, _P,
                                                     _P, _P, _P]),
    "fax_op_attention_forward": (C.c_int32, [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                             _P, _P, _P]),
    "fax_op_attention_backward_scratch_bytes": (C.c_int32, [C.c_int32] * 5 + [C.POINTER(C.c_size_t)]),
    "fax_op_attention_backward": (C.c_int32, [_P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                              _P, _P, _P, _P, _P, _P, C.c_size_t]),
}

_lib = None


def register(lib):
    global _lib
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib


def _L():
    if _lib is None:
        from . import binding
        binding.load_library()
    return _lib


def _check(s, where):
    if s != 0:
        from .binding import FaxError
        raise FaxError(s, where)


def fax_op_gemm(ctx, prec, desc: GemmDesc):
    _check(_L().fax_op_gemm(ctx, prec, C.byref(desc)), "fax_op_gemm")


def fax_op_layernorm_forward(ctx, prec, rows, d, x, gamma, beta, eps, out, mu, rstd):
    _check(_L().fax_op_layernorm_forward(ctx, prec, rows, d, x, gamma, beta, eps, out, mu, rstd),
           "fax_op_layernorm_forward")


def fax_op_layernorm_backward_scratch_bytes(rows, d) -> int:
    b = C.c_size_t()
    _check(_L().fax_op_layernorm_backward_scratch_bytes(rows, d, C.byref(b)), "fax_op_layernorm_backward_scratch_bytes")
    return b.value


def fax_op_layernorm_backward(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta, scratch,
                              scratch_bytes):
    _check(_L().fax_op_layernorm_backward(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta,
                                          scratch, scratch_bytes), "fax_op_layernorm_backward")


def fax_op_layernorm_backward_static(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma, dbeta):
    """LayerNorm backward whose scratch is a fixed array inside the library: for callers that
    cannot allocate device memory or pass any.  Same results as fax_op_layernorm_backward."""
    _check(_L().fax_op_layernorm_backward_static(ctx, prec, rows, d, da, x, mu, rstd, gamma, add, dx, dgamma,
                                                 dbeta), "fax_op_layernorm_backward_static")


def fax_op_attention_forward(ctx, prec, batch, seq, n_heads, head_dim, qkv, o, lse):
    _check(_L().fax_op_attention_forward(ctx, prec, batch, seq, n_heads, head_dim, qkv, o, lse),
           "fax_op_attention_forward")


def fax_op_attention_backward_scratch_bytes(prec, batch, seq, n_heads, head_dim) -> int:
    b = C.c_size_t()
    _check(_L().fax_op_attention_backward_scratch_bytes(prec, batch, seq, n_heads, head_dim, C.byref(b)),
           "fax_op_attention_backward_scratch_bytes")
    return b.value


def fax_op_attention_backward(ctx, prec, batch, seq, n_heads, head_dim, qkv, o, lse, d_o, dqkv, scratch,
                              scratch_bytes):
    _check(_L().fax_op_attention_backward(ctx, prec, batch, seq, n_heads, head_dim, qkv, o, lse, d_o, dqkv,
                                          scratch, scratch_bytes), "fax_op_attention_backward")
