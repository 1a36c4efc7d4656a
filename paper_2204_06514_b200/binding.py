"""ctypes binding of libfax.so: same names as include/fax.h, argument
marshalling only.  Every function raises FaxError on a non-zero status; there
is no fallback of any kind -- if the CUDA library is missing, loading fails."""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libfax.so")

FAX_OK = 0
FAX_ERR_INVALID_ARG = -1
FAX_ERR_UNSUPPORTED_SHAPE = -2
FAX_ERR_WORKSPACE_TOO_SMALL = -3
FAX_ERR_CUDA = -4
FAX_ERR_ARCH = -5
FAX_ERR_TIMEOUT = -6
FAX_PREC_BF16 = 0
FAX_PREC_FP32_VALIDATE = 1

PARAM_NAMES = ("ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
               "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2")


class FaxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


FAX_KERNEL_CLASSES = 10


class ProfileEntry(C.Structure):
    _fields_ = [("launches", C.c_int64), ("ms", C.c_double), ("flops", C.c_double), ("bytes", C.c_double)]


class BlockCfg(C.Structure):
    _fields_ = [("batch", C.c_int32), ("seq", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("ln_eps", C.c_float), ("prec", C.c_int32),
                ("recompute", C.c_int32)]


class BlockParams(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in PARAM_NAMES]


class BlockGrads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in PARAM_NAMES]


class AdamwTensor(C.Structure):
    _fields_ = [("w", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p), ("g", C.c_void_p),
                ("w_compute", C.c_void_p), ("n", C.c_uint64), ("weight_decay", C.c_float)]


class AdamwHparams(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("step", C.c_int32), ("grad_is_bf16", C.c_int32)]


class Param(C.Structure):
    _fields_ = [("w", C.c_void_p), ("w_compute", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p),
                ("g", C.c_void_p), ("n", C.c_uint64), ("weight_decay", C.c_float)]


class LayerState(C.Structure):
    _fields_ = [(n, Param) for n in PARAM_NAMES]


class BlockState(C.Structure):
    _fields_ = [("layer", LayerState), ("saved", C.c_void_p), ("saved_bytes", C.c_size_t),
                ("scratch", C.c_void_p), ("scratch_bytes", C.c_size_t)]


class LmCfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("vocab", C.c_int32), ("max_seq", C.c_int32), ("block", BlockCfg),
                ("head_rows", C.c_int32)]


class LmState(C.Structure):
    _fields_ = [("wte", Param), ("wpe", Param), ("lnf_g", Param), ("lnf_b", Param),
                ("layers", C.POINTER(LayerState)), ("saved", C.c_void_p), ("saved_bytes", C.c_size_t),
                ("scratch", C.c_void_p), ("scratch_bytes", C.c_size_t)]


_P = C.c_void_p
_SIGNATURES = {
    "fax_status_string": (C.c_char_p, [C.c_int32]),
    "fax_create": (C.c_int32, [C.POINTER(_P), C.c_int32, _P]),
    "fax_destroy": (C.c_int32, [_P]),
    "fax_last_cuda_error": (C.c_int32, [_P]),
    "fax_check_device_status": (C.c_int32, [_P, C.POINTER(C.c_int32)]),
    "fax_launch_count": (C.c_uint64, [_P]),
    "fax_set_adamw_overlap": (C.c_int32, [_P, C.c_int32]),
    "fax_set_gemm_two_cta": (C.c_int32, [_P, C.c_int32]),
    "fax_set_dependent_launch": (C.c_int32, [_P, C.c_int32]),
    "fax_set_graph_replay": (C.c_int32, [_P, C.c_int32]),
    "fax_set_attention_backward_two_chains": (C.c_int32, [_P, C.c_int32]),
    "fax_set_gemm_l2_budget": (C.c_int32, [_P, C.c_int64]),
    "fax_set_fused_update": (C.c_int32, [_P, C.c_int32, C.c_int32]),
    "fax_profile_begin": (C.c_int32, [_P]),
    "fax_profile_end": (C.c_int32, [_P, C.POINTER(ProfileEntry), C.c_int32]),
    "fax_kernel_class_name": (C.c_char_p, [C.c_int32]),
    "fax_block_sizes": (C.c_int32, [C.POINTER(BlockCfg), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "fax_block_arena_layout": (C.c_int32, [C.POINTER(BlockCfg), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "fax_lm_arena_layout": (C.c_int32, [C.POINTER(LmCfg), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t),
                                        C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "fax_block_forward": (C.c_int32, [_P, C.POINTER(BlockCfg), C.POINTER(BlockParams), _P, _P, _P,
                                      C.c_size_t, _P, C.c_size_t]),
    "fax_block_backward": (C.c_int32, [_P, C.POINTER(BlockCfg), C.POINTER(BlockParams), _P, _P, C.c_size_t,
                                       _P, C.POINTER(BlockGrads), C.c_int32, _P, C.c_size_t]),
    "fax_adamw_step": (C.c_int32, [_P, C.POINTER(AdamwTensor), C.c_int32, C.POINTER(AdamwHparams)]),
    "fax_block_step": (C.c_int32, [_P, C.POINTER(BlockCfg), C.POINTER(BlockState), _P, _P, _P, _P,
                                   C.POINTER(AdamwHparams)]),
    "fax_block_host_scratch_bytes": (C.c_int32, [C.POINTER(BlockCfg), C.POINTER(C.c_size_t)]),
    "fax_block_step_host": (C.c_int32, [_P, C.POINTER(BlockCfg), C.POINTER(BlockState), _P, _P, _P, _P,
                                        C.POINTER(AdamwHparams)]),
    "fax_lm_sizes": (C.c_int32, [C.POINTER(LmCfg), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "fax_lm_step": (C.c_int32, [_P, C.POINTER(LmCfg), C.POINTER(LmState), _P, _P, C.POINTER(AdamwHparams),
                                _P, C.POINTER(C.c_float)]),
    "fax_lm_forward_backward": (C.c_int32, [_P, C.POINTER(LmCfg), C.POINTER(LmState), _P, _P, _P]),
    "fax_lm_accumulate": (C.c_int32, [_P, C.POINTER(LmCfg), C.POINTER(LmState), _P, _P, _P, C.c_int32, C.c_float]),
    "fax_lm_apply_adamw": (C.c_int32, [_P, C.POINTER(LmCfg), C.POINTER(LmState), C.POINTER(AdamwHparams)]),
    "fax_lm_step_host": (C.c_int32, [_P, C.POINTER(LmCfg), C.POINTER(LmState), _P, _P,
                                     C.POINTER(AdamwHparams), _P, C.POINTER(C.c_float)]),
}

_lib = None


def load_library(path: str | None = None):
    """Load libfax.so (no build, no fallback).  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} not found: build it with `python -m paper_2204_06514_b200.build`; "
                           "there is no CPU or library fallback")
    lib = C.CDLL(p)
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _register_ops(lib)
    _lib = lib
    return lib


def _register_ops(lib):
    from . import binding_ops
    binding_ops.register(lib)


def status_string(status: int) -> str:
    return load_library().fax_status_string(status).decode()


def _check(status: int, where: str):
    if status != FAX_OK:
        raise FaxError(status, where)


def fax_create(device_ordinal: int, cuda_stream: int = 0) -> C.c_void_p:
    out = C.c_void_p()
    _check(load_library().fax_create(C.byref(out), device_ordinal, C.c_void_p(cuda_stream)), "fax_create")
    return out


def fax_destroy(ctx):
    _check(load_library().fax_destroy(ctx), "fax_destroy")


def fax_last_cuda_error(ctx) -> int:
    return load_library().fax_last_cuda_error(ctx)


def fax_launch_count(ctx) -> int:
    return load_library().fax_launch_count(ctx)


def fax_check_device_status(ctx) -> tuple[int, int]:
    """Returns (status, detail) without raising on FAX_ERR_TIMEOUT."""
    d = C.c_int32(0)
    s = load_library().fax_check_device_status(ctx, C.byref(d))
    if s not in (FAX_OK, FAX_ERR_TIMEOUT):
        raise FaxError(s, "fax_check_device_status")
    return s, d.value


def fax_set_adamw_overlap(ctx, enable: bool):
    _check(load_library().fax_set_adamw_overlap(ctx, int(bool(enable))), "fax_set_adamw_overlap")


def fax_set_fused_update(ctx, enable: bool, keep_gradients: bool = False):
    _check(load_library().fax_set_fused_update(ctx, int(bool(enable)), int(bool(keep_gradients))),
           "fax_set_fused_update")


def fax_set_graph_replay(ctx, enable: bool):
    _check(load_library().fax_set_graph_replay(ctx, int(bool(enable))), "fax_set_graph_replay")


def fax_set_gemm_two_cta(ctx, enable: bool):
    _check(load_library().fax_set_gemm_two_cta(ctx, int(bool(enable))), "fax_set_gemm_two_cta")


def fax_set_dependent_launch(ctx, enable: bool):
    _check(load_library().fax_set_dependent_launch(ctx, int(bool(enable))), "fax_set_dependent_launch")


def fax_set_gemm_l2_budget(ctx, nbytes: int):
    _check(load_library().fax_set_gemm_l2_budget(ctx, int(nbytes)), "fax_set_gemm_l2_budget")


def fax_set_attention_backward_two_chains(ctx, mode: int):
    _check(load_library().fax_set_attention_backward_two_chains(ctx, int(mode)),
           "fax_set_attention_backward_two_chains")


def fax_profile_begin(ctx):
    _check(load_library().fax_profile_begin(ctx), "fax_profile_begin")


def fax_profile_end(ctx) -> dict:
    """Per kernel class: dict(launches, ms, flops, bytes); classes never launched are left out."""
    arr = (ProfileEntry * FAX_KERNEL_CLASSES)()
    _check(load_library().fax_profile_end(ctx, arr, FAX_KERNEL_CLASSES), "fax_profile_end")
    out = {}
    for i in range(FAX_KERNEL_CLASSES):
        if arr[i].launches:
            out[fax_kernel_class_name(i)] = dict(launches=arr[i].launches, ms=arr[i].ms, flops=arr[i].flops,
                                                 bytes=arr[i].bytes)
    return out


def fax_kernel_class_name(cls: int) -> str:
    return load_library().fax_kernel_class_name(cls).decode()


def fax_block_sizes(cfg: BlockCfg) -> tuple[int, int]:
    a, b = C.c_size_t(), C.c_size_t()
    _check(load_library().fax_block_sizes(C.byref(cfg), C.byref(a), C.byref(b)), "fax_block_sizes")
    return a.value, b.value


SAVED_NAMES = ("x", "a", "qkv", "o", "x1", "m", "h", "g", "mu1", "rstd1", "mu2", "rstd2", "lse")
SCRATCH_NAMES = ("dh", "dqkv", "da", "dx1")


def fax_block_arena_layout(cfg: BlockCfg) -> tuple[dict, dict]:
    """(saved offsets by name, scratch offsets by name), in bytes."""
    a, b = (C.c_size_t * 13)(), (C.c_size_t * 4)()
    _check(load_library().fax_block_arena_layout(C.byref(cfg), a, b), "fax_block_arena_layout")
    return dict(zip(SAVED_NAMES, a)), dict(zip(SCRATCH_NAMES, b))


def fax_lm_arena_layout(cfg: LmCfg) -> dict:
    L = cfg.n_layers
    act, lay = (C.c_size_t * (L + 1))(), (C.c_size_t * L)()
    xf, rl, bs = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(load_library().fax_lm_arena_layout(C.byref(cfg), act, lay, C.byref(xf), C.byref(rl), C.byref(bs)),
           "fax_lm_arena_layout")
    return dict(act=list(act), layer_saved=list(lay), xf=xf.value, row_loss=rl.value, block_scratch=bs.value)


def fax_block_host_scratch_bytes(cfg: BlockCfg) -> int:
    a = C.c_size_t()
    _check(load_library().fax_block_host_scratch_bytes(C.byref(cfg), C.byref(a)), "fax_block_host_scratch_bytes")
    return a.value


def fax_block_forward(ctx, cfg, params, x, y, saved, saved_bytes, scratch, scratch_bytes):
    _check(load_library().fax_block_forward(ctx, C.byref(cfg), C.byref(params), x, y, saved, saved_bytes,
                                            scratch, scratch_bytes), "fax_block_forward")


def fax_block_backward(ctx, cfg, params, dy, saved, saved_bytes, dx, grads, accumulate, scratch, scratch_bytes):
    _check(load_library().fax_block_backward(ctx, C.byref(cfg), C.byref(params), dy, saved, saved_bytes, dx,
                                             C.byref(grads), int(accumulate), scratch, scratch_bytes),
           "fax_block_backward")


def fax_adamw_step(ctx, tensors, hp: AdamwHparams):
    arr = (AdamwTensor * len(tensors))(*tensors)
    _check(load_library().fax_adamw_step(ctx, arr, len(tensors), C.byref(hp)), "fax_adamw_step")


def fax_block_step(ctx, cfg, st, x, dy, y, dx, hp):
    _check(load_library().fax_block_step(ctx, C.byref(cfg), C.byref(st), x, dy, y, dx, C.byref(hp)),
           "fax_block_step")


def fax_block_step_host(ctx, cfg, st, x_host, dy_host, y_host, dx_host, hp):
    _check(load_library().fax_block_step_host(ctx, C.byref(cfg), C.byref(st), x_host, dy_host, y_host,
                                              dx_host, C.byref(hp)), "fax_block_step_host")


def fax_lm_sizes(cfg: LmCfg) -> tuple[int, int]:
    a, b = C.c_size_t(), C.c_size_t()
    _check(load_library().fax_lm_sizes(C.byref(cfg), C.byref(a), C.byref(b)), "fax_lm_sizes")
    return a.value, b.value


def fax_lm_step(ctx, cfg, st, ids, targets, hp, loss_device, want_host_loss=False):
    h = C.c_float(0.0)
    _check(load_library().fax_lm_step(ctx, C.byref(cfg), C.byref(st), ids, targets, C.byref(hp), loss_device,
                                      C.byref(h) if want_host_loss else None), "fax_lm_step")
    return h.value if want_host_loss else None


def fax_lm_forward_backward(ctx, cfg, st, ids, targets, loss_device):
    _check(load_library().fax_lm_forward_backward(ctx, C.byref(cfg), C.byref(st), ids, targets, loss_device),
           "fax_lm_forward_backward")


def fax_lm_accumulate(ctx, cfg, st, ids, targets, loss_device, accumulate: bool, grad_scale: float):
    _check(load_library().fax_lm_accumulate(ctx, C.byref(cfg), C.byref(st), ids, targets, loss_device,
                                            int(bool(accumulate)), grad_scale), "fax_lm_accumulate")


def fax_lm_apply_adamw(ctx, cfg, st, hp):
    _check(load_library().fax_lm_apply_adamw(ctx, C.byref(cfg), C.byref(st), C.byref(hp)), "fax_lm_apply_adamw")


def fax_lm_step_host(ctx, cfg, st, ids_host, targets_host, hp, loss_device) -> float:
    h = C.c_float(0.0)
    _check(load_library().fax_lm_step_host(ctx, C.byref(cfg), C.byref(st), ids_host, targets_host,
                                           C.byref(hp), loss_device, C.byref(h)), "fax_lm_step_host")
    return h.value
