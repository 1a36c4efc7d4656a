"""Data-parallel LM training step (include/fax_dp.h): one process per GPU, every rank holds
the whole model in flat buffers, runs forward + loss + backward on its own sequences, then

    reduce-scatter of the float32 gradients -> AdamW on this rank's shard -> all-gather of
    the bf16 compute copies

with the collectives issued through torch.distributed (NCCL on GPUs).  This module marshals
arguments, allocates the flat buffers and calls the collectives; the shard arithmetic and
every kernel are the library's.
"""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch
import torch.distributed as dist

from . import binding as fx
from .synth import Config

_P = C.c_void_p
ALIGN = 128          # elements: tensor starts and shard boundaries (256 bytes in bf16, 512 in float32)


class Piece(C.Structure):
    _fields_ = [("tensor", C.c_int32), ("begin", C.c_uint64), ("end", C.c_uint64), ("flat_begin", C.c_uint64)]


_SIGNATURES = {
    "fax_dp_layout": (C.c_int32, [C.POINTER(C.c_uint64), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_uint64),
                                  C.POINTER(C.c_uint64)]),
    "fax_dp_shard_map": (C.c_int32, [C.POINTER(C.c_uint64), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                     C.POINTER(C.c_uint64), C.POINTER(C.c_uint64), C.POINTER(Piece), C.c_int32,
                                     C.POINTER(C.c_int32)]),
    "fax_dp_adamw_shard": (C.c_int32, [_P, _P, _P, _P, _P, _P, C.POINTER(C.c_uint64), C.POINTER(C.c_float), C.c_int32,
                                       C.c_int32, C.c_int32, C.c_int32, C.POINTER(fx.AdamwHparams)]),
}
_ready = False


def _L():
    global _ready
    lib = fx.load_library()
    if not _ready:
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _ready = True
    return lib


def _check(s, where):
    if s != 0:
        raise fx.FaxError(s, where)


def _u64(values):
    return (C.c_uint64 * len(values))(*[int(v) for v in values])


def layout(sizes, world: int, align: int = ALIGN):
    """(offsets, padded_total) of the flat buffers."""
    off = (C.c_uint64 * len(sizes))()
    total = C.c_uint64()
    _check(_L().fax_dp_layout(_u64(sizes), len(sizes), align, world, off, C.byref(total)), "fax_dp_layout")
    return list(off), total.value


def shard_map(sizes, world: int, rank: int, align: int = ALIGN):
    """(shard_begin, shard_len, [(tensor, begin, end, flat_begin), ...]) of one rank."""
    pieces = (Piece * (len(sizes) + 1))()
    n = C.c_int32()
    lo, ln = C.c_uint64(), C.c_uint64()
    _check(_L().fax_dp_shard_map(_u64(sizes), len(sizes), align, world, rank, C.byref(lo), C.byref(ln), pieces,
                                 len(sizes) + 1, C.byref(n)), "fax_dp_shard_map")
    return lo.value, ln.value, [(p.tensor, p.begin, p.end, p.flat_begin) for p in pieces[:n.value]]


def adamw_shard(ctx, w, m, v, g_shard, w_compute, sizes, weight_decay, world, rank, hp, align: int = ALIGN):
    wd = (C.c_float * len(sizes))(*[float(x) for x in weight_decay])
    ptr = lambda t: C.c_void_p(0 if t is None else t.data_ptr())
    _check(_L().fax_dp_adamw_shard(ctx, ptr(w), ptr(m), ptr(v), ptr(g_shard), ptr(w_compute), _u64(sizes), wd,
                                   len(sizes), align, world, rank, C.byref(hp)), "fax_dp_adamw_shard")


def reduce_scatter_sum(flat: torch.Tensor, shard: torch.Tensor, rank: int, world: int):
    """shard <- this rank's slice of the element-wise sum of `flat` over all ranks."""
    if world == 1:
        shard.copy_(flat)
        return
    if dist.get_backend() == "nccl":
        dist.reduce_scatter_tensor(shard, flat, op=dist.ReduceOp.SUM)
    else:                       # backends without a reduce-scatter: reduce everything, keep the slice
        tmp = flat.clone()
        dist.all_reduce(tmp, op=dist.ReduceOp.SUM)
        shard.copy_(tmp[rank * shard.numel():(rank + 1) * shard.numel()])


def all_gather_shards(flat: torch.Tensor, rank: int, world: int):
    """Every rank's slice of `flat` (shard_len elements at rank * shard_len) is sent to all ranks, in place."""
    if world == 1:
        return
    n = flat.numel() // world
    if dist.get_backend() == "nccl":
        dist.all_gather_into_tensor(flat, flat[rank * n:(rank + 1) * n])
    else:
        parts = [torch.empty(n, dtype=flat.dtype, device=flat.device) for _ in range(world)]
        dist.all_gather(parts, flat[rank * n:(rank + 1) * n].clone())
        for r, p in enumerate(parts):
            flat[r * n:(r + 1) * n].copy_(p)


class _View:
    """One trainable tensor as views into the flat buffers (same fields as state.ParamSet)."""

    def __init__(self, w, wc, m, v, g, weight_decay):
        self.w, self.wc, self.m, self.v, self.g, self.weight_decay = w, wc, m, v, g, weight_decay

    def struct(self) -> fx.Param:
        p = lambda t: C.c_void_p(0 if t is None else t.data_ptr())
        return fx.Param(p(self.w), p(self.wc), p(self.m), p(self.v), p(self.g), self.w.numel(), self.weight_decay)


class DpLmRunner:
    """N-layer LM replicated on every rank, trained data-parallel.  `cfg.batch` is the GLOBAL batch; each
    rank processes cfg.batch / world sequences per step.  bf16 compute, float32 master / moments / gradients."""

    def __init__(self, sess, cfg: Config, lm: dict, weight_decay: float = 0.1, rank: int = 0, world: int = 1):
        if cfg.batch % world:
            raise ValueError("the global batch must divide evenly over the ranks")
        from .state import block_cfg
        from dataclasses import replace
        self.sess, self.cfg, self.rank, self.world = sess, cfg, rank, world
        self.local = replace(cfg, batch=cfg.batch // world)
        dev = sess.device
        names = [("wte", lm["wte"]), ("wpe", lm["wpe"])]
        for l, p in enumerate(lm["blocks"]):
            names += [(f"blocks.{l}.{k}", p[k]) for k in fx.PARAM_NAMES]
        names += [("lnf_g", lm["lnf_g"]), ("lnf_b", lm["lnf_b"])]
        self.names = [n for n, _ in names]
        self.sizes = [int(np.prod(a.shape)) for _, a in names]
        self.wd = [weight_decay] * len(names)
        self.offsets, self.total = layout(self.sizes, world)
        self.shard_begin, self.shard_len, self.pieces = shard_map(self.sizes, world, rank)
        z = lambda dt: torch.zeros(self.total, dtype=dt, device=dev)
        self.w, self.m, self.v, self.g, self.wc = z(torch.float32), z(torch.float32), z(torch.float32), \
            z(torch.float32), z(torch.bfloat16)
        self.g_shard = torch.zeros(self.shard_len, dtype=torch.float32, device=dev)
        self.params = {}
        for (name, a), off, n in zip(names, self.offsets, self.sizes):
            sl = slice(off, off + n)
            self.w[sl].copy_(torch.as_tensor(a, dtype=torch.float32).reshape(-1))
            self.params[name] = _View(self.w[sl], self.wc[sl], self.m[sl], self.v[sl], self.g[sl], weight_decay)
        self.wc.copy_(self.w)                      # initial compute copy: a cast, as state.ParamSet does
        self.lcfg = fx.LmCfg(cfg.n_layers, cfg.vocab, lm["wpe"].shape[0], block_cfg(self.local, fx.FAX_PREC_BF16, 0), 0)
        P = self.params
        self.layer_array = (fx.LayerState * cfg.n_layers)(
            *[fx.LayerState(*[P[f"blocks.{l}.{k}"].struct() for k in fx.PARAM_NAMES]) for l in range(cfg.n_layers)])
        self.saved_bytes, self.scratch_bytes = fx.fax_lm_sizes(self.lcfg)
        self.saved, self.scratch = sess.arena(self.saved_bytes), sess.arena(self.scratch_bytes)
        ptr = lambda t: C.c_void_p(t.data_ptr())
        self.state = fx.LmState(P["wte"].struct(), P["wpe"].struct(), P["lnf_g"].struct(), P["lnf_b"].struct(),
                                C.cast(self.layer_array, C.POINTER(fx.LayerState)),
                                ptr(self.saved), self.saved_bytes, ptr(self.scratch), self.scratch_bytes)
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)

    def named_params(self):
        return [(n, self.params[n]) for n in self.names]

    def local_gradients(self, ids_local: torch.Tensor, targets_local: torch.Tensor):
        """Forward + loss + backward on this rank's tokens: self.g <- gradient of (this rank's mean loss) / world,
        so that the sum over ranks is the gradient of the mean loss over the global batch."""
        ptr = lambda t: C.c_void_p(t.data_ptr())
        fx.fax_lm_accumulate(self.sess.ctx, self.lcfg, self.state, ptr(ids_local), ptr(targets_local), ptr(self.loss),
                             False, 1.0 / self.world)

    def update_shard(self, hp: fx.AdamwHparams):
        """AdamW on this rank's shard from self.g_shard (the reduced gradients)."""
        adamw_shard(self.sess.ctx, self.w, self.m, self.v, self.g_shard, self.wc, self.sizes, self.wd, self.world,
                    self.rank, hp)

    def step(self, ids_local: torch.Tensor, targets_local: torch.Tensor, hp: fx.AdamwHparams):
        """One data-parallel step on this rank's [batch / world, seq] tokens.  Afterwards every rank holds
        the same bf16 compute copies; float32 w, m, v are current only inside the rank's own shard, and
        self.g holds this rank's local gradient contribution (already divided by the world size)."""
        self.local_gradients(ids_local, targets_local)
        reduce_scatter_sum(self.g, self.g_shard, self.rank, self.world)
        self.update_shard(hp)
        all_gather_shards(self.wc, self.rank, self.world)

    def global_loss(self) -> float:
        t = self.loss.clone()
        if self.world > 1:
            dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item()) / self.world
