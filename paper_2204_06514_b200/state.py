"""Device-memory plumbing for the C-ABI library: allocates parameters,
optimizer state and arenas with torch and fills the ctypes structs.  No
arithmetic of the training step lives here -- every step runs in libfax.so."""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from . import binding as fx
from .synth import Config

PARAM_NAMES = fx.PARAM_NAMES


def _ptr(t: torch.Tensor | None):
    return C.c_void_p(0 if t is None else t.data_ptr())


def block_cfg(cfg: Config, prec: int, recompute: int = 0) -> fx.BlockCfg:
    return fx.BlockCfg(cfg.batch, cfg.seq, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ff, cfg.ln_eps, prec,
                       recompute)


def hparams(lr, beta1, beta2, eps, step, grad_is_bf16=0, **_) -> fx.AdamwHparams:
    return fx.AdamwHparams(lr, beta1, beta2, eps, step, grad_is_bf16)


class ParamSet:
    """One trainable tensor on the device: fp32 master, compute copy, m, v, g."""

    def __init__(self, w: np.ndarray | torch.Tensor, prec: int, device, weight_decay: float):
        w = torch.as_tensor(w, dtype=torch.float32)
        self.w = w.to(device).contiguous()
        self.wc = self.w.to(torch.bfloat16) if prec == fx.FAX_PREC_BF16 else None
        self.m = torch.zeros_like(self.w)
        self.v = torch.zeros_like(self.w)
        self.g = torch.zeros_like(self.w)
        self.weight_decay = weight_decay

    def compute(self) -> torch.Tensor:
        return self.w if self.wc is None else self.wc

    def struct(self) -> fx.Param:
        return fx.Param(_ptr(self.w), _ptr(self.wc), _ptr(self.m), _ptr(self.v), _ptr(self.g),
                        self.w.numel(), self.weight_decay)

    def adamw_tensor(self) -> fx.AdamwTensor:
        return fx.AdamwTensor(_ptr(self.w), _ptr(self.m), _ptr(self.v), _ptr(self.g), _ptr(self.wc),
                              self.w.numel(), self.weight_decay)


class Session:
    """Owns a fax context bound to torch's current stream on one device."""

    def __init__(self, device: int = 0):
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.stream = torch.cuda.current_stream(self.device)
        self.ctx = fx.fax_create(device, self.stream.cuda_stream)

    def close(self):
        if self.ctx is not None:
            fx.fax_destroy(self.ctx)
            self.ctx = None

    def launches(self) -> int:
        return fx.fax_launch_count(self.ctx)

    def arena(self, nbytes: int) -> torch.Tensor:
        return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device)


class BlockRunner:
    """One decoder block with its training state resident on the device."""

    def __init__(self, sess: Session, cfg: Config, params: dict, prec: int = fx.FAX_PREC_BF16,
                 weight_decay: float = 0.1, host_io: bool = False, recompute: bool = False):
        self.sess, self.cfg, self.prec = sess, cfg, prec
        self.bcfg = block_cfg(cfg, prec, int(recompute))
        self.dtype = torch.bfloat16 if prec == fx.FAX_PREC_BF16 else torch.float32
        self.p = {k: ParamSet(params[k], prec, sess.device, weight_decay) for k in PARAM_NAMES}
        self.saved_bytes, self.scratch_bytes = fx.fax_block_sizes(self.bcfg)
        if host_io:
            self.scratch_bytes = fx.fax_block_host_scratch_bytes(self.bcfg)
        self.saved = sess.arena(self.saved_bytes)
        self.scratch = sess.arena(self.scratch_bytes)
        self.params_struct = fx.BlockParams(*[_ptr(self.p[k].compute()) for k in PARAM_NAMES])
        self.grads_struct = fx.BlockGrads(*[_ptr(self.p[k].g) for k in PARAM_NAMES])
        self.state = fx.BlockState(fx.LayerState(*[self.p[k].struct() for k in PARAM_NAMES]),
                                   _ptr(self.saved), self.saved_bytes, _ptr(self.scratch), self.scratch_bytes)
        n, d = cfg.tokens, cfg.d_model
        self.y = torch.empty((n, d), dtype=self.dtype, device=sess.device)
        self.dx = torch.empty((n, d), dtype=self.dtype, device=sess.device)

    def to_device(self, a: np.ndarray) -> torch.Tensor:
        return torch.as_tensor(a, dtype=torch.float32).to(self.sess.device).to(self.dtype).contiguous()

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        fx.fax_block_forward(self.sess.ctx, self.bcfg, self.params_struct, _ptr(x), _ptr(self.y),
                             _ptr(self.saved), self.saved_bytes, _ptr(self.scratch), self.scratch_bytes)
        return self.y

    def backward(self, dy: torch.Tensor, accumulate: bool = False) -> torch.Tensor:
        fx.fax_block_backward(self.sess.ctx, self.bcfg, self.params_struct, _ptr(dy), _ptr(self.saved),
                              self.saved_bytes, _ptr(self.dx), self.grads_struct, accumulate,
                              _ptr(self.scratch), self.scratch_bytes)
        return self.dx

    def adamw(self, hp: fx.AdamwHparams):
        fx.fax_adamw_step(self.sess.ctx, [self.p[k].adamw_tensor() for k in PARAM_NAMES], hp)

    def step(self, x: torch.Tensor, dy: torch.Tensor, hp: fx.AdamwHparams):
        fx.fax_block_step(self.sess.ctx, self.bcfg, self.state, _ptr(x), _ptr(dy), _ptr(self.y), _ptr(self.dx), hp)

    def step_host(self, x_host, dy_host, y_host, dx_host, hp):
        fx.fax_block_step_host(self.sess.ctx, self.bcfg, self.state, _ptr(x_host), _ptr(dy_host),
                               _ptr(y_host), _ptr(dx_host), hp)


class LmRunner:
    """N-layer LM with its training state resident on the device."""

    def __init__(self, sess: Session, cfg: Config, lm: dict, prec: int = fx.FAX_PREC_BF16,
                 weight_decay: float = 0.1, recompute: bool = False, head_rows: int = 0):
        self.sess, self.cfg, self.prec = sess, cfg, prec
        self.lcfg = fx.LmCfg(cfg.n_layers, cfg.vocab, lm["wpe"].shape[0], block_cfg(cfg, prec, int(recompute)),
                             head_rows)
        mk = lambda a: ParamSet(a, prec, sess.device, weight_decay)
        self.wte, self.wpe = mk(lm["wte"]), mk(lm["wpe"])
        self.lnf_g, self.lnf_b = mk(lm["lnf_g"]), mk(lm["lnf_b"])
        self.layers = [{k: mk(p[k]) for k in PARAM_NAMES} for p in lm["blocks"]]
        self.layer_array = (fx.LayerState * cfg.n_layers)(
            *[fx.LayerState(*[L[k].struct() for k in PARAM_NAMES]) for L in self.layers])
        self.saved_bytes, self.scratch_bytes = fx.fax_lm_sizes(self.lcfg)
        self.saved = sess.arena(self.saved_bytes)
        self.scratch = sess.arena(self.scratch_bytes)
        self.state = fx.LmState(self.wte.struct(), self.wpe.struct(), self.lnf_g.struct(), self.lnf_b.struct(),
                                C.cast(self.layer_array, C.POINTER(fx.LayerState)),
                                _ptr(self.saved), self.saved_bytes, _ptr(self.scratch), self.scratch_bytes)
        self.loss = torch.zeros(1, dtype=torch.float32, device=sess.device)

    def named_params(self):
        out = [("wte", self.wte), ("wpe", self.wpe)]
        for l, L in enumerate(self.layers):
            out += [(f"blocks.{l}.{k}", L[k]) for k in PARAM_NAMES]
        out += [("lnf_g", self.lnf_g), ("lnf_b", self.lnf_b)]
        return out

    def forward_backward(self, ids: torch.Tensor, targets: torch.Tensor):
        fx.fax_lm_forward_backward(self.sess.ctx, self.lcfg, self.state, _ptr(ids), _ptr(targets), _ptr(self.loss))

    def step(self, ids, targets, hp, want_host_loss=False):
        return fx.fax_lm_step(self.sess.ctx, self.lcfg, self.state, _ptr(ids), _ptr(targets), hp,
                              _ptr(self.loss), want_host_loss)

    def accumulate(self, ids, targets, accumulate: bool, grad_scale: float):
        fx.fax_lm_accumulate(self.sess.ctx, self.lcfg, self.state, _ptr(ids), _ptr(targets), _ptr(self.loss),
                             accumulate, grad_scale)

    def apply_adamw(self, hp):
        fx.fax_lm_apply_adamw(self.sess.ctx, self.lcfg, self.state, hp)

    def step_host(self, ids_host, targets_host, hp) -> float:
        return fx.fax_lm_step_host(self.sess.ctx, self.lcfg, self.state, _ptr(ids_host), _ptr(targets_host),
                                   hp, _ptr(self.loss))
