"""Seeded synthetic inputs for the five benchmark configurations.

This module only draws random numbers and rounds them to storage formats; it
contains none of the training step's arithmetic, so both the CUDA path and the
test oracle can be fed the same bytes from here.

Recipe: every tensor is drawn from a counter-based Philox stream keyed on
(seed, tensor_id), so a tensor's values do not depend on which other tensors
were generated.  seed = 220406514 + config index.  x, dY ~ N(0,1) rounded to
bf16; weight matrices, wte, wpe ~ N(0, 0.02^2) as float32; biases 0; LayerNorm
gamma 1, beta 0; token ids uniform on [0, V) over [B, T+1] (inputs = first T,
targets = last T of each row).
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 220406514

PARAM_NAMES = (
    "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
    "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
)


@dataclass(frozen=True)
class Config:
    name: str
    index: int
    batch: int
    seq: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    n_layers: int = 1
    vocab: int = 0            # 0: single block, no embedding / loss
    ln_eps: float = 1e-5

    @property
    def tokens(self) -> int:
        return self.batch * self.seq

    @property
    def is_lm(self) -> bool:
        return self.vocab > 0

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    def block_param_shapes(self):
        d, f = self.d_model, self.d_ff
        return {
            "ln1_g": (d,), "ln1_b": (d,), "w_qkv": (d, 3 * d), "b_qkv": (3 * d,),
            "w_o": (d, d), "b_o": (d,), "ln2_g": (d,), "ln2_b": (d,),
            "w_fc1": (d, f), "b_fc1": (f,), "w_fc2": (f, d), "b_fc2": (d,),
        }

    @property
    def n_params(self) -> int:
        per = sum(int(np.prod(s)) for s in self.block_param_shapes().values())
        n = per * self.n_layers
        if self.is_lm:
            n += self.vocab * self.d_model + self.seq * self.d_model + 2 * self.d_model
        return n

    @property
    def n_matmul_params(self) -> int:
        d, f = self.d_model, self.d_ff
        n = self.n_layers * (4 * d * d + 2 * d * f)
        if self.is_lm:
            n += self.vocab * d
        return n

    def step_flops(self, causal_halved: bool = True) -> float:
        """6 * matmul params * tokens + attention FLOPs (fwd + bwd)."""
        attn = 6.0 * self.batch * self.seq ** 2 * self.d_model * self.n_layers
        if not causal_halved:
            attn *= 2.0
        return 6.0 * self.n_matmul_params * self.tokens + attn


CONFIGS = {
    "C1": Config("C1", 0, batch=2, seq=128, d_model=256, n_heads=4, head_dim=64, d_ff=1024),
    "C2": Config("C2", 1, batch=8, seq=1024, d_model=1024, n_heads=16, head_dim=64, d_ff=4096),
    "C3": Config("C3", 2, batch=4, seq=2048, d_model=4096, n_heads=32, head_dim=128, d_ff=16384),
    "C4": Config("C4", 3, batch=16, seq=1024, d_model=768, n_heads=12, head_dim=64, d_ff=3072,
                 n_layers=12, vocab=50304),
    "C5": Config("C5", 4, batch=1, seq=2048, d_model=12288, n_heads=96, head_dim=128, d_ff=49152),
}

# Paper-shaped workloads beyond the five benchmark configs (same kernels): Table 1's hidden sizes at
# batch 1 x seq 2048 (head_dim 128, FFN 4 d: the paper gives neither), Fig. 3's 124M model at
# batch 32 x seq 2048, and a 350M-class 24-layer LM (the model size of Fig. 2).
CONFIGS.update({
    "P1": Config("P1", 5, batch=1, seq=2048, d_model=5120, n_heads=40, head_dim=128, d_ff=20480),
    "P2": Config("P2", 6, batch=1, seq=2048, d_model=10240, n_heads=80, head_dim=128, d_ff=40960),
    "P3": Config("P3", 7, batch=1, seq=2048, d_model=16384, n_heads=128, head_dim=128, d_ff=65536),
    "F3": Config("F3", 8, batch=32, seq=2048, d_model=768, n_heads=12, head_dim=64, d_ff=3072,
                 n_layers=12, vocab=50304),
    "F2": Config("F2", 9, batch=16, seq=1024, d_model=1024, n_heads=16, head_dim=64, d_ff=4096,
                 n_layers=24, vocab=50304),
})

ADAMW = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)

# fixed tensor-id enumeration
TID_X, TID_DY, TID_IDS, TID_WTE, TID_WPE, TID_STATE_M, TID_STATE_V = 0, 1, 2, 3, 4, 5, 6
TID_LAYER0 = 16           # layer l, parameter k -> TID_LAYER0 + 16*l + k


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, tensor_id]))


def normal(seed: int, tensor_id: int, shape, std: float = 1.0) -> np.ndarray:
    """float32 N(0, std^2) tensor from the (seed, tensor_id) stream."""
    a = _rng(seed, tensor_id).standard_normal(int(np.prod(shape)), dtype=np.float64)
    return (a * std).astype(np.float32).reshape(shape)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    out = ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of bf16-representable float32 values."""
    return (np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def bf16_from_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def block_params(cfg: Config, layer: int = 0) -> dict:
    """fp32 master parameters of one block."""
    out = {}
    for k, (name, shape) in enumerate(cfg.block_param_shapes().items()):
        if name.startswith("w_"):
            out[name] = normal(cfg.seed, TID_LAYER0 + 16 * layer + k, shape, 0.02)
        elif name.endswith("_g"):
            out[name] = np.ones(shape, np.float32)
        else:
            out[name] = np.zeros(shape, np.float32)
    return out


def block_inputs(cfg: Config):
    """(x, dY), each [B*T, d] float32 holding bf16-representable values."""
    shape = (cfg.tokens, cfg.d_model)
    return (round_to_bf16(normal(cfg.seed, TID_X, shape)),
            round_to_bf16(normal(cfg.seed, TID_DY, shape)))


def lm_params(cfg: Config) -> dict:
    assert cfg.is_lm
    d = cfg.d_model
    return dict(
        wte=normal(cfg.seed, TID_WTE, (cfg.vocab, d), 0.02),
        wpe=normal(cfg.seed, TID_WPE, (cfg.seq, d), 0.02),
        blocks=[block_params(cfg, l) for l in range(cfg.n_layers)],
        lnf_g=np.ones((d,), np.float32), lnf_b=np.zeros((d,), np.float32),
    )


def lm_tokens(cfg: Config):
    """(ids, targets) int32 [B,T]: one [B, T+1] draw, shifted by one."""
    raw = _rng(cfg.seed, TID_IDS).integers(0, cfg.vocab, size=(cfg.batch, cfg.seq + 1), dtype=np.int64)
    return (np.ascontiguousarray(raw[:, :-1]).astype(np.int32),
            np.ascontiguousarray(raw[:, 1:]).astype(np.int32))


def warm_state(seed: int, tensor_id: int, shape, scale: float):
    """Non-zero optimizer state: m ~ N(0, scale^2), v = m^2 + positive noise with a
    floor of (scale/2)^2, so that the update stays Lipschitz in the gradient."""
    m = normal(seed, TID_STATE_M + 1000 * tensor_id, shape, scale)
    n = normal(seed, TID_STATE_V + 1000 * tensor_id, shape, scale)
    v = m.astype(np.float64) ** 2 + n.astype(np.float64) ** 2 + (0.5 * scale) ** 2
    return m, v.astype(np.float32)


def scaled(cfg: Config, **kw) -> Config:
    """A config with some fields replaced (reduced-size parity cases)."""
    from dataclasses import replace
    return replace(cfg, **kw)
