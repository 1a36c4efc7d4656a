"""fp64 CPU oracle for the decoder-only Transformer training step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, double-precision
statement of what the CUDA library computes.  Only the tests, the smoke entry
and the benchmark's CPU-baseline leg may import it; the product path never
does.  It shares no code, table or helper with the CUDA sources and imports
nothing from the package.

What the paper fixes (arXiv 2204.06514): the workload is a decoder-only
Transformer with multi-head attention (Fig. 1 caption, Sec. 3.2); one training
step is forward pass, loss and backward pass (Fig. 3 caption); the optimizer is
Adam (Table 1 caption); parameters are stored as float32 (Sec. 3).  The paper
prints no formula, so every operator below is the textbook definition of the
operator it names, with these readings:

  * pre-LayerNorm residual block: x1 = x + Attn(LN1(x)); y = x1 + MLP(LN2(x1))
  * LayerNorm: biased variance, eps inside the square root
  * attention: S = q k^T / sqrt(hd), strictly-upper triangle masked to -inf,
    row softmax, no dropout
  * GELU: tanh form, 0.5 h (1 + tanh(sqrt(2/pi) (h + 0.044715 h^3)))
  * LM: x0 = wte[ids] + wpe[pos]; L blocks; final LayerNorm; logits = xf wte^T
    (tied); loss = mean over all B*T positions of (logsumexp - target logit)
  * AdamW: Adam with bias correction, eps added after the correction,
    decoupled weight decay scaled by lr

Every intermediate stays in float64; there is no blocking, fusion or
reordering beyond the definitions.  numpy's matmul is used as the library
primitive for the contractions.

Pins (tests/test_oracle_*.py): central finite differences on tiny shapes for
every gradient, causal invariance, softmax row sums, closed-form attention
cases, LayerNorm/GELU identities, uniform-logit cross-entropy = ln V, the
closed-form first AdamW step, brute-force pure-Python loops, and an
independently written torch float64 autograd module.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

PARAM_NAMES = (
    "ln1_g", "ln1_b", "w_qkv", "b_qkv", "w_o", "b_o",
    "ln2_g", "ln2_b", "w_fc1", "b_fc1", "w_fc2", "b_fc2",
)

_GELU_C = math.sqrt(2.0 / math.pi)
_GELU_A = 0.044715


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# LayerNorm (block steps F1/F5 forward, B3/B7 backward)
# --------------------------------------------------------------------------
def layernorm_fwd(x, gamma, beta, eps):
    """Row-wise LayerNorm.  x [N,d] -> (a [N,d], mu [N], rstd [N])."""
    x = _f64(x)
    mu = x.mean(axis=1)
    var = ((x - mu[:, None]) ** 2).mean(axis=1)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu[:, None]) * rstd[:, None]
    return xhat * _f64(gamma)[None, :] + _f64(beta)[None, :], mu, rstd


def layernorm_bwd(da, x, mu, rstd, gamma):
    """Reverse of layernorm_fwd.  Returns (dx, dgamma, dbeta)."""
    da = _f64(da)
    xhat = (_f64(x) - mu[:, None]) * rstd[:, None]
    u = da * _f64(gamma)[None, :]
    dx = rstd[:, None] * (u - u.mean(axis=1, keepdims=True)
                          - xhat * (u * xhat).mean(axis=1, keepdims=True))
    return dx, (da * xhat).sum(axis=0), da.sum(axis=0)


# --------------------------------------------------------------------------
# GELU, tanh form (step F6, and B1 for the derivative)
# --------------------------------------------------------------------------
def gelu_tanh(h):
    h = _f64(h)
    return 0.5 * h * (1.0 + np.tanh(_GELU_C * (h + _GELU_A * h ** 3)))


def gelu_tanh_grad(h):
    h = _f64(h)
    t = np.tanh(_GELU_C * (h + _GELU_A * h ** 3))
    return 0.5 * (1.0 + t) + 0.5 * h * (1.0 - t * t) * _GELU_C * (1.0 + 3.0 * _GELU_A * h * h)


# --------------------------------------------------------------------------
# Causal multi-head attention (steps F3 / B5)
# --------------------------------------------------------------------------
def _split_heads(qkv, B, T, H, hd):
    """qkv [B*T, 3*H*hd] with column blocks q|k|v, head h at columns h*hd.."""
    d = H * hd
    r = _f64(qkv).reshape(B, T, 3, H, hd)
    assert qkv.shape == (B * T, 3 * d)
    q = r[:, :, 0].transpose(0, 2, 1, 3)   # [B,H,T,hd]
    k = r[:, :, 1].transpose(0, 2, 1, 3)
    v = r[:, :, 2].transpose(0, 2, 1, 3)
    return q, k, v


def attention_fwd(qkv, B, T, H, hd):
    """Returns (o [B*T, H*hd], lse [B,H,T], P [B,H,T,T] or None if large)."""
    q, k, v = _split_heads(qkv, B, T, H, hd)
    o = np.empty((B, T, H, hd))
    lse = np.empty((B, H, T))
    keep_p = B * H * T * T <= (1 << 22)
    P_all = np.empty((B, H, T, T)) if keep_p else None
    future = np.triu(np.ones((T, T), dtype=bool), k=1)
    for b in range(B):
        for h in range(H):
            S = (q[b, h] @ k[b, h].T) / math.sqrt(hd)
            S[future] = -np.inf
            mx = S.max(axis=1)
            E = np.exp(S - mx[:, None])
            den = E.sum(axis=1)
            P = E / den[:, None]
            lse[b, h] = mx + np.log(den)
            o[b, :, h, :] = P @ v[b, h]
            if keep_p:
                P_all[b, h] = P
    return o.reshape(B * T, H * hd), lse, P_all


def attention_bwd(do, qkv, o, lse, B, T, H, hd):
    """Reverse of attention_fwd.  Returns dqkv [B*T, 3*H*hd]."""
    q, k, v = _split_heads(qkv, B, T, H, hd)
    do_h = _f64(do).reshape(B, T, H, hd).transpose(0, 2, 1, 3)
    o_h = _f64(o).reshape(B, T, H, hd).transpose(0, 2, 1, 3)
    dqkv = np.zeros((B, T, 3, H, hd))
    future = np.triu(np.ones((T, T), dtype=bool), k=1)
    scale = 1.0 / math.sqrt(hd)
    for b in range(B):
        for h in range(H):
            S = (q[b, h] @ k[b, h].T) * scale
            S[future] = -np.inf
            P = np.exp(S - lse[b, h][:, None])
            D = (do_h[b, h] * o_h[b, h]).sum(axis=1)
            dV = P.T @ do_h[b, h]
            dP = do_h[b, h] @ v[b, h].T
            dS = P * (dP - D[:, None])
            dqkv[b, :, 0, h, :] = (dS @ k[b, h]) * scale
            dqkv[b, :, 1, h, :] = (dS.T @ q[b, h]) * scale
            dqkv[b, :, 2, h, :] = dV
    return dqkv.reshape(B * T, 3 * H * hd)


# --------------------------------------------------------------------------
# Decoder block (steps F1..F7, B1..B7)
# --------------------------------------------------------------------------
def block_forward(x, p, B, T, H, hd, eps=1e-5):
    """Pre-LN decoder block.  x [B*T, d]; p maps PARAM_NAMES -> arrays
    (weights stored [in, out]).  Returns (y, saved dict)."""
    x = _f64(x)
    p = {k: _f64(v) for k, v in p.items()}
    a, mu1, rstd1 = layernorm_fwd(x, p["ln1_g"], p["ln1_b"], eps)
    qkv = a @ p["w_qkv"] + p["b_qkv"][None, :]
    o, lse, _ = attention_fwd(qkv, B, T, H, hd)
    x1 = x + o @ p["w_o"] + p["b_o"][None, :]
    m, mu2, rstd2 = layernorm_fwd(x1, p["ln2_g"], p["ln2_b"], eps)
    h = m @ p["w_fc1"] + p["b_fc1"][None, :]
    g = gelu_tanh(h)
    y = x1 + g @ p["w_fc2"] + p["b_fc2"][None, :]
    saved = dict(x=x, mu1=mu1, rstd1=rstd1, a=a, qkv=qkv, o=o, lse=lse, x1=x1,
                 mu2=mu2, rstd2=rstd2, m=m, h=h, g=g)
    return y, saved


def block_backward(dy, s, p, B, T, H, hd):
    """Reverse of block_forward.  Returns (dx, grads dict keyed like p)."""
    dy = _f64(dy)
    p = {k: _f64(v) for k, v in p.items()}
    gr = {}
    # y = x1 + g W2 + b2
    dg = dy @ p["w_fc2"].T
    gr["w_fc2"] = s["g"].T @ dy
    gr["b_fc2"] = dy.sum(axis=0)
    dh = dg * gelu_tanh_grad(s["h"])
    # h = m W1 + b1
    dm = dh @ p["w_fc1"].T
    gr["w_fc1"] = s["m"].T @ dh
    gr["b_fc1"] = dh.sum(axis=0)
    # m = LN2(x1); x1 also feeds the residual
    dx1_ln, gr["ln2_g"], gr["ln2_b"] = layernorm_bwd(dm, s["x1"], s["mu2"], s["rstd2"], p["ln2_g"])
    dx1 = dy + dx1_ln
    # x1 = x + o Wo + bo
    do = dx1 @ p["w_o"].T
    gr["w_o"] = s["o"].T @ dx1
    gr["b_o"] = dx1.sum(axis=0)
    dqkv = attention_bwd(do, s["qkv"], s["o"], s["lse"], B, T, H, hd)
    # qkv = a Wqkv + bqkv
    da = dqkv @ p["w_qkv"].T
    gr["w_qkv"] = s["a"].T @ dqkv
    gr["b_qkv"] = dqkv.sum(axis=0)
    dx_ln, gr["ln1_g"], gr["ln1_b"] = layernorm_bwd(da, s["x"], s["mu1"], s["rstd1"], p["ln1_g"])
    dx = dx1 + dx_ln
    extras = dict(dg=dg, dh=dh, dm=dm, dx1=dx1, do=do, dqkv=dqkv, da=da)
    return dx, gr, extras


# --------------------------------------------------------------------------
# AdamW (step U)
# --------------------------------------------------------------------------
def adamw(w, m, v, g, lr, beta1, beta2, eps, weight_decay, step):
    """One decoupled-weight-decay Adam update at step t >= 1.
    Returns new (w, m, v) in float64; inputs are not modified."""
    w, m, v, g = _f64(w), _f64(m), _f64(v), _f64(g)
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    w = w - lr * weight_decay * w - lr * mhat / (np.sqrt(vhat) + eps)
    return w, m, v


# --------------------------------------------------------------------------
# Language-model step (steps LM-E, LM-F, LM-H, LM-B)
# --------------------------------------------------------------------------
def cross_entropy(logits, targets):
    """Mean softmax cross-entropy over rows.  Returns (loss, dlogits)."""
    logits = _f64(logits)
    n = logits.shape[0]
    mx = logits.max(axis=1)
    e = np.exp(logits - mx[:, None])
    den = e.sum(axis=1)
    lse = mx + np.log(den)
    loss = (lse - logits[np.arange(n), targets]).mean()
    dl = e / den[:, None]
    dl[np.arange(n), targets] -= 1.0
    return loss, dl / n


def lm_forward_backward(ids, targets, lm, B, T, H, hd, eps=1e-5):
    """ids, targets: int arrays [B,T].  lm = dict(wte [V,d], wpe [>=T,d],
    blocks = list of block param dicts, lnf_g, lnf_b).
    Returns (loss, grads) with grads shaped like lm."""
    wte, wpe = _f64(lm["wte"]), _f64(lm["wpe"])
    ids = np.asarray(ids).reshape(-1)
    tg = np.asarray(targets).reshape(-1)
    pos = np.tile(np.arange(T), B)
    x = wte[ids] + wpe[pos]
    saved = []
    for p in lm["blocks"]:
        x, s = block_forward(x, p, B, T, H, hd, eps)
        saved.append(s)
    xf, muf, rstdf = layernorm_fwd(x, lm["lnf_g"], lm["lnf_b"], eps)
    logits = xf @ wte.T
    loss, dlogits = cross_entropy(logits, tg)
    # backward
    dwte = dlogits.T @ xf
    dxf = dlogits @ wte
    dx, dlnf_g, dlnf_b = layernorm_bwd(dxf, x, muf, rstdf, lm["lnf_g"])
    gblocks = [None] * len(lm["blocks"])
    for l in range(len(lm["blocks"]) - 1, -1, -1):
        dx, gblocks[l], _ = block_backward(dx, saved[l], lm["blocks"][l], B, T, H, hd)
    np.add.at(dwte, ids, dx)                       # tied embedding: scatter part
    dwpe = np.zeros_like(wpe)
    dwpe[:T] = dx.reshape(B, T, -1).sum(axis=0)
    grads = dict(wte=dwte, wpe=dwpe, blocks=gblocks, lnf_g=dlnf_g, lnf_b=dlnf_b)
    return loss, grads


def lm_tensors(lm):
    """Flat (name, array) enumeration: wte, wpe, per-layer params, final LN."""
    out = [("wte", lm["wte"]), ("wpe", lm["wpe"])]
    for l, p in enumerate(lm["blocks"]):
        out += [(f"blocks.{l}.{k}", p[k]) for k in PARAM_NAMES]
    out += [("lnf_g", lm["lnf_g"]), ("lnf_b", lm["lnf_b"])]
    return out


def lm_step(ids, targets, lm, opt_m, opt_v, B, T, H, hd, hp, eps=1e-5, lm_master=None):
    """Full step: loss, gradients, then AdamW on every tensor.
    lm holds the compute-precision weights used for forward/backward;
    lm_master (default lm) the float32 masters the optimizer updates (Sec. 3).
    opt_m / opt_v: dicts name -> array (same flat names as lm_tensors).
    hp: dict(lr, beta1, beta2, eps, weight_decay, step).
    Returns (loss, grads, new_w, new_m, new_v) with flat-name dicts."""
    loss, grads = lm_forward_backward(ids, targets, lm, B, T, H, hd, eps)
    gflat = dict(lm_tensors(grads))
    new_w, new_m, new_v = {}, {}, {}
    for name, w in lm_tensors(lm if lm_master is None else lm_master):
        new_w[name], new_m[name], new_v[name] = adamw(
            w, opt_m[name], opt_v[name], gflat[name], hp["lr"], hp["beta1"],
            hp["beta2"], hp["eps"], hp["weight_decay"], hp["step"])
    return loss, gflat, new_w, new_m, new_v


def block_step(x, dy, p, opt_m, opt_v, B, T, H, hd, hp, eps=1e-5, p_master=None):
    """Block forward + backward + AdamW.  p are the compute-precision weights
    used for forward/backward; p_master (default p) are the fp32 masters the
    optimizer updates.  Returns (y, dx, grads, new_w, new_m, new_v)."""
    y, s = block_forward(x, p, B, T, H, hd, eps)
    dx, gr, _ = block_backward(dy, s, p, B, T, H, hd)
    pm = p if p_master is None else p_master
    new_w, new_m, new_v = {}, {}, {}
    for k in PARAM_NAMES:
        new_w[k], new_m[k], new_v[k] = adamw(
            pm[k], opt_m[k], opt_v[k], gr[k], hp["lr"], hp["beta1"], hp["beta2"],
            hp["eps"], hp["weight_decay"], hp["step"])
    return y, dx, gr, new_w, new_m, new_v
