"""Pins for the fp64 oracle: every check here is something other than the
oracle's own formula retyped -- finite differences, invariants, closed forms,
brute-force loops and an independently written torch float64 autograd model."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fax_oracle as O

RNG = np.random.default_rng(1234)
B, T, H, HD, F, V, L = 2, 5, 2, 4, 16, 11, 2
D = H * HD


def rand_block_params(rng, d=D, f=F, scale=0.3):
    shapes = {"ln1_g": (d,), "ln1_b": (d,), "w_qkv": (d, 3 * d), "b_qkv": (3 * d,),
              "w_o": (d, d), "b_o": (d,), "ln2_g": (d,), "ln2_b": (d,),
              "w_fc1": (d, f), "b_fc1": (f,), "w_fc2": (f, d), "b_fc2": (d,)}
    p = {k: rng.standard_normal(s) * scale for k, s in shapes.items()}
    p["ln1_g"] += 1.0
    p["ln2_g"] += 1.0
    return p


def rand_lm(rng):
    return dict(wte=rng.standard_normal((V, D)) * 0.5, wpe=rng.standard_normal((T, D)) * 0.5,
                blocks=[rand_block_params(rng) for _ in range(L)],
                lnf_g=1.0 + 0.3 * rng.standard_normal(D), lnf_b=0.3 * rng.standard_normal(D))


# ---------------------------------------------------------------- finite differences
def _fd_check(fun, theta, analytic, rel=1e-6):
    """Central differences of scalar fun wrt every element of theta (in place)."""
    flat = theta.reshape(-1)
    ana = analytic.reshape(-1)
    num = np.empty_like(flat)
    for i in range(flat.size):
        old = flat[i]
        h = 1e-5 * max(1.0, abs(old))
        flat[i] = old + h
        fp = fun()
        flat[i] = old - h
        fm = fun()
        flat[i] = old
        num[i] = (fp - fm) / (2 * h)
    scale = max(np.abs(num).max(), 1e-12)
    assert np.abs(num - ana).max() / scale <= rel, (np.abs(num - ana).max(), scale)


def test_block_gradients_match_finite_differences():
    rng = np.random.default_rng(7)
    p = rand_block_params(rng)
    x = rng.standard_normal((B * T, D))
    dy = rng.standard_normal((B * T, D))

    def probe():
        y, _ = O.block_forward(x, p, B, T, H, HD)
        return float((y * dy).sum())

    y, s = O.block_forward(x, p, B, T, H, HD)
    dx, gr, _ = O.block_backward(dy, s, p, B, T, H, HD)
    _fd_check(probe, x, dx)
    for k in O.PARAM_NAMES:
        _fd_check(probe, p[k], gr[k])


def test_lm_gradients_match_finite_differences():
    rng = np.random.default_rng(8)
    lm = rand_lm(rng)
    ids = rng.integers(0, V, (B, T))
    ids[0, 1] = ids[0, 0]                       # repeated token: scatter must accumulate
    tg = rng.integers(0, V, (B, T))

    def probe():
        return float(O.lm_forward_backward(ids, tg, lm, B, T, H, HD)[0])

    loss, g = O.lm_forward_backward(ids, tg, lm, B, T, H, HD)
    _fd_check(probe, lm["wte"], g["wte"])
    _fd_check(probe, lm["wpe"], g["wpe"])
    _fd_check(probe, lm["lnf_g"], g["lnf_g"])
    _fd_check(probe, lm["lnf_b"], g["lnf_b"])
    for l in range(L):
        for k in ("w_qkv", "b_o", "ln2_g", "w_fc2", "b_fc1", "ln1_b"):
            _fd_check(probe, lm["blocks"][l][k], g["blocks"][l][k])


def test_attention_gradient_finite_differences_alone():
    rng = np.random.default_rng(9)
    qkv = rng.standard_normal((B * T, 3 * D))
    do = rng.standard_normal((B * T, D))
    o, lse, _ = O.attention_fwd(qkv, B, T, H, HD)
    dqkv = O.attention_bwd(do, qkv, o, lse, B, T, H, HD)
    _fd_check(lambda: float((O.attention_fwd(qkv, B, T, H, HD)[0] * do).sum()), qkv, dqkv)


# ---------------------------------------------------------------- independent torch fp64 model
def _torch_block(x, p, b, t, h, hd, eps=1e-5):
    d = h * hd
    F_ = torch.nn.functional
    a = F_.layer_norm(x, (d,), p["ln1_g"], p["ln1_b"], eps)
    qkv = F_.linear(a, p["w_qkv"].t(), p["b_qkv"]).view(b, t, 3, h, hd)
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    o = F_.scaled_dot_product_attention(q, k, v, is_causal=True)
    o = o.permute(0, 2, 1, 3).reshape(b * t, d)
    x1 = x + F_.linear(o, p["w_o"].t(), p["b_o"])
    m = F_.layer_norm(x1, (d,), p["ln2_g"], p["ln2_b"], eps)
    g = F_.gelu(F_.linear(m, p["w_fc1"].t(), p["b_fc1"]), approximate="tanh")
    return x1 + F_.linear(g, p["w_fc2"].t(), p["b_fc2"])


@pytest.mark.parametrize("shape", [(2, 5, 2, 4, 16), (2, 128, 4, 64, 1024)])
def test_block_matches_torch_float64_autograd(shape):
    b, t, h, hd, f = shape
    d = h * hd
    rng = np.random.default_rng(10)
    p = rand_block_params(rng, d, f, scale=0.05)
    x = rng.standard_normal((b * t, d))
    dy = rng.standard_normal((b * t, d))
    y, s = O.block_forward(x, p, b, t, h, hd)
    dx, gr, _ = O.block_backward(dy, s, p, b, t, h, hd)
    tp = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in p.items()}
    tx = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    ty = _torch_block(tx, tp, b, t, h, hd)
    ty.backward(torch.tensor(dy))

    def rel(a, bb):
        return np.abs(a - bb).max() / max(np.abs(bb).max(), 1e-300)

    assert rel(y, ty.detach().numpy()) < 1e-10
    assert rel(dx, tx.grad.numpy()) < 1e-10
    for k in O.PARAM_NAMES:
        assert rel(gr[k], tp[k].grad.numpy()) < 1e-10, k


def test_lm_matches_torch_float64_autograd():
    rng = np.random.default_rng(11)
    lm = rand_lm(rng)
    ids = rng.integers(0, V, (B, T))
    tg = rng.integers(0, V, (B, T))
    loss, g = O.lm_forward_backward(ids, tg, lm, B, T, H, HD)
    t = lambda a: torch.tensor(a, dtype=torch.float64, requires_grad=True)
    wte, wpe, lg, lb = t(lm["wte"]), t(lm["wpe"]), t(lm["lnf_g"]), t(lm["lnf_b"])
    blocks = [{k: t(v) for k, v in p.items()} for p in lm["blocks"]]
    x = wte[torch.tensor(ids).reshape(-1)] + wpe[:T].repeat(B, 1)
    for p in blocks:
        x = _torch_block(x, p, B, T, H, HD)
    xf = torch.nn.functional.layer_norm(x, (D,), lg, lb, 1e-5)
    tl = torch.nn.functional.cross_entropy(xf @ wte.t(), torch.tensor(tg).reshape(-1))
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    for mine, ref in [(g["wte"], wte.grad), (g["wpe"], wpe.grad), (g["lnf_g"], lg.grad),
                      (g["lnf_b"], lb.grad), (g["blocks"][0]["w_qkv"], blocks[0]["w_qkv"].grad),
                      (g["blocks"][1]["b_fc1"], blocks[1]["b_fc1"].grad)]:
        assert np.abs(mine - ref.numpy()).max() / np.abs(ref.numpy()).max() < 1e-10


# ---------------------------------------------------------------- brute force
def test_attention_matches_pure_python_loops():
    rng = np.random.default_rng(12)
    b, t, h, hd = 1, 4, 2, 3
    d = h * hd
    qkv = rng.standard_normal((b * t, 3 * d))
    o, lse, P = O.attention_fwd(qkv, b, t, h, hd)
    for hh in range(h):
        for i in range(t):
            s = []
            for j in range(i + 1):
                acc = 0.0
                for c in range(hd):
                    acc += qkv[i, hh * hd + c] * qkv[j, d + hh * hd + c]
                s.append(acc / math.sqrt(hd))
            den = sum(math.exp(v) for v in s)
            assert abs(lse[0, hh, i] - math.log(den)) < 1e-12
            for c in range(hd):
                want = sum(math.exp(s[j]) / den * qkv[j, 2 * d + hh * hd + c] for j in range(i + 1))
                assert abs(o[i, hh * hd + c] - want) < 1e-12


def test_layernorm_matches_pure_python_loops():
    rng = np.random.default_rng(13)
    x = rng.standard_normal((3, 6))
    g, b = rng.standard_normal(6), rng.standard_normal(6)
    a, mu, rstd = O.layernorm_fwd(x, g, b, 1e-5)
    for n in range(3):
        m = sum(x[n]) / 6
        var = sum((v - m) ** 2 for v in x[n]) / 6
        for j in range(6):
            assert abs(a[n, j] - ((x[n, j] - m) / math.sqrt(var + 1e-5) * g[j] + b[j])) < 1e-13


# ---------------------------------------------------------------- invariants and closed forms
def test_causal_invariance_is_bit_exact():
    rng = np.random.default_rng(14)
    p = rand_block_params(rng)
    x = rng.standard_normal((B * T, D))
    y0, _ = O.block_forward(x, p, B, T, H, HD)
    t = 2
    x2 = x.copy().reshape(B, T, D)
    x2[:, t + 1:, :] = rng.standard_normal((B, T - t - 1, D)) * 50
    y1, _ = O.block_forward(x2.reshape(B * T, D), p, B, T, H, HD)
    a, b_ = y0.reshape(B, T, D), y1.reshape(B, T, D)
    assert np.array_equal(a[:, :t + 1], b_[:, :t + 1])
    assert not np.allclose(a[:, t + 1:], b_[:, t + 1:])


def test_backward_causality_dx_depends_only_on_later_dy():
    rng = np.random.default_rng(15)
    p = rand_block_params(rng)
    x = rng.standard_normal((B * T, D))
    dy = rng.standard_normal((B, T, D))
    _, s = O.block_forward(x, p, B, T, H, HD)
    dx0, _, _ = O.block_backward(dy.reshape(B * T, D), s, p, B, T, H, HD)
    t = 3
    dy2 = dy.copy()
    dy2[:, :t] = rng.standard_normal((B, t, D))
    dx1, _, _ = O.block_backward(dy2.reshape(B * T, D), s, p, B, T, H, HD)
    assert np.allclose(dx0.reshape(B, T, D)[:, t:], dx1.reshape(B, T, D)[:, t:], rtol=0, atol=1e-13)


def test_softmax_rows_and_mask():
    rng = np.random.default_rng(16)
    qkv = rng.standard_normal((B * T, 3 * D)) * 3
    _, _, P = O.attention_fwd(qkv, B, T, H, HD)
    assert np.abs(P.sum(-1) - 1).max() < 1e-14
    assert np.all(P[..., np.triu(np.ones((T, T), bool), 1)] == 0.0)


def test_attention_closed_forms():
    rng = np.random.default_rng(17)
    # T = 1: o = v
    qkv = rng.standard_normal((3, 3 * D))
    o, lse, _ = O.attention_fwd(qkv, 3, 1, H, HD)
    assert np.allclose(o, qkv[:, 2 * D:], atol=1e-15)
    # q = 0: uniform weights over the prefix -> running mean of v, lse = ln(i+1)
    qkv = rng.standard_normal((B * T, 3 * D))
    qkv[:, :D] = 0
    o, lse, _ = O.attention_fwd(qkv, B, T, H, HD)
    v = qkv[:, 2 * D:].reshape(B, T, D)
    want = np.cumsum(v, axis=1) / np.arange(1, T + 1)[None, :, None]
    assert np.allclose(o.reshape(B, T, D), want, atol=1e-14)
    assert np.allclose(lse, np.log(np.arange(1, T + 1))[None, None, :], atol=1e-14)
    # identical keys: same result
    qkv = rng.standard_normal((B * T, 3 * D))
    qkv[:, D:2 * D] = qkv[0, D:2 * D]
    o, _, _ = O.attention_fwd(qkv, B, T, H, HD)
    v = qkv[:, 2 * D:].reshape(B, T, D)
    want = np.cumsum(v, axis=1) / np.arange(1, T + 1)[None, :, None]
    assert np.allclose(o.reshape(B, T, D), want, atol=1e-13)


def test_attention_backward_rows_of_ds_sum_to_zero_via_dq_for_constant_k():
    # with identical key rows k_j = c, dq_i = scale * (sum_j dS_ij) c = 0
    rng = np.random.default_rng(18)
    qkv = rng.standard_normal((B * T, 3 * D))
    qkv[:, D:2 * D] = qkv[0, D:2 * D]
    do = rng.standard_normal((B * T, D))
    o, lse, _ = O.attention_fwd(qkv, B, T, H, HD)
    dqkv = O.attention_bwd(do, qkv, o, lse, B, T, H, HD)
    assert np.abs(dqkv[:, :D]).max() < 1e-12 * np.abs(dqkv).max() + 1e-14


def test_layernorm_invariants():
    rng = np.random.default_rng(19)
    x = rng.standard_normal((7, 32)) * 3 + 1
    ones, zeros = np.ones(32), np.zeros(32)
    a, mu, rstd = O.layernorm_fwd(x, ones, zeros, 1e-5)
    assert np.abs(a.mean(1)).max() < 1e-14
    var = x.var(axis=1)
    assert np.allclose(a.var(axis=1), var / (var + 1e-5), atol=1e-13)
    da = rng.standard_normal((7, 32))
    dx, dg, db = O.layernorm_bwd(da, x, mu, rstd, ones)
    assert np.abs(dx.sum(1)).max() < 1e-13
    # sum_j dx_j xhat_j = rstd * sum_j(u_j xhat_j) * eps / (var + eps): zero up to eps
    want = rstd * (da * a).sum(1) * 1e-5 / (var + 1e-5)
    assert np.abs((dx * a).sum(1) - want).max() < 1e-13
    assert np.allclose(db, da.sum(0))
    assert np.allclose(dg, (da * a).sum(0))


def test_gelu_identities():
    h = np.linspace(-6, 6, 101)
    assert O.gelu_tanh(np.array([0.0]))[0] == 0.0
    assert O.gelu_tanh_grad(np.array([0.0]))[0] == 0.5
    assert np.allclose(O.gelu_tanh(h) - O.gelu_tanh(-h), h, atol=1e-15)
    assert np.allclose(O.gelu_tanh_grad(h) + O.gelu_tanh_grad(-h), 1.0, atol=1e-15)
    # against the exact erf GELU: the tanh form is within 5e-4 everywhere
    erf = np.array([0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in h])
    assert np.abs(O.gelu_tanh(h) - erf).max() < 5e-4
    # library cross-check of value and slope
    th = torch.tensor(h, dtype=torch.float64, requires_grad=True)
    tg = torch.nn.functional.gelu(th, approximate="tanh")
    tg.sum().backward()
    assert np.allclose(O.gelu_tanh(h), tg.detach().numpy(), atol=1e-15)
    assert np.allclose(O.gelu_tanh_grad(h), th.grad.numpy(), atol=1e-14)


def test_block_special_cases():
    rng = np.random.default_rng(20)
    p = rand_block_params(rng)
    for k in ("w_o", "w_fc2", "b_o", "b_fc2"):
        p[k] = np.zeros_like(p[k])
    x = rng.standard_normal((B * T, D))
    dy = rng.standard_normal((B * T, D))
    y, s = O.block_forward(x, p, B, T, H, HD)
    assert np.array_equal(y, x)
    dx, gr, _ = O.block_backward(dy, s, p, B, T, H, HD)
    assert np.array_equal(dx, dy)
    assert np.allclose(gr["b_fc2"], dy.sum(0))
    # batch elements are independent
    p = rand_block_params(rng)
    y, _ = O.block_forward(x, p, B, T, H, HD)
    xs = x.reshape(B, T, D)[::-1].reshape(B * T, D)
    ys, _ = O.block_forward(xs, p, B, T, H, HD)
    assert np.allclose(ys.reshape(B, T, D)[::-1], y.reshape(B, T, D), atol=1e-14)


def test_cross_entropy_uniform_logits_is_log_vocab():
    v, n = 50304, 6
    tg = np.arange(n) * 7
    loss, dl = O.cross_entropy(np.zeros((n, v)), tg)
    assert abs(loss - math.log(v)) < 1e-12
    assert abs(loss - 10.825840) < 1e-6
    assert np.abs(dl.sum(1)).max() < 1e-15
    want = np.full((n, v), 1.0 / v / n)
    want[np.arange(n), tg] -= 1.0 / n
    assert np.allclose(dl, want, atol=1e-18)


def test_lm_zero_wte_gives_log_vocab():
    rng = np.random.default_rng(21)
    lm = rand_lm(rng)
    lm["wte"] = np.zeros_like(lm["wte"])
    ids = rng.integers(0, V, (B, T))
    loss, _ = O.lm_forward_backward(ids, ids, lm, B, T, H, HD)
    assert abs(loss - math.log(V)) < 1e-13


def test_adamw_closed_forms():
    rng = np.random.default_rng(22)
    w = rng.standard_normal(100)
    g = rng.standard_normal(100)
    g[:5] = [0.0, 1e-9, -1e-9, 1e-8, -3e-8]
    lr, b1, b2, eps, wd = 1e-3, 0.9, 0.95, 1e-8, 0.1
    z = np.zeros(100)
    w1, m1, v1 = O.adamw(w, z, z, g, lr, b1, b2, eps, wd, 1)
    assert np.allclose(w1, w * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=0, atol=1e-15)
    assert np.allclose(m1, (1 - b1) * g, atol=1e-18) and np.allclose(v1, (1 - b2) * g * g, atol=1e-18)
    # zero gradient: pure decay
    w1, _, _ = O.adamw(w, z, z, z, lr, b1, b2, eps, wd, 1)
    assert np.allclose(w1, w * (1 - lr * wd), atol=1e-16)
    # constant gradient, no decay: n equal steps
    ww, mm, vv = w.copy(), z, z
    for t in range(1, 8):
        ww, mm, vv = O.adamw(ww, mm, vv, g, lr, b1, b2, eps, 0.0, t)
    assert np.allclose(ww, w - 7 * lr * g / (np.abs(g) + eps), atol=1e-12)
    # library cross-check with warm state
    tw = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([tw], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    ww, mm, vv = w.copy(), z, z
    for t in range(1, 4):
        gt = rng.standard_normal(100)
        tw.grad = torch.tensor(gt)
        opt.step()
        ww, mm, vv = O.adamw(ww, mm, vv, gt, lr, b1, b2, eps, wd, t)
    assert np.allclose(ww, tw.detach().numpy(), rtol=0, atol=1e-13)


def test_planted_mistakes_are_caught():
    """A dropped term in a copy of the LayerNorm backward must fail the
    finite-difference pin (guards the pin, not the oracle)."""
    rng = np.random.default_rng(23)
    x = rng.standard_normal((3, 8))
    g = 1 + 0.2 * rng.standard_normal(8)
    da = rng.standard_normal((3, 8))

    def probe():
        return float((O.layernorm_fwd(x, g, np.zeros(8), 1e-5)[0] * da).sum())

    a, mu, rstd = O.layernorm_fwd(x, g, np.zeros(8), 1e-5)
    dx, _, _ = O.layernorm_bwd(da, x, mu, rstd, g)
    _fd_check(probe, x, dx)
    bad = rstd[:, None] * (da * g - (da * g).mean(1, keepdims=True))     # missing xhat term
    with pytest.raises(AssertionError):
        _fd_check(probe, x, bad)


def test_paper_numbers_golden():
    from paper_2204_06514_b200 import synth
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_numbers.txt")
    vals = {}
    for line in open(path):
        line = line.split("#")[0].split()
        if len(line) == 2:
            vals[line[0]] = float(line[1])
    assert round(6.7e9 * 4 / 2 ** 30) == vals["params_6p7b_fp32_gib"]
    c4 = synth.CONFIGS["C4"]
    assert c4.n_params == 124_475_904
    assert c4.n_params // 10 ** 6 == vals["fig3_model_params_millions"]
    f3 = synth.CONFIGS["F3"]                 # Fig. 3's workload: the same 124M model at the caption's sequence length
    assert f3.seq == vals["fig3_seq_len"] and f3.n_params - c4.n_params == (f3.seq - c4.seq) * f3.d_model
    c5 = synth.CONFIGS["C5"]
    assert c5.seq == vals["table1_seq_len"] and c5.batch == vals["table1_batch"]
