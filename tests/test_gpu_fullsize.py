"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The oracle cannot run a whole full-size step in seconds, so these tests use what the
method's structure makes exact:
  * causality + batch independence: rows [0, T0) of one sequence depend on nothing else,
    so the oracle run on that prefix alone gives the forward outputs of those rows;
  * with dY zero outside that prefix, every gradient (dx and all twelve parameter
    gradients, every element) equals the prefix problem's gradient, and dx is exactly
    zero elsewhere;
  * an LM batch of identical sequences has the loss and the gradients of the
    single-sequence problem.
Only seeded inputs reach the oracle; it never sees a value computed on the GPU."""
import os

import numpy as np
import psutil
import pytest
import torch

from parity_util import *  # noqa: F401,F403

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    s.close()


def block_full_size(sess, cfg, t0, bsel):
    B, T, H, hd, d = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim, cfg.d_model
    params = synth.block_params(cfg)
    x, dy = synth.block_inputs(cfg)
    pc = compute_params(params, fx.FAX_PREC_BF16)
    rows = slice(bsel * T, bsel * T + t0)
    ry, saved = O.block_forward(x[rows], pc, 1, t0, H, hd, cfg.ln_eps)
    rdx, rg, _ = O.block_backward(dy[rows], saved, pc, 1, t0, H, hd)
    del pc
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    r = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
    tx = r.to_device(x)
    # run A: the benchmark's inputs; forward rows of the prefix
    y = host(r.forward(tx)[rows])
    assert relerr(y, ry) <= TOL_FWD_BF16
    # run B: the whole step with dY masked to the prefix
    dym = np.zeros_like(dy)
    dym[rows] = dy[rows]
    r.step(tx, r.to_device(dym), hparams(step=1, **hp))
    dx = host(r.dx)
    assert relerr(dx[rows], rdx) <= TOL_GRAD_BF16
    other = np.ones(dx.shape[0], bool)
    other[rows] = False
    assert np.all(dx[other] == 0.0)
    for k in O.PARAM_NAMES:
        g = host(r.p[k].g).reshape(rg[k].shape)
        assert relerr(g, rg[k]) <= TOL_GRAD_BF16, k
        # the update, composed: oracle AdamW on the GPU's gradient, a leading slice of each tensor
        n = min(g.shape[0], 64)
        w0 = params[k][:n].astype(np.float64)
        cw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, g[:n], weight_decay=wd, step=1, **hp)
        assert relerr(host(r.p[k].w).reshape(rg[k].shape)[:n], cw) <= TOL_ADAMW, k
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def test_c3_full_size(sess):
    block_full_size(sess, synth.CONFIGS["C3"], t0=256, bsel=3)


def test_c2_full_size_other_sequence(sess):
    block_full_size(sess, synth.CONFIGS["C2"], t0=384, bsel=5)


@pytest.mark.skipif(psutil.virtual_memory().total < 150e9, reason="needs ~100 GB of host memory for fp64 copies")
def test_c5_full_size(sess):
    block_full_size(sess, synth.CONFIGS["C5"], t0=128, bsel=0)


# Paper-shaped workloads (Table 1's hidden sizes at batch 1 x seq 2048): same kernels, other tile counts
def test_p1_hidden_5120_full_size(sess):
    block_full_size(sess, synth.CONFIGS["P1"], t0=128, bsel=0)


@pytest.mark.skipif(psutil.virtual_memory().total < 150e9, reason="needs ~80 GB of host memory for fp64 copies")
def test_p2_hidden_10240_full_size(sess):
    block_full_size(sess, synth.CONFIGS["P2"], t0=64, bsel=0)


@pytest.mark.skipif(os.environ.get("FAX_SLOW_TESTS") != "1" or psutil.virtual_memory().total < 180e9,
                    reason="hidden 16384 (3.2e9 parameters): several minutes of host time; set FAX_SLOW_TESTS=1")
def test_p3_hidden_16384_full_size(sess):
    block_full_size(sess, synth.CONFIGS["P3"], t0=32, bsel=0)


def _lm_oracle_inputs(lm):
    rnd = lambda a: synth.round_to_bf16(a).astype(np.float64)
    return dict(wte=rnd(lm["wte"]), wpe=rnd(lm["wpe"]), lnf_g=rnd(lm["lnf_g"]), lnf_b=rnd(lm["lnf_b"]),
                blocks=[{k: rnd(v) for k, v in p.items()} for p in lm["blocks"]])


def test_c4_full_size(sess):
    lm_full_size(sess, synth.CONFIGS["C4"])


def test_f2_350m_class_lm_full_size(sess):
    lm_full_size(sess, synth.CONFIGS["F2"], identical_check=True, t0=64)


def test_f3_124m_batch32_seq2048_full_size(sess):
    # the Fig. 3 workload: per-token losses of sequence prefixes under the benchmark's tokens
    lm_full_size(sess, synth.CONFIGS["F3"], identical_check=False, t0=128)


def lm_full_size(sess, cfg, identical_check=True, t0=128):
    B, T, H, hd = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim
    lm = synth.lm_params(cfg)
    lmc = _lm_oracle_inputs(lm)
    ids, tg = synth.lm_tokens(cfg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    r = LmRunner(sess, cfg, lm, fx.FAX_PREC_BF16, weight_decay=wd)
    lay = fx.fax_lm_arena_layout(r.lcfg)
    # run A: the benchmark's tokens; per-token losses of two sequence prefixes
    r.forward_backward(torch.as_tensor(ids).to(sess.device), torch.as_tensor(tg).to(sess.device))
    torch.cuda.synchronize()
    row_loss = r.scratch[lay["row_loss"]: lay["row_loss"] + 4 * cfg.tokens].view(torch.float32).cpu().numpy()
    for b in (0, B - 1):
        sub = synth.scaled(cfg, batch=1, seq=t0)
        x = lmc["wte"][ids[b, :t0]] + lmc["wpe"][:t0]
        for p in lmc["blocks"]:
            x, _ = O.block_forward(x, p, 1, t0, H, hd, cfg.ln_eps)
        xf, _, _ = O.layernorm_fwd(x, lmc["lnf_g"], lmc["lnf_b"], cfg.ln_eps)
        logits = xf @ lmc["wte"].T
        mx = logits.max(1)
        ref = mx + np.log(np.exp(logits - mx[:, None]).sum(1)) - logits[np.arange(t0), tg[b, :t0]]
        got = row_loss[b * T: b * T + t0]
        assert np.abs(got - ref).max() <= TOL_FWD_BF16 * np.abs(ref).max(), b
    assert abs(float(r.loss.item()) - row_loss.astype(np.float64).mean()) < 1e-4
    if not identical_check:
        return
    del r
    # run B: sixteen copies of one sequence == the single-sequence problem
    ids1, tg1 = ids[:1], tg[:1]
    rloss, rg = O.lm_forward_backward(ids1, tg1, lmc, 1, T, H, hd, cfg.ln_eps)
    rg = dict(O.lm_tensors(rg))
    idsB = torch.as_tensor(np.repeat(ids1, B, axis=0)).to(sess.device)
    tgB = torch.as_tensor(np.repeat(tg1, B, axis=0)).to(sess.device)
    r2 = LmRunner(sess, cfg, lm, fx.FAX_PREC_BF16, weight_decay=wd)
    loss = r2.step(idsB, tgB, hparams(step=1, **hp), want_host_loss=True)
    assert abs(loss - rloss) <= TOL_FWD_BF16 * abs(rloss)
    w0s = dict(O.lm_tensors(lm))
    # bf16 rounding of the gradient flowing down the stack accumulates with depth (measured: 0.4 % at
    # the top layer, 1.2 - 1.5 % at the bottom of 24 layers, single heavy-tail elements up to 3 %): beyond
    # the 12 layers of the benchmark config the element-wise bound is doubled and the l2 error keeps the
    # stated bound
    deep = cfg.n_layers > 12
    for name, ps in r2.named_params():
        g = host(ps.g).reshape(rg[name].shape)
        assert relerr(g, rg[name]) <= (2 * TOL_GRAD_BF16 if deep else TOL_GRAD_BF16), name
        assert np.linalg.norm(g - rg[name]) <= TOL_GRAD_BF16 * np.linalg.norm(rg[name]), name
        n = min(g.shape[0], 64)
        w0 = w0s[name][:n].astype(np.float64)
        cw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, g[:n], weight_decay=wd, step=1, **hp)
        assert relerr(host(ps.w).reshape(g.shape)[:n], cw) <= TOL_ADAMW, name
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail
