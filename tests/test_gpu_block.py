"""GPU parity of the block and LM entry points against the fp64 oracle."""
import numpy as np
import pytest
import torch

from parity_util import *  # noqa: F401,F403

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    s.close()


def run_block_case(sess, cfg, prec, params, check_update=True):
    x, dy = synth.block_inputs(cfg)
    if prec == fx.FAX_PREC_FP32_VALIDATE:       # un-rounded inputs in validation mode
        x = synth.normal(cfg.seed, synth.TID_X, x.shape)
        dy = synth.normal(cfg.seed, synth.TID_DY, dy.shape)
    pc = compute_params(params, prec)
    B, T, H, hd = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim
    ry, saved = O.block_forward(x, pc, B, T, H, hd, cfg.ln_eps)
    rdx, rg, _ = O.block_backward(dy, saved, pc, B, T, H, hd)
    r = BlockRunner(sess, cfg, params, prec)
    tx, tdy = r.to_device(x), r.to_device(dy)
    tol_f = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    tol_g = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    y = host(r.forward(tx))
    assert relerr(y, ry) <= tol_f, "y"
    dx = host(r.backward(tdy))
    assert relerr(dx, rdx) <= tol_g, "dx"
    grads = {k: host(r.p[k].g).reshape(rg[k].shape) for k in O.PARAM_NAMES}
    for k in O.PARAM_NAMES:
        assert relerr(grads[k], rg[k]) <= tol_g, k
    # accumulate = 1 adds a second copy
    r.backward(tdy, accumulate=True)
    for k in ("w_fc1", "b_qkv", "ln1_g"):
        assert relerr(host(r.p[k].g).reshape(rg[k].shape), 2 * rg[k]) <= tol_g, k + " (accumulate)"
    if not check_update:
        return
    # fresh state, whole step through fax_block_step
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    r2 = BlockRunner(sess, cfg, params, prec, weight_decay=wd)
    r2.step(tx, tdy, hparams(step=1, **hp))
    assert relerr(host(r2.y), ry) <= tol_f and relerr(host(r2.dx), rdx) <= tol_g
    for k in O.PARAM_NAMES:
        g_gpu = host(r2.p[k].g).reshape(rg[k].shape)
        w_gpu = host(r2.p[k].w).reshape(rg[k].shape)
        w0 = params[k].astype(np.float64)
        # composition: the oracle's AdamW applied to the GPU's own gradients
        cw, cm, cv = O.adamw(w0, 0 * w0, 0 * w0, g_gpu, weight_decay=wd, step=1, **hp)
        assert relerr(w_gpu, cw) <= TOL_ADAMW, k
        assert relerr(host(r2.p[k].m).reshape(w0.shape), cm) <= TOL_ADAMW, k
        # direct: oracle gradients all the way, sign-ambiguous elements bounded separately
        rw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, rg[k], weight_decay=wd, step=1, **hp)
        check_adamw_update(k, w_gpu, w0, rg[k], rw, hp["lr"], wd, tol_g, tol_g)
        if prec == 0:
            assert torch.equal(r2.p[k].wc, r2.p[k].w.to(torch.bfloat16)), k
    # warm state at t = 10: the update is Lipschitz in g, plain bound on every tensor
    r3 = BlockRunner(sess, cfg, params, prec, weight_decay=wd)
    ref_state = {}
    for i, k in enumerate(O.PARAM_NAMES):
        gs = max(np.abs(rg[k]).max(), 1e-12)
        m0, v0 = synth.warm_state(cfg.seed, i, params[k].shape, gs)
        r3.p[k].m.copy_(torch.as_tensor(m0)); r3.p[k].v.copy_(torch.as_tensor(v0))
        ref_state[k] = (m0, v0)
    r3.step(tx, tdy, hparams(step=10, **hp))
    for k in O.PARAM_NAMES:
        m0, v0 = ref_state[k]
        w0 = params[k].astype(np.float64)
        rw, _, _ = O.adamw(w0, m0, v0, rg[k], weight_decay=wd, step=10, **hp)
        # compare the step taken, relative to the largest step
        step_ref = rw - w0
        step_gpu = host(r3.p[k].w).reshape(w0.shape) - w0
        assert np.abs(step_gpu - step_ref).max() <= tol_g * max(np.abs(step_ref).max(), 1e-30) + 1e-7, k
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK


def test_block_fp32_validate_tiny_ragged(sess):
    cfg = synth.Config("tiny", 7, batch=2, seq=5, d_model=8, n_heads=2, head_dim=4, d_ff=16)
    run_block_case(sess, cfg, fx.FAX_PREC_FP32_VALIDATE, perturbed_block_params(cfg))
    cfg = synth.Config("odd", 8, batch=3, seq=37, d_model=96, n_heads=3, head_dim=32, d_ff=200)
    run_block_case(sess, cfg, fx.FAX_PREC_FP32_VALIDATE, perturbed_block_params(cfg))


def test_block_fp32_validate_c1(sess):
    cfg = synth.CONFIGS["C1"]
    run_block_case(sess, cfg, fx.FAX_PREC_FP32_VALIDATE, synth.block_params(cfg))


def test_block_bf16_c1(sess):
    cfg = synth.CONFIGS["C1"]
    run_block_case(sess, cfg, fx.FAX_PREC_BF16, synth.block_params(cfg))
    run_block_case(sess, cfg, fx.FAX_PREC_BF16, perturbed_block_params(cfg), check_update=False)


def test_block_bf16_c2(sess):
    cfg = synth.CONFIGS["C2"]
    run_block_case(sess, cfg, fx.FAX_PREC_BF16, synth.block_params(cfg))


def test_block_bf16_c3_width_reduced_tokens(sess):
    # C3's widths (d 4096, 32 heads x 128, FFN 16384) on one 384-token sequence and
    # a ragged 3 x 128 batch: spans many tiles, finishes in seconds on the CPU side
    cfg = synth.scaled(synth.CONFIGS["C3"], batch=3, seq=128)
    run_block_case(sess, cfg, fx.FAX_PREC_BF16, perturbed_block_params(cfg), check_update=False)


def test_block_causal_invariance_on_gpu(sess):
    cfg = synth.CONFIGS["C1"]
    params = synth.block_params(cfg)
    x, _ = synth.block_inputs(cfg)
    r = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16)
    y0 = r.forward(r.to_device(x)).clone()
    t = 70
    x2 = x.reshape(cfg.batch, cfg.seq, -1).copy()
    x2[:, t + 1:] = synth.round_to_bf16(5 * np.random.default_rng(0).standard_normal(x2[:, t + 1:].shape).astype(np.float32))
    y1 = r.forward(r.to_device(x2.reshape(x.shape)))
    a = y0.view(cfg.batch, cfg.seq, -1)[:, :t + 1]
    b = y1.view(cfg.batch, cfg.seq, -1)[:, :t + 1]
    assert torch.equal(a, b)


def test_block_step_host_matches_device_step(sess):
    """The host-buffer entry point (copies inside, on its own copy stream) gives bit-identical results."""
    for name in ("C1", "C2"):
        cfg = synth.CONFIGS[name]
        params = synth.block_params(cfg)
        x, dy = synth.block_inputs(cfg)
        hp = dict(synth.ADAMW)
        wd = hp.pop("weight_decay")
        a = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
        b = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd, host_io=True)
        tx, tdy = a.to_device(x), a.to_device(dy)
        xh, dyh = tx.cpu().pin_memory(), tdy.cpu().pin_memory()
        yh, dxh = torch.empty_like(xh).pin_memory(), torch.empty_like(xh).pin_memory()
        for step in (1, 2):
            a.step(tx, tdy, hparams(step=step, **hp))
            b.step_host(xh, dyh, yh, dxh, hparams(step=step, **hp))
            torch.cuda.synchronize()
            if step == 1:
                assert torch.equal(a.y.cpu(), yh)            # same weights, same kernels: identical forward
            # backward adds dQ tiles and split-K partial tiles in arrival order (float32), so
            # gradients agree to rounding, not bit for bit
            # (from the second step on the two runs' weights differ by first-step sign choices)
            tol = 5e-3 if step == 1 else TOL_GRAD_BF16
            assert relerr(host(dxh), host(a.dx)) <= tol
            for k in O.PARAM_NAMES:
                assert relerr(host(b.p[k].g), host(a.p[k].g)) <= tol, k
            if step == 2:
                assert relerr(host(yh), host(a.y)) <= TOL_FWD_BF16


def test_dependent_launch_switch_leaves_results_unchanged(sess):
    """Kernels launched with programmatic dependent launch wait for their predecessor before they
    touch global memory, so a step gives the same forward bits and the same gradients (to the
    rounding of the arrival-order adds) as with every launch fully serialised; repeated steps go
    through the captured graph as well."""
    cfg = synth.CONFIGS["C2"]
    params = synth.block_params(cfg)
    x, dy = synth.block_inputs(cfg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    runs = {}
    try:
        for on in (True, False):
            fx.fax_set_dependent_launch(sess.ctx, on)
            r = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
            tx, tdy = r.to_device(x), r.to_device(dy)
            ys = []
            for step in (1, 2, 3, 4):
                r.step(tx, tdy, hparams(step=step, **hp))
                torch.cuda.synchronize()
                ys.append(r.y.clone())
            runs[on] = (ys, r.dx.clone(), {k: r.p[k].g.clone() for k in O.PARAM_NAMES})
    finally:
        fx.fax_set_dependent_launch(sess.ctx, True)
    assert torch.equal(runs[True][0][0], runs[False][0][0])          # first forward: identical weights
    for a, b in zip(runs[True][0][1:], runs[False][0][1:]):
        assert relerr(host(a), host(b)) <= TOL_FWD_BF16
    assert relerr(host(runs[True][1]), host(runs[False][1])) <= TOL_GRAD_BF16
    for k in O.PARAM_NAMES:
        assert relerr(host(runs[True][2][k]), host(runs[False][2][k])) <= TOL_GRAD_BF16, k
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK


def test_graph_replay_patches_the_adamw_scalars(sess):
    """From the third call on a whole step is a replayed CUDA graph; the only arguments that change
    are AdamW's scalars.  A step with lr = 0 must leave every weight exactly as it was."""
    cfg = synth.CONFIGS["C1"]
    params = synth.block_params(cfg)
    x, dy = synth.block_inputs(cfg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    a = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
    tx, tdy = a.to_device(x), a.to_device(dy)
    l0 = sess.launches()
    a.step(tx, tdy, hparams(step=1, **hp))                 # as is
    per_step = sess.launches() - l0
    a.step(tx, tdy, hparams(step=2, **hp))                 # captured
    torch.cuda.synchronize()
    w2 = {k: a.p[k].w.clone() for k in O.PARAM_NAMES}
    m2 = a.p["w_fc1"].m.clone()
    frozen = dict(hp, lr=0.0)
    a.step(tx, tdy, hparams(step=3, **frozen))             # replayed, lr = 0
    torch.cuda.synchronize()
    assert sess.launches() - l0 == 3 * per_step
    for k in O.PARAM_NAMES:
        assert torch.equal(a.p[k].w, w2[k]), k
    assert not torch.equal(a.p["w_fc1"].m, m2)             # the step did run
    a.step(tx, tdy, hparams(step=4, **hp))                 # replayed, lr back
    torch.cuda.synchronize()
    assert not torch.equal(a.p["w_fc1"].w, w2["w_fc1"])
    # and the replayed forward equals a run without graphs on the same weights
    fx.fax_set_graph_replay(sess.ctx, False)
    y_graph = a.y.clone()
    b = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
    for k in O.PARAM_NAMES:
        b.p[k].w.copy_(w2[k]); b.p[k].wc.copy_(w2[k].to(torch.bfloat16))
    # step 4 ran on the weights of step 2/3 (lr = 0 in between): same forward
    b.forward(tx)
    torch.cuda.synchronize()
    fx.fax_set_graph_replay(sess.ctx, True)
    assert torch.equal(b.y, y_graph)
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


@pytest.mark.parametrize("name", ["C1", "C2"])
def test_fused_update_matches_separate_update(sess, name):
    """AdamW in the epilogue of the weight-gradient GEMMs gives the weights of the separate update."""
    cfg = synth.CONFIGS[name]
    params = perturbed_block_params(cfg)
    x, dy = synth.block_inputs(cfg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    mats = ("w_qkv", "w_o", "w_fc1", "w_fc2")
    try:
        runs = {}
        for mode in ("separate", "fused_keep", "fused"):
            fx.fax_set_fused_update(sess.ctx, mode != "separate", mode == "fused_keep")
            r = BlockRunner(sess, cfg, params, fx.FAX_PREC_BF16, weight_decay=wd)
            tx, tdy = r.to_device(x), r.to_device(dy)
            r.step(tx, tdy, hparams(step=1, **hp))
            torch.cuda.synchronize()
            runs[mode] = r
        a, b, c = runs["separate"], runs["fused_keep"], runs["fused"]
        for k in O.PARAM_NAMES:
            ga = host(a.p[k].g)
            assert relerr(host(b.p[k].g), ga) <= 1e-3, k                 # gradients kept
            if k in mats and name == "C1":                               # (C2's narrow shapes slice K: not fused)
                assert float(c.p[k].g.abs().max()) == 0.0, k             # not materialised
            # the update itself: oracle AdamW on this run's own gradient
            w0 = params[k].astype(np.float64)
            gb = host(b.p[k].g).reshape(w0.shape)
            cw, cm, cv = O.adamw(w0, 0 * w0, 0 * w0, gb, weight_decay=wd, step=1, **hp)
            assert relerr(host(b.p[k].w).reshape(w0.shape), cw) <= TOL_ADAMW, k
            assert relerr(host(b.p[k].m).reshape(w0.shape), cm) <= TOL_ADAMW, k
            assert relerr(host(b.p[k].v).reshape(w0.shape), cv) <= 1e-5, k
            assert torch.equal(b.p[k].wc, b.p[k].w.to(torch.bfloat16)), k
            assert torch.equal(c.p[k].wc, c.p[k].w.to(torch.bfloat16)), k
            # moments are linear / quadratic in the gradient: all three runs agree
            assert relerr(host(c.p[k].m), host(a.p[k].m)) <= 1e-3, k
        # graph replay patches the scalars inside the fused GEMMs too: a step with lr = 0 freezes the weights
        c.step(c.to_device(x), c.to_device(dy), hparams(step=2, **hp))
        torch.cuda.synchronize()
        w2 = {k: c.p[k].w.clone() for k in O.PARAM_NAMES}
        c.step(c.to_device(x), c.to_device(dy), hparams(step=3, **dict(hp, lr=0.0)))
        torch.cuda.synchronize()
        for k in O.PARAM_NAMES:
            assert torch.equal(c.p[k].w, w2[k]), k
    finally:
        fx.fax_set_fused_update(sess.ctx, False, False)
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def test_block_error_paths(sess):
    cfg = synth.CONFIGS["C1"]
    r = BlockRunner(sess, cfg, synth.block_params(cfg), fx.FAX_PREC_BF16)
    x = r.to_device(synth.block_inputs(cfg)[0])
    with pytest.raises(fx.FaxError) as e:
        fx.fax_block_forward(sess.ctx, r.bcfg, r.params_struct, ptr(x), ptr(r.y), ptr(r.saved), 1024,
                             ptr(r.scratch), r.scratch_bytes)
    assert e.value.status == fx.FAX_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(fx.FaxError) as e:
        fx.fax_block_forward(sess.ctx, r.bcfg, r.params_struct, ptr(x), ptr(x), ptr(r.saved), r.saved_bytes,
                             ptr(r.scratch), r.scratch_bytes)
    assert e.value.status == fx.FAX_ERR_INVALID_ARG


def lm_case(sess, cfg, prec, lm, head_rows=0):
    ids, tg = synth.lm_tokens(cfg)
    B, T, H, hd = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim
    rnd = (lambda a: synth.round_to_bf16(a).astype(np.float64)) if prec == 0 else (lambda a: a.astype(np.float64))
    lmc = dict(wte=rnd(lm["wte"]), wpe=rnd(lm["wpe"]), lnf_g=rnd(lm["lnf_g"]), lnf_b=rnd(lm["lnf_b"]),
               blocks=[{k: rnd(v) for k, v in p.items()} for p in lm["blocks"]])
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    zeros = {n: np.zeros_like(a, dtype=np.float64) for n, a in O.lm_tensors(lm)}
    rloss, rg, rw, rm, rv = O.lm_step(ids, tg, lmc, zeros, zeros, B, T, H, hd,
                                      dict(weight_decay=wd, step=1, **hp), cfg.ln_eps, lm_master=lm)
    r = LmRunner(sess, cfg, lm, prec, weight_decay=wd, head_rows=head_rows)
    tids = torch.as_tensor(ids).to(sess.device)
    ttg = torch.as_tensor(tg).to(sess.device)
    tol_f = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    tol_g = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    r.forward_backward(tids, ttg)
    loss = float(r.loss.item())
    assert abs(loss - rloss) <= tol_f * abs(rloss)
    for name, ps in r.named_params():
        assert relerr(host(ps.g).reshape(rg[name].shape), rg[name]) <= tol_g, name
    # full step on fresh state, host loss readback
    r2 = LmRunner(sess, cfg, lm, prec, weight_decay=wd, head_rows=head_rows)
    l2 = r2.step(tids, ttg, hparams(step=1, **hp), want_host_loss=True)
    assert abs(l2 - rloss) <= tol_f * abs(rloss)
    for name, ps in r2.named_params():
        w0 = dict(O.lm_tensors(lm))[name].astype(np.float64)
        g_gpu = host(ps.g).reshape(w0.shape)
        cw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, g_gpu, weight_decay=wd, step=1, **hp)
        assert relerr(host(ps.w).reshape(w0.shape), cw) <= TOL_ADAMW, name
        check_adamw_update(name, host(ps.w).reshape(w0.shape), w0, rg[name], rw[name], hp["lr"], wd, tol_g, tol_g)
    # host-buffer entry point gives the same loss
    r3 = LmRunner(sess, cfg, lm, prec, weight_decay=wd, head_rows=head_rows)
    l3 = r3.step_host(torch.as_tensor(ids).pin_memory(), torch.as_tensor(tg).pin_memory(), hparams(step=1, **hp))
    assert l3 == l2
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK


def test_lm_fp32_validate_tiny(sess):
    cfg = synth.Config("lm_tiny", 9, batch=2, seq=5, d_model=8, n_heads=2, head_dim=4, d_ff=16, n_layers=2, vocab=11)
    lm = synth.lm_params(cfg)
    for l in range(cfg.n_layers):
        lm["blocks"][l] = perturbed_block_params(cfg, l)
    lm["wte"] *= 10; lm["wpe"] *= 10
    ids, _ = synth.lm_tokens(cfg)
    lm_case(sess, cfg, fx.FAX_PREC_FP32_VALIDATE, lm)


def test_lm_bf16_c4_shape_reduced(sess):
    # C4's widths and full vocabulary (d 768, 12 x 64, FFN 3072, V 50304), 2 layers, 2 x 128 tokens
    cfg = synth.scaled(synth.CONFIGS["C4"], batch=2, seq=128, n_layers=2)
    lm_case(sess, cfg, fx.FAX_PREC_BF16, synth.lm_params(cfg))


@pytest.mark.parametrize("prec", [fx.FAX_PREC_FP32_VALIDATE, fx.FAX_PREC_BF16])
def test_lm_head_in_row_chunks(sess, prec):
    # 3 x 128 tokens with 256 logits rows at a time: a full chunk and a shorter last one, the
    # gradient of the tied embedding accumulated over both (the path batches above ~42k tokens take)
    cfg = synth.Config("lm_chunks", 11, batch=3, seq=128, d_model=256, n_heads=4, head_dim=64, d_ff=1024, n_layers=1,
                       vocab=1024)
    lm_case(sess, cfg, prec, synth.lm_params(cfg), head_rows=256)


def test_lm_three_steps_and_resume_fp32(sess):
    """Three consecutive LM steps in the float32 validation mode follow the oracle's trajectory (loss,
    weights, moments), and a run resumed from copied-out state (w, m, v, step) continues identically."""
    cfg = synth.Config("lm_multi", 10, batch=2, seq=6, d_model=16, n_heads=2, head_dim=8, d_ff=32, n_layers=2, vocab=13)
    lm = synth.lm_params(cfg)
    for l in range(cfg.n_layers):
        lm["blocks"][l] = perturbed_block_params(cfg, l)
    lm["wte"] *= 10; lm["wpe"] *= 10
    ids, tg = synth.lm_tokens(cfg)
    B, T, H, hd = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    names = [n for n, _ in O.lm_tensors(lm)]
    # warm optimizer state keeps the update smooth in the gradient (no first-step sign function)
    m0 = {n: synth.warm_state(cfg.seed, i, a.shape, 1e-2)[0] for i, (n, a) in enumerate(O.lm_tensors(lm))}
    v0 = {n: synth.warm_state(cfg.seed, i, a.shape, 1e-2)[1] for i, (n, a) in enumerate(O.lm_tensors(lm))}

    def unflatten(flat):
        return dict(wte=flat["wte"], wpe=flat["wpe"], lnf_g=flat["lnf_g"], lnf_b=flat["lnf_b"],
                    blocks=[{k: flat[f"blocks.{l}.{k}"] for k in O.PARAM_NAMES} for l in range(cfg.n_layers)])

    def set_state(r, w, m, v):
        for n, ps in r.named_params():
            ps.w.copy_(torch.as_tensor(np.asarray(w[n], dtype=np.float32)))
            ps.m.copy_(torch.as_tensor(np.asarray(m[n], dtype=np.float32)))
            ps.v.copy_(torch.as_tensor(np.asarray(v[n], dtype=np.float32)))

    w = {n: a.astype(np.float64) for n, a in O.lm_tensors(lm)}
    m, v = dict(m0), dict(v0)
    r = LmRunner(sess, cfg, lm, fx.FAX_PREC_FP32_VALIDATE, weight_decay=wd)
    set_state(r, w, m, v)
    tids, ttg = torch.as_tensor(ids).to(sess.device), torch.as_tensor(tg).to(sess.device)
    snap = None
    for step in (5, 6, 7):
        loss_ref, _, w, m, v = O.lm_step(ids, tg, unflatten(w), m, v, B, T, H, hd,
                                         dict(weight_decay=wd, step=step, **hp), cfg.ln_eps)
        loss = r.step(tids, ttg, hparams(step=step, **hp), want_host_loss=True)
        assert abs(loss - loss_ref) <= TOL_FP32 * abs(loss_ref), step
        for n, ps in r.named_params():
            assert relerr(host(ps.w).reshape(w[n].shape), w[n]) <= TOL_FP32, (step, n)
            assert relerr(host(ps.m).reshape(w[n].shape), m[n]) <= TOL_FP32, (step, n)
        if step == 6:
            snap = {n: (ps.w.clone(), ps.m.clone(), ps.v.clone()) for n, ps in r.named_params()}
    # resume: a fresh runner given the state after step 6 reproduces step 7 bit for bit
    r2 = LmRunner(sess, cfg, lm, fx.FAX_PREC_FP32_VALIDATE, weight_decay=wd)
    for n, ps in r2.named_params():
        ps.w.copy_(snap[n][0]); ps.m.copy_(snap[n][1]); ps.v.copy_(snap[n][2])
    loss2 = r2.step(tids, ttg, hparams(step=7, **hp), want_host_loss=True)
    assert loss2 == loss
    for (n, a), (_, b) in zip(r.named_params(), r2.named_params()):
        if n == "wte":        # its gradient includes the embedding scatter: float atomics, arrival order
            assert relerr(host(b.w), host(a.w)) <= 1e-6
        else:
            assert torch.equal(a.w, b.w), n


def test_lm_and_adamw_error_paths(sess):
    cfg = synth.Config("lm_err", 11, batch=2, seq=128, d_model=128, n_heads=2, head_dim=64, d_ff=256, n_layers=1, vocab=256)
    lm = synth.lm_params(cfg)
    r = LmRunner(sess, cfg, lm, fx.FAX_PREC_BF16)
    ids, tg = synth.lm_tokens(cfg)
    tids, ttg = torch.as_tensor(ids).to(sess.device), torch.as_tensor(tg).to(sess.device)
    hp = dict(synth.ADAMW); hp.pop("weight_decay")
    # step < 1
    with pytest.raises(fx.FaxError) as e:
        r.step(tids, ttg, hparams(step=0, **hp))
    assert e.value.status == fx.FAX_ERR_INVALID_ARG
    # scratch arena too small
    import ctypes as C
    small = fx.LmState.from_buffer_copy(r.state)
    small.scratch_bytes = 1024
    with pytest.raises(fx.FaxError) as e:
        fx.fax_lm_forward_backward(sess.ctx, r.lcfg, small, ptr(tids), ptr(ttg), ptr(r.loss))
    assert e.value.status == fx.FAX_ERR_WORKSPACE_TOO_SMALL
    # vocabulary that the bf16 tiles do not divide
    bad = fx.LmCfg(1, 250, 128, r.lcfg.block)
    with pytest.raises(fx.FaxError) as e:
        fx.fax_lm_sizes(bad)
    assert e.value.status == fx.FAX_ERR_UNSUPPORTED_SHAPE
    # AdamW: misaligned pointer, bad beta
    w = torch.zeros(1024, device=sess.device)
    t = fx.AdamwTensor(C.c_void_p(w.data_ptr() + 4), ptr(w), ptr(w), ptr(w), None, 8, 0.0)
    with pytest.raises(fx.FaxError) as e:
        fx.fax_adamw_step(sess.ctx, [t], hparams(step=1, **hp))
    assert e.value.status == fx.FAX_ERR_INVALID_ARG
    t = fx.AdamwTensor(ptr(w), ptr(w), ptr(w), ptr(w), None, 8, 0.0)
    with pytest.raises(fx.FaxError):
        fx.fax_adamw_step(sess.ctx, [t], hparams(step=1, **dict(hp, beta1=1.0)))
    # the context is still usable afterwards
    r.step(tids, ttg, hparams(step=1, **hp))
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK and torch.isfinite(r.loss).all()
    # once the step is replayed from a graph (third call on) bad hyper-parameters are still refused,
    # before anything is enqueued: the weights stay as they are and finite
    for s in (2, 3, 4):
        r.step(tids, ttg, hparams(step=s, **hp))
    torch.cuda.synchronize()
    before = r.wte.w.clone()
    for bad_hp in (dict(hp, beta1=1.0), dict(hp, beta2=-0.1), dict(hp, lr=float("nan")), dict(hp, eps=float("inf"))):
        with pytest.raises(fx.FaxError) as e:
            r.step(tids, ttg, hparams(step=5, **bad_hp))
        assert e.value.status == fx.FAX_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.equal(before, r.wte.w) and torch.isfinite(r.wte.w).all()
    r.step(tids, ttg, hparams(step=5, **hp))
    torch.cuda.synchronize()
    assert torch.isfinite(r.wte.w).all() and not torch.equal(before, r.wte.w)


@pytest.mark.parametrize("prec", [fx.FAX_PREC_FP32_VALIDATE, fx.FAX_PREC_BF16])
def test_lm_gradient_accumulation_equals_the_big_batch(sess, prec):
    """Two micro-batches accumulated with grad_scale 1/2, then fax_lm_apply_adamw == one step on the whole batch."""
    if prec == fx.FAX_PREC_BF16:
        big = synth.Config("lm_acc", 12, batch=4, seq=128, d_model=128, n_heads=2, head_dim=64, d_ff=256, n_layers=2, vocab=256)
    else:
        big = synth.Config("lm_acc32", 13, batch=4, seq=6, d_model=16, n_heads=2, head_dim=8, d_ff=32, n_layers=2, vocab=13)
    half = synth.scaled(big, batch=2)
    lm = synth.lm_params(big)
    ids, tg = synth.lm_tokens(big)
    B, T, H, hd = big.batch, big.seq, big.n_heads, big.head_dim
    rnd = (lambda a: synth.round_to_bf16(a).astype(np.float64)) if prec == 0 else (lambda a: a.astype(np.float64))
    lmc = dict(wte=rnd(lm["wte"]), wpe=rnd(lm["wpe"]), lnf_g=rnd(lm["lnf_g"]), lnf_b=rnd(lm["lnf_b"]),
               blocks=[{k: rnd(v) for k, v in p.items()} for p in lm["blocks"]])
    rloss, rg = O.lm_forward_backward(ids, tg, lmc, B, T, H, hd, big.ln_eps)
    rg = dict(O.lm_tensors(rg))
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    r = LmRunner(sess, half, lm, prec, weight_decay=wd)
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a)).to(sess.device)
    r.accumulate(dev(ids[:2]), dev(tg[:2]), False, 0.5)
    l0 = float(r.loss.item())
    r.accumulate(dev(ids[2:]), dev(tg[2:]), True, 0.5)
    l1 = float(r.loss.item())
    tol_f = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    tol_g = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    assert abs(0.5 * (l0 + l1) - rloss) <= tol_f * abs(rloss)
    for name, ps in r.named_params():
        assert relerr(host(ps.g).reshape(rg[name].shape), rg[name]) <= tol_g, name
    grads = {n: host(ps.g) for n, ps in r.named_params()}
    r.apply_adamw(hparams(step=1, **hp))
    for (name, ps), (_, w0) in zip(r.named_params(), O.lm_tensors(lm)):
        w0 = w0.astype(np.float64)
        cw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, grads[name].reshape(w0.shape), weight_decay=wd, step=1, **hp)
        assert relerr(host(ps.w).reshape(w0.shape), cw) <= TOL_ADAMW, name
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


@pytest.mark.parametrize("prec,cfg_name", [(fx.FAX_PREC_FP32_VALIDATE, "C1"), (fx.FAX_PREC_BF16, "C1"), (fx.FAX_PREC_BF16, "C2")])
def test_block_activation_recompute(sess, prec, cfg_name):
    """recompute=1: a smaller saved arena, the same y, dx and gradients (bitwise where the kernels are deterministic)."""
    cfg = synth.CONFIGS[cfg_name]
    params = synth.block_params(cfg)
    x, dy = synth.block_inputs(cfg)
    keep = BlockRunner(sess, cfg, params, prec)
    rec = BlockRunner(sess, cfg, params, prec, recompute=True)
    n, d, f = cfg.tokens, cfg.d_model, cfg.d_ff
    es = 2 if prec == fx.FAX_PREC_BF16 else 4
    assert keep.saved_bytes - rec.saved_bytes >= n * (2 * d + f) * es
    assert rec.scratch_bytes == keep.scratch_bytes
    off_saved, _ = fx.fax_block_arena_layout(rec.bcfg)
    assert {k for k, v in off_saved.items() if v == 2 ** 64 - 1} == {"a", "m", "g"}
    if prec == fx.FAX_PREC_FP32_VALIDATE:
        x = synth.normal(cfg.seed, synth.TID_X, x.shape)
        dy = synth.normal(cfg.seed, synth.TID_DY, dy.shape)
    out = {}
    for name, r in (("keep", keep), ("rec", rec)):
        y = host(r.forward(r.to_device(x))).copy()
        dx = host(r.backward(r.to_device(dy))).copy()
        out[name] = (y, dx, {k: host(r.p[k].g).copy() for k in O.PARAM_NAMES})
    assert np.array_equal(out["keep"][0], out["rec"][0])
    tol = TOL_GRAD_BF16 if prec == fx.FAX_PREC_BF16 else TOL_FP32
    # against the oracle, like the plain path
    pc = compute_params(params, prec)
    B, T, H, hd = cfg.batch, cfg.seq, cfg.n_heads, cfg.head_dim
    ry, saved = O.block_forward(x, pc, B, T, H, hd, cfg.ln_eps)
    rdx, rg, _ = O.block_backward(dy, saved, pc, B, T, H, hd)
    assert relerr(out["rec"][1], rdx) <= tol
    for k in O.PARAM_NAMES:
        assert relerr(out["rec"][2][k].reshape(rg[k].shape), rg[k]) <= tol, k
        # deterministic kernels feed these: identical bits with and without recomputation
        if k in ("b_fc2", "b_fc1", "ln2_g", "ln2_b"):
            assert np.array_equal(out["keep"][2][k], out["rec"][2][k]), k
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def test_lm_activation_recompute_step(sess):
    """A whole LM step with recomputation ends on the weights of the plain step (bf16, tiny model)."""
    cfg = synth.Config("lm_rc", 14, batch=2, seq=128, d_model=128, n_heads=2, head_dim=64, d_ff=256, n_layers=3, vocab=256)
    lm = synth.lm_params(cfg)
    ids, tg = synth.lm_tokens(cfg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    dev = lambda a: torch.as_tensor(np.ascontiguousarray(a)).to(sess.device)
    res = {}
    for name, rc in (("keep", False), ("rec", True)):
        r = LmRunner(sess, cfg, lm, fx.FAX_PREC_BF16, weight_decay=wd, recompute=rc)
        r.step(dev(ids), dev(tg), hparams(step=1, **hp))
        res[name] = (float(r.loss.item()), {n: host(ps.w).copy() for n, ps in r.named_params()}, r.saved_bytes)
    assert res["rec"][2] < res["keep"][2]
    assert res["keep"][0] == res["rec"][0]
    for n in res["keep"][1]:
        assert relerr(res["rec"][1][n], res["keep"][1][n]) <= 1e-6, n
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail
