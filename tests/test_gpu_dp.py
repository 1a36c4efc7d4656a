"""Data-parallel LM step on the GPU (include/fax_dp.h).  One GPU is all there is here, so the ranks of a
world of two are run one after the other in this process and the two collectives are done by hand on
their flat buffers (a sum and a slice; a concatenation): everything else -- local forward + loss +
backward on half the batch with the 1 / world scale, the shard map, AdamW on a shard -- is the code the
multi-GPU path runs.  The summed gradients are compared with the oracle on the WHOLE batch."""
import numpy as np
import pytest
import torch

from parity_util import *  # noqa: F401,F403
from paper_2204_06514_b200 import dp

pytestmark = pytest.mark.gpu

CFG = synth.Config("lm_dp", 14, batch=4, seq=128, d_model=128, n_heads=2, head_dim=64, d_ff=256, n_layers=2, vocab=384)


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    s.close()


def _oracle(lm, ids, tg):
    rnd = lambda a: synth.round_to_bf16(a).astype(np.float64)
    lmc = dict(wte=rnd(lm["wte"]), wpe=rnd(lm["wpe"]), lnf_g=rnd(lm["lnf_g"]), lnf_b=rnd(lm["lnf_b"]),
               blocks=[{k: rnd(v) for k, v in p.items()} for p in lm["blocks"]])
    loss, g = O.lm_forward_backward(ids, tg, lmc, CFG.batch, CFG.seq, CFG.n_heads, CFG.head_dim, CFG.ln_eps)
    return loss, dict(O.lm_tensors(g))


@pytest.mark.parametrize("world", [1, 2, 4])
def test_data_parallel_step_equals_the_whole_batch_step(sess, world):
    lm = synth.lm_params(CFG)
    ids, tg = synth.lm_tokens(CFG)
    rloss, rg = _oracle(lm, ids, tg)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    ranks = [dp.DpLmRunner(sess, CFG, lm, weight_decay=wd, rank=r, world=world) for r in range(world)]
    per = CFG.batch // world
    losses = []
    for r, run in enumerate(ranks):
        tid = torch.as_tensor(ids[r * per:(r + 1) * per]).to(sess.device).contiguous()
        ttg = torch.as_tensor(tg[r * per:(r + 1) * per]).to(sess.device).contiguous()
        run.local_gradients(tid, ttg)
        losses.append(float(run.loss.item()))
    assert abs(sum(losses) / world - rloss) <= TOL_FWD_BF16 * abs(rloss)
    # reduce-scatter by hand: the sum of the ranks' flat gradient buffers, each rank keeps its slice
    gsum = torch.zeros_like(ranks[0].g)
    for run in ranks:
        gsum += run.g
    for name, off, n in zip(ranks[0].names, ranks[0].offsets, ranks[0].sizes):
        assert relerr(host(gsum[off:off + n]).reshape(rg[name].shape), rg[name]) <= TOL_GRAD_BF16, name
    for run in ranks:
        run.g_shard.copy_(gsum[run.shard_begin:run.shard_begin + run.shard_len])
        run.update_shard(hparams(step=1, **hp))
    # all-gather by hand: every rank's slice of the compute copy
    wc = torch.cat([run.wc[run.shard_begin:run.shard_begin + run.shard_len] for run in ranks])
    w = torch.cat([run.w[run.shard_begin:run.shard_begin + run.shard_len] for run in ranks])
    torch.cuda.synchronize()
    w0s = dict(O.lm_tensors(lm))
    for name, off, n in zip(ranks[0].names, ranks[0].offsets, ranks[0].sizes):
        w0 = w0s[name].astype(np.float64).reshape(-1)
        cw, _, _ = O.adamw(w0, 0 * w0, 0 * w0, host(gsum[off:off + n]), weight_decay=wd, step=1, **hp)
        assert relerr(host(w[off:off + n]), cw) <= TOL_ADAMW, name
        assert torch.equal(wc[off:off + n], w[off:off + n].to(torch.bfloat16)), name
    # a rank touches nothing outside its shard
    for run in ranks:
        lo, hi = run.shard_begin, run.shard_begin + run.shard_len
        assert torch.count_nonzero(run.m[:lo]) == 0 and torch.count_nonzero(run.m[hi:]) == 0
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def test_world_of_one_step_matches_the_single_gpu_step(sess):
    """DpLmRunner.step with one rank (collectives are identities) against fax_lm_step on the same model."""
    lm = synth.lm_params(CFG)
    ids, tg = synth.lm_tokens(CFG)
    hp = dict(synth.ADAMW)
    wd = hp.pop("weight_decay")
    tid, ttg = torch.as_tensor(ids).to(sess.device), torch.as_tensor(tg).to(sess.device)
    a = dp.DpLmRunner(sess, CFG, lm, weight_decay=wd)
    b = LmRunner(sess, CFG, lm, fx.FAX_PREC_BF16, weight_decay=wd)
    for s in (1, 2):
        a.step(tid, ttg, hparams(step=s, **hp))
        b.step(tid, ttg, hparams(step=s, **hp))
    torch.cuda.synchronize()
    assert abs(a.global_loss() - float(b.loss.item())) <= 1e-5 * abs(float(b.loss.item()))
    for (name, pa), (_, pb) in zip(a.named_params(), b.named_params()):
        # same kernels; the float32 additions of dQ and of the tied-embedding scatter arrive in another
        # order from run to run, and a first-step Adam update is lr * sign(g): compare the moments
        # (linear in g) tightly and the weights within two updates
        assert relerr(host(pa.m), host(pb.m).reshape(-1)) <= 1e-4, name
        assert float((pa.w - pb.w.reshape(-1)).abs().max()) <= 2.1 * 2 * hp["lr"], name
