"""LayerNorm backward through the entry point that needs no scratch from the caller and
allocates nothing (for hosts whose memory pool owns the whole GPU, fixed-budget plug-ins and
latency-critical loops that cannot call cudaMalloc).  It must give what the ordinary entry
point gives and what the oracle gives, on calls in a row (each sees the array as the one
before left it, here even filled with NaN partial sums), must leave the device's free memory
as it found it, and must refuse sizes beyond its fixed array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from parity_util import O, fx, ptr, synth, Session, host, relerr, TOL_GRAD_BF16, TOL_FP32
from paper_2204_06514_b200 import binding_ops as ops

pytestmark = pytest.mark.gpu


def _case(sess, prec, rows, d, seed, poison=False):
    """One problem through both entry points; returns nothing, asserts everything."""
    dev = sess.device
    dt = torch.bfloat16 if prec == 0 else torch.float32
    rnd = synth.round_to_bf16 if prec == 0 else (lambda a: a)
    rng = np.random.default_rng(seed)
    x = rnd((rng.standard_normal((rows, d)) * 2 + 0.5).astype(np.float32))
    gam = rnd((1 + 0.2 * rng.standard_normal(d)).astype(np.float32))
    bet = rnd((0.2 * rng.standard_normal(d)).astype(np.float32))
    da = rnd(rng.standard_normal((rows, d)).astype(np.float32))
    add = rnd(rng.standard_normal((rows, d)).astype(np.float32))
    if poison:
        da[:] = np.nan
    up = lambda a: torch.as_tensor(a).to(dev).to(dt).contiguous()
    tx, tg, tb, tda, tadd = (up(a) for a in (x, gam, bet, da, add))
    out = torch.empty_like(tx)
    mu = torch.empty(rows, dtype=torch.float32, device=dev)
    rstd = torch.empty_like(mu)
    ops.fax_op_layernorm_forward(sess.ctx, prec, rows, d, ptr(tx), ptr(tg), ptr(tb), 1e-5, ptr(out), ptr(mu), ptr(rstd))
    nb = ops.fax_op_layernorm_backward_scratch_bytes(rows, d)
    scratch = sess.arena(nb)
    ref = [torch.empty_like(tx), torch.empty(d, dtype=torch.float32, device=dev),
           torch.empty(d, dtype=torch.float32, device=dev)]
    ops.fax_op_layernorm_backward(sess.ctx, prec, rows, d, ptr(tda), ptr(tx), ptr(mu), ptr(rstd), ptr(tg), ptr(tadd),
                                  ptr(ref[0]), ptr(ref[1]), ptr(ref[2]), ptr(scratch), nb)
    got = [torch.full_like(t, float("nan")) for t in ref]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info(dev)[0]
    ops.fax_op_layernorm_backward_static(sess.ctx, prec, rows, d, ptr(tda), ptr(tx), ptr(mu), ptr(rstd), ptr(tg),
                                         ptr(tadd), ptr(got[0]), ptr(got[1]), ptr(got[2]))
    torch.cuda.synchronize()
    # the property the entry point is named for: the driver's free-memory figure did not move
    assert torch.cuda.mem_get_info(dev)[0] == free_before
    if poison:
        assert torch.isnan(got[1]).all()         # the array now holds NaN partial sums for the next call
        return
    _, rmu, rrstd = O.layernorm_fwd(x, gam, bet, 1e-5)
    rdx, rdg, rdb = O.layernorm_bwd(da, x, rmu, rrstd, gam)
    tol = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    for a, b, r, name in zip(got, ref, (rdx + add, rdg, rdb), ("dx", "dgamma", "dbeta")):
        assert torch.equal(a, b), name                      # same kernels, same order as the scratch-taking call
        assert relerr(host(a), r) <= tol, name              # and both are what the oracle computes


def test_layernorm_backward_static_matches_scratch_version_and_oracle():
    sess = Session(0)
    try:
        dev = sess.device
        # bf16 rows take the fused kernel (partials per block); float32 rows of 4096 (1024 vectors) take the
        # dx kernel plus the column reduction, whose partials fill the array differently
        _case(sess, 0, 1024, 4096, 11)
        _case(sess, 0, 515, 768, 12)
        _case(sess, 1, 515, 4096, 13, poison=True)          # leaves NaN in the shared array ...
        _case(sess, 1, 515, 4096, 13)                        # ... which the next calls must not see
        _case(sess, 0, 1024, 4096, 14)
        # beyond the fixed array: refused, outputs untouched (the limit itself, d = 4096, ran above)
        for rows, d in ((256, 16384), (64, 4096 + 8)):
            z = torch.zeros((rows, d), dtype=torch.bfloat16, device=dev)
            f = torch.zeros(rows, dtype=torch.float32, device=dev)
            dg = torch.full((d,), 7.0, dtype=torch.float32, device=dev)
            with pytest.raises(fx.FaxError) as e:
                ops.fax_op_layernorm_backward_static(sess.ctx, 0, rows, d, ptr(z), ptr(z), ptr(f), ptr(f), ptr(z), None,
                                                     ptr(z), ptr(dg), ptr(dg))
            assert e.value.status == fx.FAX_ERR_WORKSPACE_TOO_SMALL
            assert float(dg.min()) == 7.0
        st, _ = fx.fax_check_device_status(sess.ctx)
        assert st == fx.FAX_OK
    finally:
        sess.close()
