"""LayerNorm backward through the entry point that needs no scratch from the caller and
allocates nothing (for hosts whose memory pool owns the whole GPU, fixed-budget plug-ins and
latency-critical loops that cannot call cudaMalloc).  It must give what the ordinary entry
point gives, on two calls in a row (the second one sees the array as the first left it),
and refuse sizes beyond its fixed array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from parity_util import fx, ptr, Session, host, relerr, TOL_GRAD_BF16
from paper_2204_06514_b200 import binding_ops as ops

pytestmark = pytest.mark.gpu


def test_layernorm_backward_static_matches_scratch_version():
    sess = Session(0)
    try:
        dev = sess.device
        g = torch.Generator(device=dev)
        g.manual_seed(11)
        for call, (rows, d) in enumerate([(1024, 4096), (515, 768)]):
            rn = lambda *s: torch.randn(s, generator=g, device=dev).to(torch.bfloat16)
            x, da, add, gam, bet = rn(rows, d), rn(rows, d), rn(rows, d), rn(d), rn(d)
            out = torch.empty_like(x)
            mu = torch.empty(rows, dtype=torch.float32, device=dev)
            rstd = torch.empty_like(mu)
            ops.fax_op_layernorm_forward(sess.ctx, 0, rows, d, ptr(x), ptr(gam), ptr(bet), 1e-5, ptr(out), ptr(mu), ptr(rstd))
            nb = ops.fax_op_layernorm_backward_scratch_bytes(rows, d)
            scratch = sess.arena(nb)
            ref = [torch.empty_like(x), torch.empty(d, dtype=torch.float32, device=dev),
                   torch.empty(d, dtype=torch.float32, device=dev)]
            ops.fax_op_layernorm_backward(sess.ctx, 0, rows, d, ptr(da), ptr(x), ptr(mu), ptr(rstd), ptr(gam), ptr(add),
                                          ptr(ref[0]), ptr(ref[1]), ptr(ref[2]), ptr(scratch), nb)
            got = [torch.full_like(t, float("nan")) for t in ref]
            ops.fax_op_layernorm_backward_static(sess.ctx, 0, rows, d, ptr(da), ptr(x), ptr(mu), ptr(rstd), ptr(gam),
                                                 ptr(add), ptr(got[0]), ptr(got[1]), ptr(got[2]))
            torch.cuda.synchronize()
            for a, b, name in zip(got, ref, ("dx", "dgamma", "dbeta")):
                assert relerr(host(a), host(b)) <= TOL_GRAD_BF16, (call, name)
                assert torch.equal(a, b), (call, name)          # same kernels, same order: identical
        # beyond the fixed array: refused, outputs untouched
        rows, d = 256, 16384
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
