"""GPU parity of the single operators against the fp64 oracle, through the C ABI."""
import ctypes as C

import numpy as np
import pytest
import torch

from parity_util import *  # noqa: F401,F403
from paper_2204_06514_b200 import binding_ops as ops

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sess():
    s = Session(0)
    yield s
    s.close()


def dev(a, dtype, sess):
    return torch.as_tensor(np.asarray(a, dtype=np.float32)).to(sess.device).to(dtype).contiguous()


@pytest.mark.parametrize("step", [1, 2, 10, 1000])
@pytest.mark.parametrize("n", [1, 7, 4096, 1_000_003, 4 * 1_000_003])
def test_adamw_isolated(sess, step, n):
    rng = np.random.default_rng(step * 131 + n)
    w = rng.standard_normal(n).astype(np.float32)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-9, 0, n)).astype(np.float32)
    m = (0.1 * rng.standard_normal(n)).astype(np.float32) if step > 1 else np.zeros(n, np.float32)
    v = (m.astype(np.float64) ** 2 + 1e-3 * rng.random(n)).astype(np.float32) if step > 1 else np.zeros(n, np.float32)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8)
    tw, tm, tv, tg = (dev(a, torch.float32, sess) for a in (w, m, v, g))
    twc = torch.zeros(n, dtype=torch.bfloat16, device=sess.device)
    t = fx.AdamwTensor(ptr(tw), ptr(tm), ptr(tv), ptr(tg), ptr(twc), n, 0.1)
    fx.fax_adamw_step(sess.ctx, [t], hparams(step=step, **hp))
    rw, rm, rv = O.adamw(w, m, v, g, weight_decay=0.1, step=step, **hp)
    assert relerr(host(tw), rw) <= TOL_ADAMW
    assert relerr(host(tm), rm) <= TOL_ADAMW
    assert relerr(host(tv), rv) <= TOL_ADAMW
    # the compute copy is the bf16 rounding of the new float32 weight, bit for bit
    assert torch.equal(twc, tw.to(torch.bfloat16))


def test_adamw_many_tensors_and_bf16_grads(sess):
    rng = np.random.default_rng(5)
    sizes = [3, 128, 4096, 4097, 100_000] * 20            # 100 tensors: several launches
    tens, refs = [], []
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8)
    for i, n in enumerate(sizes):
        w = rng.standard_normal(n).astype(np.float32)
        g = synth.round_to_bf16(rng.standard_normal(n).astype(np.float32))
        tw = dev(w, torch.float32, sess)
        tm = torch.zeros_like(tw); tv = torch.zeros_like(tw)
        tg = dev(g, torch.bfloat16, sess)
        wd = 0.1 if i % 2 else 0.0
        tens.append((tw, tm, tv, tg))
        refs.append(O.adamw(w, 0 * w, 0 * w, g, weight_decay=wd, step=1, **hp)[0])
    structs = [fx.AdamwTensor(ptr(a), ptr(b), ptr(c), ptr(d), None, a.numel(), 0.1 if i % 2 else 0.0)
               for i, (a, b, c, d) in enumerate(tens)]
    fx.fax_adamw_step(sess.ctx, structs, hparams(step=1, grad_is_bf16=1, **hp))
    for (tw, _, _, _), r in zip(tens, refs):
        assert relerr(host(tw), r) <= TOL_ADAMW


# rows wider than 4096 bf16 / 2048 float elements take the one-row-per-block backward (2, 3 or 4 vectors per
# thread); 20480 bf16 and 16384 float are past it (separate dx and column-sum kernels)
@pytest.mark.parametrize("prec,rows,d", [(0, 256, 256), (0, 515, 768), (0, 64, 4096), (0, 33, 12288),
                                         (0, 300, 5120), (0, 515, 8192), (0, 161, 10240), (0, 310, 12288),
                                         (0, 150, 16384), (0, 20, 20480),
                                         (1, 10, 8), (1, 300, 1000), (1, 17, 4096), (1, 160, 2052), (1, 40, 8192),
                                         (1, 9, 16384)])
def test_layernorm_forward_backward(sess, prec, rows, d):
    rng = np.random.default_rng(rows + d)
    dt = torch.bfloat16 if prec == 0 else torch.float32
    rnd = synth.round_to_bf16 if prec == 0 else (lambda a: a)
    x = rnd((rng.standard_normal((rows, d)) * 2 + 0.5).astype(np.float32))
    gam = rnd((1 + 0.2 * rng.standard_normal(d)).astype(np.float32))
    bet = rnd((0.2 * rng.standard_normal(d)).astype(np.float32))
    da = rnd(rng.standard_normal((rows, d)).astype(np.float32))
    add = rnd(rng.standard_normal((rows, d)).astype(np.float32))
    tx, tg, tb, tda, tadd = (dev(a, dt, sess) for a in (x, gam, bet, da, add))
    out = torch.empty_like(tx)
    mu = torch.empty(rows, dtype=torch.float32, device=sess.device)
    rstd = torch.empty_like(mu)
    ops.fax_op_layernorm_forward(sess.ctx, prec, rows, d, ptr(tx), ptr(tg), ptr(tb), 1e-5, ptr(out), ptr(mu), ptr(rstd))
    ra, rmu, rrstd = O.layernorm_fwd(x, gam, bet, 1e-5)
    tol = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    assert relerr(host(out), ra) <= tol
    assert relerr(host(mu), rmu) <= 1e-5 and relerr(host(rstd), rrstd) <= 1e-5
    nb = ops.fax_op_layernorm_backward_scratch_bytes(rows, d)
    scratch = sess.arena(nb)
    dx = torch.empty_like(tx)
    dg = torch.empty(d, dtype=torch.float32, device=sess.device)
    db = torch.empty_like(dg)
    ops.fax_op_layernorm_backward(sess.ctx, prec, rows, d, ptr(tda), ptr(tx), ptr(mu), ptr(rstd), ptr(tg),
                                  ptr(tadd), ptr(dx), ptr(dg), ptr(db), ptr(scratch), nb)
    rdx, rdg, rdb = O.layernorm_bwd(da, x, rmu, rrstd, gam)
    tolg = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    assert relerr(host(dx), rdx + add) <= tolg
    assert relerr(host(dg), rdg) <= tolg and relerr(host(db), rdb) <= tolg


GEMM_SHAPES = [(128, 128, 64), (256, 384, 192), (100, 36, 50), (512, 1024, 2048), (384, 128, 4096 + 64),
               (256, 1408, 128), (1408, 256, 128)]       # the last two: 256-multiple part + 128 tail


@pytest.mark.parametrize("prec", [0, 1])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 1), (0, 0), (1, 1), (1, 0)])
@pytest.mark.parametrize("shape", GEMM_SHAPES)
@pytest.mark.parametrize("force_simt", [0, 1])
def test_gemm_layouts(sess, prec, a_mn, b_mn, shape, force_simt):
    M, N, K = shape
    if prec == 1 and force_simt == 0:
        pytest.skip("float32 has one kernel")
    rng = np.random.default_rng(M * 7 + N * 3 + K + a_mn * 2 + b_mn)
    dt = torch.bfloat16 if prec == 0 else torch.float32
    rnd = synth.round_to_bf16 if prec == 0 else (lambda a: a)
    A = rnd(rng.standard_normal((M, K)).astype(np.float32))
    B = rnd(rng.standard_normal((N, K)).astype(np.float32))
    tA = dev(A.T if a_mn else A, dt, sess)
    tB = dev(B.T if b_mn else B, dt, sess)
    tC = torch.empty((M, N), dtype=dt, device=sess.device)
    desc = ops.GemmDesc(M, N, K, ptr(tA), M if a_mn else K, a_mn, ptr(tB), N if b_mn else K, b_mn,
                        ptr(tC), N, 0, 0, ops.FAX_EPI_NONE, None, None, 0, None, 0, 1.0, force_simt)
    if prec == 0 and not force_simt and (M % 128 or N % 64 or K % 64):
        # a bf16 shape the tensor-core kernels do not take is refused, never run on the SIMT kernel unasked
        with pytest.raises(fx.FaxError) as e:
            ops.fax_op_gemm(sess.ctx, prec, desc)
        assert e.value.status == fx.FAX_ERR_UNSUPPORTED_SHAPE
        return
    ops.fax_op_gemm(sess.ctx, prec, desc)
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    assert relerr(host(tC), ref) <= (TOL_FWD_BF16 if prec == 0 else TOL_FP32)


@pytest.mark.parametrize("prec", [0, 1])
@pytest.mark.parametrize("force_simt", [0, 1])
def test_gemm_epilogues(sess, prec, force_simt):
    if prec == 1 and force_simt == 0:
        pytest.skip("float32 has one kernel")
    M, N, K = 384, 256, 320
    rng = np.random.default_rng(99)
    dt = torch.bfloat16 if prec == 0 else torch.float32
    rnd = synth.round_to_bf16 if prec == 0 else (lambda a: a)
    tol = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    A = rnd(rng.standard_normal((M, K)).astype(np.float32))
    B = rnd((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    bias = rnd(rng.standard_normal(N).astype(np.float32))
    res = rnd(rng.standard_normal((M, N)).astype(np.float32))
    tA, tB, tbias, tres = (dev(a, dt, sess) for a in (A, B, bias, res))
    acc = A.astype(np.float64) @ B.astype(np.float64).T

    def run(epi, c_f32=0, accumulate=0, aux=None, C0=None, alpha=1.0):
        tC = torch.zeros((M, N), dtype=torch.float32 if c_f32 else dt, device=sess.device)
        if C0 is not None:
            tC.copy_(torch.as_tensor(C0))
        desc = ops.GemmDesc(M, N, K, ptr(tA), K, 0, ptr(tB), K, 0, ptr(tC), N, c_f32, accumulate, epi,
                            ptr(tbias), ptr(tres), N, ptr(aux), N, alpha, force_simt)
        ops.fax_op_gemm(sess.ctx, prec, desc)
        return host(tC)

    assert relerr(run(ops.FAX_EPI_BIAS), acc + bias) <= tol
    assert relerr(run(ops.FAX_EPI_BIAS_RESID), acc + bias + res) <= tol
    assert relerr(run(ops.FAX_EPI_NONE, alpha=0.125), 0.125 * acc) <= tol
    aux = torch.zeros((M, N), dtype=dt, device=sess.device)
    h = run(ops.FAX_EPI_BIAS_GELU, aux=aux)
    assert relerr(h, acc + bias) <= tol
    assert relerr(host(aux), O.gelu_tanh(acc + bias)) <= tol
    hpre = rnd(rng.standard_normal((M, N)).astype(np.float32))
    auxin = dev(hpre, dt, sess)
    assert relerr(run(ops.FAX_EPI_DGELU, aux=auxin), acc * O.gelu_tanh_grad(hpre)) <= tol
    C0 = rng.standard_normal((M, N)).astype(np.float32)
    assert relerr(run(ops.FAX_EPI_NONE, c_f32=1), acc) <= (1e-5 if prec == 1 else tol)
    assert relerr(run(ops.FAX_EPI_NONE, c_f32=1, accumulate=1, C0=C0), acc + C0) <= (1e-5 if prec == 1 else tol)


# (768, 2304, 16384): 27 tiles on 74 SM pairs, five slices; (2560, 2560, 4096): 100 tiles, sliced to fill the second wave
@pytest.mark.parametrize("M,N,K", [(128, 256, 4096), (768, 768, 16384), (256, 128, 1088), (768, 2304, 16384),
                                   (2560, 2560, 4096)])
@pytest.mark.parametrize("accumulate", [0, 1])
def test_gemm_weight_gradient_shapes_split_k(sess, M, N, K, accumulate):
    """Few output tiles, long K: the kernel slices K and adds partial tiles into the float output."""
    rng = np.random.default_rng(M + N + K)
    A = synth.round_to_bf16(rng.standard_normal((K, M)).astype(np.float32))      # stored [K, M]
    B = synth.round_to_bf16(rng.standard_normal((K, N)).astype(np.float32))      # stored [K, N]
    C0 = rng.standard_normal((M, N)).astype(np.float32)
    tA, tB = dev(A, torch.bfloat16, sess), dev(B, torch.bfloat16, sess)
    tC = torch.as_tensor(C0).to(sess.device).contiguous()
    desc = ops.GemmDesc(M, N, K, ptr(tA), M, 1, ptr(tB), N, 1, ptr(tC), N, 1, accumulate, ops.FAX_EPI_NONE,
                        None, None, 0, None, 0, 1.0, 0)
    for _ in range(2 if not accumulate else 1):          # overwrite mode is idempotent
        ops.fax_op_gemm(sess.ctx, 0, desc)
    ref = A.astype(np.float64).T @ B.astype(np.float64) + (C0 if accumulate else 0.0)
    assert relerr(host(tC), ref) <= 1e-5
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def _step_gemm_shapes(cfg):
    """The twelve contractions of one block step at a config's full size:
    (name, M, N, K, a_mn, b_mn, epilogue, float output)."""
    n, d, f = cfg.tokens, cfg.d_model, cfg.d_ff
    E = ops
    return [
        ("qkv", n, 3 * d, d, 0, 1, E.FAX_EPI_BIAS, 0), ("out_proj", n, d, d, 0, 1, E.FAX_EPI_BIAS_RESID, 0),
        ("fc1", n, f, d, 0, 1, E.FAX_EPI_BIAS_GELU, 0), ("fc2", n, d, f, 0, 1, E.FAX_EPI_BIAS_RESID, 0),
        ("fc2_dx", n, f, d, 0, 0, E.FAX_EPI_DGELU, 0), ("fc1_dx", n, d, f, 0, 0, E.FAX_EPI_NONE, 0),
        ("out_proj_dx", n, d, d, 0, 0, E.FAX_EPI_NONE, 0), ("qkv_dx", n, d, 3 * d, 0, 0, E.FAX_EPI_NONE, 0),
        ("fc2_dw", f, d, n, 1, 1, E.FAX_EPI_NONE, 1), ("fc1_dw", d, f, n, 1, 1, E.FAX_EPI_NONE, 1),
        ("out_proj_dw", d, d, n, 1, 1, E.FAX_EPI_NONE, 1), ("qkv_dw", d, 3 * d, n, 1, 1, E.FAX_EPI_NONE, 1),
    ]


@pytest.mark.parametrize("name", ["C3", "C5"])
def test_gemm_full_size_sampled(sess, name):
    """Dense seeded data through every GEMM shape of a full-size block step (forward, dX with the
    transposed weight, dW with the long token contraction, all fused epilogues): sampled output rows,
    all their columns, against float64.  A K block skipped or read twice, or a tile written to the
    wrong place, shows up here; the full-size block tests feed the dW products mostly zeros."""
    cfg = synth.CONFIGS[name]
    rng = np.random.default_rng(cfg.seed + 4242)
    bf = torch.bfloat16
    cache = {}

    def operand(rows, cols, scale):
        # one bf16 matrix per (rows, cols): weights are reused by the forward and the dX product
        key = (rows, cols)
        if key not in cache:
            a = synth.round_to_bf16(rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(scale))
            cache[key] = (a, dev(a, bf, sess))
        return cache[key]

    for gname, M, N, K, a_mn, b_mn, epi, c_f32 in _step_gemm_shapes(cfg):
        A, tA = operand(K, M, 1.0) if a_mn else operand(M, K, 1.0)
        B, tB = operand(K, N, K ** -0.5) if b_mn else operand(N, K, K ** -0.5)
        rows = np.sort(rng.choice(M, size=96, replace=False))
        bias = synth.round_to_bf16(rng.standard_normal(N).astype(np.float32))
        extra = synth.round_to_bf16(rng.standard_normal((M, N), dtype=np.float32))      # residual or pre-activation
        tbias, textra = dev(bias, bf, sess), dev(extra, bf, sess)
        tC = torch.empty((M, N), dtype=torch.float32 if c_f32 else bf, device=sess.device)
        taux = torch.empty((M, N), dtype=bf, device=sess.device) if epi == ops.FAX_EPI_BIAS_GELU else textra
        desc = ops.GemmDesc(M, N, K, ptr(tA), M if a_mn else K, a_mn, ptr(tB), N if b_mn else K, b_mn, ptr(tC), N,
                            c_f32, 0, epi, ptr(tbias), ptr(textra), N, ptr(taux), N, 1.0, 0)
        ops.fax_op_gemm(sess.ctx, 0, desc)
        a_rows = (A[:, rows].T if a_mn else A[rows]).astype(np.float64)
        acc = a_rows @ (B.astype(np.float64) if b_mn else B.astype(np.float64).T)
        if epi == ops.FAX_EPI_BIAS:
            ref = acc + bias
        elif epi == ops.FAX_EPI_BIAS_RESID:
            ref = acc + bias + extra[rows]
        elif epi == ops.FAX_EPI_BIAS_GELU:
            ref = acc + bias
            g = taux[torch.as_tensor(rows, device=sess.device)]
            assert relerr(host(g), O.gelu_tanh(ref)) <= TOL_FWD_BF16, (gname, "gelu")
        elif epi == ops.FAX_EPI_DGELU:
            ref = acc * O.gelu_tanh_grad(extra[rows])
        else:
            ref = acc
        got = host(tC[torch.as_tensor(rows, device=sess.device)])
        # float output: float32 accumulation over K = 2048 .. 8192 terms against float64 (a few sqrt(K) * 2^-24)
        assert relerr(got, ref) <= (5e-5 if c_f32 else TOL_FWD_BF16), gname
        del tC, tbias, textra, taux
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


@pytest.mark.parametrize("M,N,K", [(2560, 1024, 1024), (1024, 3072, 512), (1280, 1408, 256), (2048, 2048, 2048)])
def test_gemm_raster_order_leaves_results_unchanged(sess, M, N, K):
    """The tile order (groups along rows or along columns, sized by the L2 budget) only changes which tile
    a CTA takes when: every budget gives the same bits, each tile computed exactly once."""
    rng = np.random.default_rng(M + 3 * N + 7 * K)
    A = synth.round_to_bf16(rng.standard_normal((M, K), dtype=np.float32))
    B = synth.round_to_bf16(rng.standard_normal((N, K), dtype=np.float32))
    tA, tB = dev(A, torch.bfloat16, sess), dev(B, torch.bfloat16, sess)
    outs = []
    try:
        for budget in (0, 1 << 20, 3 << 20, 8 << 20, 48_000_000, 1 << 30):
            fx.fax_set_gemm_l2_budget(sess.ctx, budget)
            tC = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=sess.device)
            desc = ops.GemmDesc(M, N, K, ptr(tA), K, 0, ptr(tB), K, 0, ptr(tC), N, 0, 0, ops.FAX_EPI_NONE,
                                None, None, 0, None, 0, 1.0, 0)
            ops.fax_op_gemm(sess.ctx, 0, desc)
            outs.append(tC)
    finally:
        fx.fax_set_gemm_l2_budget(sess.ctx, 48_000_000)
    for o in outs[1:]:
        assert torch.equal(outs[0], o)
    assert relerr(host(outs[0]), A.astype(np.float64) @ B.astype(np.float64).T) <= TOL_FWD_BF16
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


def test_gemm_two_cta_accumulators_recycled_many_times(sess):
    """Far more 256 x 256 tiles than SM pairs with a single K block each: the next tile's product is
    issued the moment an accumulator is handed back, so a hand-back that came before the epilogue had
    read the accumulator would corrupt tiles.  Tile-dependent data; compared bit for bit with the
    one-CTA kernel and against float64."""
    M, N, K = 256 * 40, 256 * 12, 64                       # 480 tiles for 74 SM pairs
    rng = np.random.default_rng(2026)
    A = synth.round_to_bf16(rng.standard_normal((M, K), dtype=np.float32) * (1 + np.arange(M, dtype=np.float32)[:, None] % 7))
    B = synth.round_to_bf16(rng.standard_normal((N, K), dtype=np.float32))
    tA, tB = dev(A, torch.bfloat16, sess), dev(B, torch.bfloat16, sess)
    outs = []
    for two_cta in (1, 0):
        fx.fax_set_gemm_two_cta(sess.ctx, two_cta)
        tC = torch.zeros((M, N), dtype=torch.bfloat16, device=sess.device)
        desc = ops.GemmDesc(M, N, K, ptr(tA), K, 0, ptr(tB), K, 0, ptr(tC), N, 0, 0, ops.FAX_EPI_NONE,
                            None, None, 0, None, 0, 1.0, 0)
        for _ in range(3):
            ops.fax_op_gemm(sess.ctx, 0, desc)
        outs.append(tC)
    fx.fax_set_gemm_two_cta(sess.ctx, 1)
    assert torch.equal(outs[0], outs[1])
    assert relerr(host(outs[0]), A.astype(np.float64) @ B.astype(np.float64).T) <= TOL_FWD_BF16
    st, detail = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK, detail


# T a multiple of 256 takes the two-tile persistent forward kernel; the last two bf16 shapes give it more
# work items than the GPU has SMs, so CTAs loop over several query-tile pairs
ATTN_SHAPES = [(0, 2, 128, 4, 64), (0, 1, 128, 1, 128), (0, 1, 384, 2, 128), (0, 2, 1024, 2, 64), (0, 1, 2048, 1, 128),
               (0, 8, 512, 24, 64), (0, 4, 768, 13, 128),
               (1, 2, 5, 2, 4), (1, 2, 130, 3, 64), (1, 1, 77, 2, 128)]


@pytest.mark.parametrize("prec,B,T,H,hd", ATTN_SHAPES)
def test_attention_forward_backward(sess, prec, B, T, H, hd):
    rng = np.random.default_rng(B * 1000 + T + H + hd)
    d = H * hd
    dt = torch.bfloat16 if prec == 0 else torch.float32
    rnd = synth.round_to_bf16 if prec == 0 else (lambda a: a)
    qkv = rnd(rng.standard_normal((B * T, 3 * d)).astype(np.float32))
    do = rnd(rng.standard_normal((B * T, d)).astype(np.float32))
    tq, tdo = dev(qkv, dt, sess), dev(do, dt, sess)
    o = torch.empty((B * T, d), dtype=dt, device=sess.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=sess.device)
    ops.fax_op_attention_forward(sess.ctx, prec, B, T, H, hd, ptr(tq), ptr(o), ptr(lse))
    ro, rlse, _ = O.attention_fwd(qkv, B, T, H, hd)
    tol = TOL_FWD_BF16 if prec == 0 else TOL_FP32
    assert relerr(host(o), ro) <= tol
    assert np.abs(host(lse) - rlse).max() <= (2e-2 if prec == 0 else 1e-4)
    nb = ops.fax_op_attention_backward_scratch_bytes(prec, B, T, H, hd)
    scratch = sess.arena(nb)
    dqkv = torch.empty_like(tq)
    ops.fax_op_attention_backward(sess.ctx, prec, B, T, H, hd, ptr(tq), ptr(o), ptr(lse), ptr(tdo), ptr(dqkv),
                                  ptr(scratch), nb)
    # the reference backward consumes the same o and lse the kernel saved? No: the oracle's own.
    rd = O.attention_bwd(do, qkv, ro, rlse, B, T, H, hd)
    tolg = TOL_GRAD_BF16 if prec == 0 else TOL_FP32
    got = host(dqkv)
    for i, name in enumerate("qkv"):
        assert relerr(got[:, i * d:(i + 1) * d], rd[:, i * d:(i + 1) * d]) <= tolg, name
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK


@pytest.mark.parametrize("B,T,H,hd", [(2, 640, 5, 128), (2, 640, 6, 64), (1, 1152, 3, 64), (1, 128, 1, 64), (3, 256, 2, 64),
                                      (5, 2048, 31, 64)])
def test_attention_backward_kernels_agree(sess, B, T, H, hd):
    """The three backward kernels (mode 2: two score tiles in flight at head_dim 64; mode 1: sixteen row
    warps with half-tile hand-offs; mode 0: the single hand-off kernel): the same inputs through each,
    each against the oracle."""
    rng = np.random.default_rng(77 + hd + T)
    d = H * hd
    qkv = synth.round_to_bf16(rng.standard_normal((B * T, 3 * d)).astype(np.float32))
    do = synth.round_to_bf16(rng.standard_normal((B * T, d)).astype(np.float32))
    tq, tdo = dev(qkv, torch.bfloat16, sess), dev(do, torch.bfloat16, sess)
    o = torch.empty((B * T, d), dtype=torch.bfloat16, device=sess.device)
    lse = torch.empty((B, H, T), dtype=torch.float32, device=sess.device)
    ops.fax_op_attention_forward(sess.ctx, 0, B, T, H, hd, ptr(tq), ptr(o), ptr(lse))
    ro, rlse, _ = O.attention_fwd(qkv, B, T, H, hd)
    rd = O.attention_bwd(do, qkv, ro, rlse, B, T, H, hd)
    nb = ops.fax_op_attention_backward_scratch_bytes(0, B, T, H, hd)
    scratch = sess.arena(nb)
    try:
        for enable in (2, 1, 0):
            fx.fax_set_attention_backward_two_chains(sess.ctx, enable)
            dqkv = torch.full_like(tq, float("nan"))
            ops.fax_op_attention_backward(sess.ctx, 0, B, T, H, hd, ptr(tq), ptr(o), ptr(lse), ptr(tdo), ptr(dqkv),
                                          ptr(scratch), nb)
            got = host(dqkv)
            for i, name in enumerate("qkv"):
                assert relerr(got[:, i * d:(i + 1) * d], rd[:, i * d:(i + 1) * d]) <= TOL_GRAD_BF16, (enable, name)
    finally:
        fx.fax_set_attention_backward_two_chains(sess.ctx, 2)
    st, _ = fx.fax_check_device_status(sess.ctx)
    assert st == fx.FAX_OK
