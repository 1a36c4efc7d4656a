"""Per-operator micro-benchmark through the C ABI: times one operator with CUDA
events on the launching stream and prints one JSON line with its achieved
TFLOP/s or GB/s.  Also the small, self-contained workload to put under a
profiler.

  python -m paper_2204_06514_b200.opbench gemm --m 8192 --n 4096 --k 4096 [--a-mn 0 --b-mn 1 --epi 1 --f32-out 0]
  python -m paper_2204_06514_b200.opbench attn_fwd --batch 4 --seq 2048 --heads 32 --hd 128
  python -m paper_2204_06514_b200.opbench attn_bwd --batch 4 --seq 2048 --heads 32 --hd 128
  python -m paper_2204_06514_b200.opbench ln_fwd --rows 8192 --d 4096
  python -m paper_2204_06514_b200.opbench ln_bwd --rows 8192 --d 4096
  python -m paper_2204_06514_b200.opbench adamw --n 201379840
"""
from __future__ import annotations

import argparse
import ctypes as C
import json

import torch

from . import binding as fx
from . import binding_ops as ops
from . import build
from .state import Session, hparams


def P(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["gemm", "attn_fwd", "attn_bwd", "ln_fwd", "ln_bwd", "adamw"])
    ap.add_argument("--m", type=int, default=8192); ap.add_argument("--n", type=int, default=4096)
    ap.add_argument("--k", type=int, default=4096)
    ap.add_argument("--a-mn", type=int, default=0); ap.add_argument("--b-mn", type=int, default=1)
    ap.add_argument("--epi", type=int, default=0); ap.add_argument("--f32-out", type=int, default=0)
    ap.add_argument("--batch", type=int, default=4); ap.add_argument("--seq", type=int, default=2048)
    ap.add_argument("--heads", type=int, default=32); ap.add_argument("--hd", type=int, default=128)
    ap.add_argument("--rows", type=int, default=8192); ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--iters", type=int, default=20); ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--l2-budget-mb", type=float, default=-1.0, help="GEMM raster: L2 bytes for resident panels (0: fixed order)")
    a = ap.parse_args()
    build.build()
    s = Session(0)
    if a.l2_budget_mb >= 0:
        fx.fax_set_gemm_l2_budget(s.ctx, int(a.l2_budget_mb * 1e6))
    dev, bf = s.device, torch.bfloat16
    g = torch.Generator(device=dev); g.manual_seed(1)
    rn = lambda *shape: torch.randn(shape, generator=g, device=dev).to(bf)
    flops = bytes_ = 0.0
    if a.op == "gemm":
        M, N, K = a.m, a.n, a.k
        A = rn(K, M) if a.a_mn else rn(M, K)
        B = rn(K, N) if a.b_mn else rn(N, K)
        Cc = torch.zeros((M, N), device=dev, dtype=torch.float32 if a.f32_out else bf)
        bias, aux = rn(N), rn(M, N)
        desc = ops.GemmDesc(M, N, K, P(A), M if a.a_mn else K, a.a_mn, P(B), N if a.b_mn else K, a.b_mn, P(Cc), N,
                            a.f32_out, 0, a.epi, P(bias), P(aux), N, P(aux), N, 1.0, 0)
        fn = lambda: ops.fax_op_gemm(s.ctx, 0, desc)
        flops = 2.0 * M * N * K
    elif a.op in ("attn_fwd", "attn_bwd"):
        Bn, T, H, hd = a.batch, a.seq, a.heads, a.hd
        d = H * hd
        qkv, do = rn(Bn * T, 3 * d), rn(Bn * T, d)
        o = torch.empty((Bn * T, d), device=dev, dtype=bf)
        lse = torch.empty((Bn, H, T), device=dev, dtype=torch.float32)
        ops.fax_op_attention_forward(s.ctx, 0, Bn, T, H, hd, P(qkv), P(o), P(lse))
        if a.op == "attn_fwd":
            fn = lambda: ops.fax_op_attention_forward(s.ctx, 0, Bn, T, H, hd, P(qkv), P(o), P(lse))
            flops = 2.0 * Bn * H * T * T * hd
        else:
            nb = ops.fax_op_attention_backward_scratch_bytes(0, Bn, T, H, hd)
            scratch, dqkv = s.arena(nb), torch.empty_like(qkv)
            fn = lambda: ops.fax_op_attention_backward(s.ctx, 0, Bn, T, H, hd, P(qkv), P(o), P(lse), P(do), P(dqkv),
                                                       P(scratch), nb)
            flops = 4.0 * Bn * H * T * T * hd
    elif a.op in ("ln_fwd", "ln_bwd"):
        R, d = a.rows, a.d
        x, da, gam, bet = rn(R, d), rn(R, d), rn(d), rn(d)
        out = torch.empty_like(x)
        mu = torch.empty(R, device=dev, dtype=torch.float32); rstd = torch.empty_like(mu)
        ops.fax_op_layernorm_forward(s.ctx, 0, R, d, P(x), P(gam), P(bet), 1e-5, P(out), P(mu), P(rstd))
        if a.op == "ln_fwd":
            fn = lambda: ops.fax_op_layernorm_forward(s.ctx, 0, R, d, P(x), P(gam), P(bet), 1e-5, P(out), P(mu), P(rstd))
            bytes_ = 2.0 * R * d * 2
        else:
            nb = ops.fax_op_layernorm_backward_scratch_bytes(R, d)
            scratch = s.arena(nb)
            dg = torch.empty(d, device=dev, dtype=torch.float32); db = torch.empty_like(dg)
            fn = lambda: ops.fax_op_layernorm_backward(s.ctx, 0, R, d, P(da), P(x), P(mu), P(rstd), P(gam), P(x),
                                                       P(out), P(dg), P(db), P(scratch), nb)
            bytes_ = 4.0 * R * d * 2
    else:
        n = a.n if a.n > 4096 else 201379840
        w = torch.randn(n, generator=g, device=dev); m = torch.zeros_like(w); v = torch.zeros_like(w)
        gr = torch.randn(n, generator=g, device=dev); wc = torch.empty(n, device=dev, dtype=bf)
        t = [fx.AdamwTensor(P(w), P(m), P(v), P(gr), P(wc), n, 0.1)]
        hp = hparams(1e-3, 0.9, 0.95, 1e-8, 1)
        fn = lambda: fx.fax_adamw_step(s.ctx, t, hp)
        bytes_ = 30.0 * n
    for _ in range(a.warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s.stream)
    for _ in range(a.iters):
        fn()
    e1.record(s.stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    st, detail = fx.fax_check_device_status(s.ctx)
    out = {"op": a.op, "ms": ms, "status": st, "detail": detail}
    if flops:
        out.update(tflops=flops / ms / 1e9, flops=flops)
    else:
        out.update(gbs=bytes_ / ms / 1e6, bytes=bytes_)
    print(json.dumps(out))
    s.close()


if __name__ == "__main__":
    main()
