#!/usr/bin/env python
"""Benchmark of the single-GPU training step (forward + backward + AdamW).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C1..C5] [--impl ours|reference]

Prints ONE JSON line.  `value` = training tokens/s of the whole job with the
inputs resident in HBM; `e2e` = the same through the host-buffer entry point
(host->device copies of the step's inputs and device->host read of its results
inside the timed region).  N > 1: block workloads (C1-C3, C5, P*), whose inputs
are activations, run as N independent replicas (one process per GPU, no
data-path collective, "scaling": "weak"); LM workloads (C4, F*) train
data-parallel over the workload's batch ("strong": reduce-scatter of the
gradients, AdamW on each rank's shard, all-gather of the bf16 weights).
`--impl reference` times the fp64 CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "training tokens/sec, fwd+bwd+AdamW, 1 GPU (MFU reported beside it)"
UNIT = "tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0        # B200 dense bf16, datasheet
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "gemm_dram_traffic.json")
# A tensor kernel is compared with the burst GEMM peak when the GPU never settled into the power-capped
# state the sustained figure was measured in: timed region under a second, or SM clock sampled above this
BURST_MHZ = 1600.0
BURST_REGION_MS = 1000.0


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def gemm_source_digest() -> str:
    """sha256 over the GEMM kernel sources: a stored traffic figure holds only for the kernels it was taken on."""
    h = hashlib.sha256()
    for name in ("gemm_tcgen05_2cta.cu", "gemm_tcgen05.cu", "gemm_common.cuh", "tc_common.cuh"):
        with open(os.path.join(ROOT, "paper_2204_06514_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def stored_gemm_traffic(workload: str):
    """DRAM bytes (read + written) per GEMM launch of a workload's step, the mean over its launches, taken
    from one-launch ncu captures of each shape; None when no capture exists for the workload or the GEMM
    sources have changed since."""
    try:
        d = json.load(open(TRAFFIC_FILE))
    except (OSError, ValueError):
        return None
    if d.get("gemm_source_digest") != gemm_source_digest():
        return None
    w = d.get("workloads", {}).get(workload)
    return float(w["dram_bytes_per_launch_mean"]) if w else None


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for the life of the run; windows are cut out afterwards."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()

    def window(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        allrows = list(self.rows)
        rows = [r for t, r in allrows if t0 <= t <= t1 + 0.05]
        if not rows:      # a region shorter than the sampling period: the nearest sample
            rows = [r for _, r in sorted(allrows, key=lambda tr: abs(tr[0] - 0.5 * (t0 + t1)))[:1]]
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# The oracle on host cores.  Where host memory and a few minutes allow, ONE whole full-size step
# is timed (forward, loss, backward, AdamW on every tensor).  Otherwise a bounded sample at the
# full sequence length: fewer sequences of the batch (time scales with tokens, attention included),
# or AdamW on a leading slice of every tensor (time scales with elements); the line then says
# "extrapolated": true and gives the factors.
# name -> (sequences timed, AdamW divisor)
ORACLE_PLAN = {"C1": (None, 1), "C2": (None, 1), "C3": (None, 1), "C4": (None, 1),
               "C5": (None, 16), "P1": (None, 16), "P2": (None, 16), "P3": (None, 16),
               "F2": (4, 1), "F3": (4, 1)}
_ORACLE_INPUTS = {}


def oracle_step_seconds(cfg):
    """Seconds the oracle needs for one step of `cfg` on this host, with what was timed.
    Returns (seconds for the full step, cores, description, extrapolated, factors)."""
    import numpy as np
    import threadpoolctl
    from oracle import fax_oracle as O
    from paper_2204_06514_b200 import synth
    seqs, adam_div = ORACLE_PLAN[cfg.name]
    batch = cfg.batch if seqs is None else min(seqs, cfg.batch)
    small = synth.scaled(cfg, batch=batch)
    hp = dict(synth.ADAMW, step=1)
    info = threadpoolctl.threadpool_info()
    cores = max((i.get("num_threads", 1) for i in info), default=1)
    key = (cfg.name, batch)
    if key not in _ORACLE_INPUTS:
        rng = np.random.default_rng(0)
        blocks = [{k: (rng.standard_normal(s) * 0.02 if k.startswith("w_") else
                       (np.ones(s) if k.endswith("_g") else np.zeros(s)))
                   for k, s in small.block_param_shapes().items()} for _ in range(small.n_layers)]
        if small.is_lm:
            _ORACLE_INPUTS[key] = dict(
                lm=dict(wte=rng.standard_normal((small.vocab, small.d_model)) * 0.02,
                        wpe=rng.standard_normal((small.seq, small.d_model)) * 0.02, blocks=blocks,
                        lnf_g=np.ones(small.d_model), lnf_b=np.zeros(small.d_model)),
                ids=rng.integers(0, small.vocab, (batch, small.seq + 1)))
        else:
            _ORACLE_INPUTS[key] = dict(p=blocks[0], x=rng.standard_normal((small.tokens, small.d_model)),
                                       dy=rng.standard_normal((small.tokens, small.d_model)))
    inp = _ORACLE_INPUTS[key]
    tok_factor = cfg.tokens / small.tokens
    if small.is_lm:
        lm, ids = inp["lm"], inp["ids"]
        zeros = {n: np.zeros(a.shape) for n, a in O.lm_tensors(lm)}
        t0 = time.perf_counter()
        O.lm_step(ids[:, :-1], ids[:, 1:], lm, zeros, zeros, batch, small.seq, small.n_heads, small.head_dim, hp,
                  small.ln_eps)
        dt = time.perf_counter() - t0
        if tok_factor == 1:
            return dt, cores, f"one whole oracle lm_step (forward, loss, backward, AdamW) at full size", False, {}
        # AdamW does not scale with tokens: time it apart on the same tensors
        t0 = time.perf_counter()
        for n, a in O.lm_tensors(lm):
            O.adamw(a, zeros[n], zeros[n], zeros[n], hp["lr"], hp["beta1"], hp["beta2"], hp["eps"], hp["weight_decay"], 1)
        t_ad = time.perf_counter() - t0
        full = (dt - t_ad) * tok_factor + t_ad
        return (full, cores, f"oracle lm_step on {batch} of {cfg.batch} sequences at the full sequence length and depth; "
                f"forward+loss+backward time scaled by tokens, AdamW (all tensors) counted once", True,
                {"tokens": tok_factor})
    p, x, dy = inp["p"], inp["x"], inp["dy"]
    t0 = time.perf_counter()
    y, sv = O.block_forward(x, p, small.batch, small.seq, small.n_heads, small.head_dim, small.ln_eps)
    dx, gr, _ = O.block_backward(dy, sv, p, small.batch, small.seq, small.n_heads, small.head_dim)
    t_fb = time.perf_counter() - t0
    del sv
    t0 = time.perf_counter()
    for k in O.PARAM_NAMES:
        n = max(1, p[k].shape[0] // adam_div)
        w, g = p[k][:n], gr[k][:n]
        O.adamw(w, np.zeros_like(w), np.zeros_like(w), g, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                hp["weight_decay"], 1)
    t_ad = (time.perf_counter() - t0) * adam_div
    full = t_fb * tok_factor + t_ad
    if adam_div == 1 and tok_factor == 1:
        return full, cores, "one whole oracle block step (forward, backward, AdamW on all twelve tensors) at full size", False, {}
    return (full, cores, f"oracle block forward+backward at full size (all {cfg.tokens} tokens) + oracle AdamW on the leading "
            f"1/{adam_div} of every tensor, that time scaled by {adam_div} (float64 copies of the optimizer state of "
            f"{cfg.n_params / 1e9:.1f}e9 parameters do not fit beside the gradients)", True, {"adamw": adam_div})


def run_reference(args):
    """Reference arm: the fp64 oracle on host cores.  Small workloads: warm-up and K real steps; from C3 on,
    one real step (or the bounded sample), timed once."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2204_06514_b200 import synth
    cfg = synth.CONFIGS[args.config]
    t_proc = time.perf_counter()
    repeat = cfg.name in ("C1", "C2")
    secs, cores, what, extrap, factors = [], 1, "", False, {}
    for i in range((args.warmup + args.steps) if repeat else 1):
        s, cores, what, extrap, factors = oracle_step_seconds(cfg)
        if not repeat or i >= args.warmup:
            secs.append(s)
    sec = sum(secs) / len(secs)
    tps = cfg.tokens / sec
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "steps_timed": len(secs), "ms_per_step": 1e3 * sec,
            "extrapolated": extrap, "extrapolation_factors": factors,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": workload_name(cfg)},
            "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what,
                             "extrapolated": extrap},
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "process_seconds": time.perf_counter() - t_proc}
    print(json.dumps(line), flush=True)


def workload_name(cfg):
    if cfg.is_lm:
        return (f"{cfg.name}: {cfg.n_layers}-layer LM step d{cfg.d_model} {cfg.n_heads}x{cfg.head_dim} "
                f"ffn{cfg.d_ff} vocab{cfg.vocab} batch{cfg.batch} seq{cfg.seq}")
    return (f"{cfg.name}: pre-LN decoder block fwd+bwd+AdamW d{cfg.d_model} {cfg.n_heads}x{cfg.head_dim} "
            f"ffn{cfg.d_ff} batch{cfg.batch} seq{cfg.seq}")


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2204_06514_b200 import binding as fx
    from paper_2204_06514_b200 import build, dist_util, synth
    from paper_2204_06514_b200.state import BlockRunner, LmRunner, Session, hparams

    rank, world, local = dist_util.env_rank()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    if rank == 0:
        build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    torch.cuda.set_device(local)
    fx.load_library()
    cfg = synth.CONFIGS[args.config]
    peaks, peaks_kind = load_peaks()
    sess = Session(local)
    dev = sess.device
    fx.fax_set_fused_update(sess.ctx, args.fused_update != "off", args.fused_update == "keep")
    hp0 = dict(synth.ADAMW)
    wd = hp0.pop("weight_decay")
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed + rank)

    def rand(shape, std):
        return torch.randn(shape, generator=gen, device=dev, dtype=torch.float32) * std

    # seeded synthetic state, generated on the device (same recipe as the parity inputs:
    # N(0, 0.02) matrices, zero biases, unit LayerNorm gains; N(0,1) bf16 activations)
    def block_params():
        out = {}
        for k, s in cfg.block_param_shapes().items():
            out[k] = rand(s, 0.02) if k.startswith("w_") else (torch.ones(s) if k.endswith("_g") else torch.zeros(s))
        return out

    step_no = [0]
    # LM workloads on several GPUs train data-parallel over the batch (the global batch is the workload's:
    # strong scaling, one reduce-scatter and one all-gather per step); block workloads, whose inputs are
    # activations, run as independent replicas
    data_parallel = cfg.is_lm and world > 1
    if data_parallel:
        from paper_2204_06514_b200 import dp
        gen.manual_seed(cfg.seed)                   # every rank starts from the same model and the same global batch
        lm = dict(wte=rand((cfg.vocab, cfg.d_model), 0.02), wpe=rand((cfg.seq, cfg.d_model), 0.02),
                  blocks=[block_params() for _ in range(cfg.n_layers)],
                  lnf_g=torch.ones(cfg.d_model), lnf_b=torch.zeros(cfg.d_model))
        lm = {k: ([{n: t.cpu().numpy() for n, t in b.items()} for b in v] if k == "blocks" else v.cpu().numpy())
              for k, v in lm.items()}
        runner = dp.DpLmRunner(sess, cfg, lm, weight_decay=wd, rank=rank, world=world)
        raw = torch.randint(0, cfg.vocab, (cfg.batch, cfg.seq + 1), generator=gen, device=dev, dtype=torch.int32)
        per = cfg.batch // world
        ids = raw[rank * per:(rank + 1) * per, :-1].contiguous()
        tg = raw[rank * per:(rank + 1) * per, 1:].contiguous()
        ids_h, tg_h = ids.cpu().pin_memory(), tg.cpu().pin_memory()
        h2d, d2h = 2 * ids_h.numel() * 4 * world, 4 * world

        def step():
            step_no[0] += 1
            runner.step(ids, tg, hparams(step=step_no[0], **hp0))

        def step_host():
            step_no[0] += 1
            ids.copy_(ids_h, non_blocking=True)
            tg.copy_(tg_h, non_blocking=True)
            runner.step(ids, tg, hparams(step=step_no[0], **hp0))
            runner.loss.item()
    elif cfg.is_lm:
        lm = dict(wte=rand((cfg.vocab, cfg.d_model), 0.02), wpe=rand((cfg.seq, cfg.d_model), 0.02),
                  blocks=[block_params() for _ in range(cfg.n_layers)],
                  lnf_g=torch.ones(cfg.d_model), lnf_b=torch.zeros(cfg.d_model))
        runner = LmRunner(sess, cfg, lm, fx.FAX_PREC_BF16, weight_decay=wd, recompute=args.recompute)
        raw = torch.randint(0, cfg.vocab, (cfg.batch, cfg.seq + 1), generator=gen, device=dev, dtype=torch.int32)
        ids, tg = raw[:, :-1].contiguous(), raw[:, 1:].contiguous()
        ids_h, tg_h = ids.cpu().pin_memory(), tg.cpu().pin_memory()
        h2d, d2h = 2 * ids_h.numel() * 4, 4

        def step():
            step_no[0] += 1
            runner.step(ids, tg, hparams(step=step_no[0], **hp0))

        def step_host():
            step_no[0] += 1
            runner.step_host(ids_h, tg_h, hparams(step=step_no[0], **hp0))
    else:
        runner = BlockRunner(sess, cfg, block_params(), fx.FAX_PREC_BF16, weight_decay=wd, host_io=True,
                             recompute=args.recompute)
        x = torch.randn((cfg.tokens, cfg.d_model), generator=gen, device=dev).to(torch.bfloat16)
        dy = torch.randn((cfg.tokens, cfg.d_model), generator=gen, device=dev).to(torch.bfloat16)
        x_h, dy_h = x.cpu().pin_memory(), dy.cpu().pin_memory()
        y_h, dx_h = torch.empty_like(x_h).pin_memory(), torch.empty_like(x_h).pin_memory()
        h2d = 2 * x_h.numel() * 2
        d2h = 2 * x_h.numel() * 2

        def step():
            step_no[0] += 1
            runner.step(x, dy, hparams(step=step_no[0], **hp0))

        def step_host():
            step_no[0] += 1
            runner.step_host(x_h, dy_h, y_h, dx_h, hparams(step=step_no[0], **hp0))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_marks = []
    windows = {}

    def timed(fn, steps, marks=None, tag=None):
        """K steps between two CUDA events on the launching stream; max over ranks.  With `marks`, an event
        after every step as well (per-step median / minimum; the total is what the metric uses)."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps)] if marks is not None else None
        barrier()
        h0 = time.time()
        e0.record(sess.stream)
        for i in range(steps):
            fn()
            if evs:
                evs[i].record(sess.stream)
        e1.record(sess.stream)
        barrier()
        if tag:
            a, b = windows.get(tag, (h0, h0))
            windows[tag] = (min(a, h0) if tag in windows else h0, time.time())
        if evs:
            prev = e0
            for e in evs:
                marks.append(prev.elapsed_time(e))
                prev = e
        return dist_util.max_over_ranks(e0.elapsed_time(e1), dev)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.25)              # the sampler's first readings; same pause before the timed region as ever
    l0 = sess.launches()
    ms = timed(step, args.steps, step_marks, tag="timed")
    launches = sess.launches() - l0
    st, detail = fx.fax_check_device_status(sess.ctx)
    if st != fx.FAX_OK:
        raise RuntimeError(f"device status {st} detail {detail}")

    # end to end through the host-buffer entry point
    step_host()
    e2e_steps = max(1, min(args.steps, 10))
    ms_e2e = timed(step_host, e2e_steps, tag="e2e")

    # per-kernel profile over whole steps (events around every operator launch)
    # (AdamW is kept on the main stream here so that no kernel's events include another's work)
    fx.fax_set_adamw_overlap(sess.ctx, False)
    fx.fax_profile_begin(sess.ctx)
    prof_steps = max(1, min(args.steps, 5))
    hp_t0 = time.time()
    for _ in range(prof_steps):
        step()
    prof = fx.fax_profile_end(sess.ctx)
    windows["profile"] = (hp_t0, time.time())
    fx.fax_set_adamw_overlap(sess.ctx, True)

    # per-phase split (the paper's Fig. 3 reports forward, loss and backward separately): the phase
    # entry points timed on their own, outside the step's timed region
    ph_steps = max(1, min(args.steps, 5))
    if data_parallel:
        fb = timed(lambda: runner.local_gradients(ids, tg), ph_steps, tag="phases") / ph_steps
        phases = {"forward_loss_backward_ms": fb, "exchange_and_adamw_ms": max(ms / args.steps - fb, 0.0),
                  "note": "local forward + loss + backward; the rest of the step is reduce-scatter, sharded AdamW, all-gather"}
        sum_phases = None
    elif cfg.is_lm:
        fb = timed(lambda: runner.forward_backward(ids, tg), ph_steps, tag="phases") / ph_steps
        phases = {"forward_loss_backward_ms": fb, "adamw_ms": max(ms / args.steps - fb, 0.0),
                  "note": "forward + loss + backward through fax_lm_forward_backward; AdamW = step - that"}
        sum_phases = None
    else:
        hp_ph = hparams(step=1, **hp0)
        fwd = timed(lambda: runner.forward(x), ph_steps, tag="phases") / ph_steps
        bwd = timed(lambda: runner.backward(dy), ph_steps, tag="phases") / ph_steps
        adw = timed(lambda: runner.adamw(hp_ph), ph_steps, tag="phases") / ph_steps
        phases = {"forward_ms": fwd, "backward_ms": bwd, "adamw_ms": adw,
                  "note": "fax_block_forward, fax_block_backward, fax_adamw_step timed separately"}
        sum_phases = fwd + bwd + adw
    sampler.stop()
    clocks = {k: sampler.window(*w) for k, w in windows.items()}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_step = ms / args.steps
    tokens = cfg.tokens
    tps = tokens / (ms_step * 1e-3) if data_parallel else dist_util.whole_job_rate(tokens, world, ms_step)
    flops = cfg.step_flops()
    achieved_tf = flops / (ms_step * 1e-3) / 1e12 / (world if data_parallel else 1)     # per GPU
    # which measured GEMM peak fits this run: the burst figure unless the run sat in the power-capped state
    # the sustained figure was taken in (a timed region of a second or more AND the SM clock sampled low)
    timed_mhz = clocks["timed"].get("sm_mhz")
    burst = ms < BURST_REGION_MS or (timed_mhz is not None and timed_mhz >= BURST_MHZ)
    regime = "burst" if burst else "sustained"
    tensor_peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
    kernels = {}
    total_ms = sum(v["ms"] for v in prof.values()) or 1.0
    for name, v in prof.items():
        per = v["ms"] / v["launches"]
        ent = {"launches_per_step": v["launches"] / prof_steps, "ms_per_step": v["ms"] / prof_steps,
               "share": v["ms"] / total_ms, "avg_launch_ms": per}
        if v["flops"] > 0:
            ach = v["flops"] / (v["ms"] * 1e-3) / 1e12
            ent.update(bound="tensor", achieved=ach, unit="TFLOP/s", frac=ach / tensor_peak,
                       frac_burst=ach / peaks["bf16_tflops"], frac_sustained=ach / peaks["bf16_tflops_sustained"])
        else:
            ent.update(bound="hbm", achieved=v["bytes"] / (v["ms"] * 1e-3) / 1e9, unit="GB/s")
            ent["frac"] = ent["achieved"] / peaks["hbm_gbs"]
        kernels[name] = ent
    top = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    tk = kernels[top]
    traffic = stored_gemm_traffic(cfg.name) if top == "gemm_tcgen05" and not args.recompute else None
    roofline = {"kernel": top, "bound": tk["bound"], "achieved": tk["achieved"],
                "peak": tensor_peak if tk["bound"] == "tensor" else peaks["hbm_gbs"],
                "unit": tk["unit"], "frac": tk["frac"], "traffic": traffic,
                "peak_source": (f"{peaks_kind} ({regime} bf16 GEMM: burst when the timed region is under "
                                f"{BURST_REGION_MS:.0f} ms or the SM clock sampled in it is at least {BURST_MHZ:.0f} MHz, "
                                f"sustained otherwise)" if tk["bound"] == "tensor" else f"{peaks_kind} (copy)"),
                "per_launch": {"avg_ms": tk["avg_launch_ms"],
                               "algorithmic": (prof[top]["flops"] or prof[top]["bytes"]) / prof[top]["launches"]}}
    if tk["bound"] == "tensor":
        roofline.update(frac_burst=tk["frac_burst"], frac_sustained=tk["frac_sustained"], regime=regime)
    # where the step's time is: the step as timed, the per-kernel events of the profile pass (AdamW not
    # overlapped there) and the phase calls, each with the SM clock sampled while it ran
    sum_kernels = total_ms / prof_steps
    mhz = {k: c.get("sm_mhz") for k, c in clocks.items()}
    accounting = {"step_ms": ms_step, "sum_kernels_ms": sum_kernels, "sum_phases_ms": sum_phases, "sm_mhz": mhz,
                  "step_minus_kernels_ms": ms_step - sum_kernels,
                  "sum_kernels_ms_at_timed_clock": (sum_kernels * mhz["profile"] / mhz["timed"]
                                                    if mhz.get("profile") and mhz.get("timed") else None),
                  "note": "the profile pass runs a few steps from idle at a higher clock than the timed region; "
                          "sum_kernels_ms_at_timed_clock rescales it by the sampled clocks (tensor kernels follow "
                          "the SM clock, HBM-bound ones do not)"}

    cpu_sec, cores, what, extrap, factors = oracle_step_seconds(cfg)

    line = {
        "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step,
        "ms_step_median": sorted(step_marks)[len(step_marks) // 2], "ms_step_min": min(step_marks),
        "higher_is_better": True, "scaling": "strong" if data_parallel else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(cfg), "tokens_per_step": tokens, "params": cfg.n_params,
                   "replicas": 1 if data_parallel else world,
                   "parallelism": f"dp{world}: batch sharded, gradients reduce-scattered, AdamW on shards, bf16 weights all-gathered"
                   if data_parallel else ("single GPU" if world == 1 else f"{world} independent replicas"),
                   "fused_update": args.fused_update, "recompute": bool(args.recompute), "l2": "working set per step far exceeds the 126 MB L2"
                   if cfg.n_params * 2 > 200e6 else "working set is L2-resident (small parity config)"},
        "mfu": {"step_flops": flops, "achieved_tflops": achieved_tf,
                "vs_nominal_2250": achieved_tf / NOMINAL_BF16_TFLOPS,
                "vs_measured_burst": achieved_tf / peaks["bf16_tflops"],
                "vs_measured_sustained": achieved_tf / peaks["bf16_tflops_sustained"], "regime": regime,
                "flops_convention": "6*matmul_params*tokens + causal-halved attention (6*B*T^2*d per layer)"},
        "roofline": roofline, "kernels": kernels, "phases": phases, "accounting": accounting,
        "cpu_baseline": {"value": cfg.tokens / cpu_sec, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what,
                         "extrapolated": extrap, "extrapolation_factors": factors, "seconds_per_step": cpu_sec},
        "e2e": {"value": (tokens / (ms_e2e / e2e_steps * 1e-3) if data_parallel
                          else dist_util.whole_job_rate(tokens, world, ms_e2e / e2e_steps)), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches, "clocks": clocks["timed"], "clocks_by_pass": clocks,
    }
    print(json.dumps(line), flush=True)
    sess.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="C3", choices=["C1", "C2", "C3", "C4", "C5", "P1", "P2", "P3", "F3", "F2"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--recompute", action="store_true",
                    help="backward recomputes the LayerNorm outputs and GELU(h) instead of reading saved copies")
    ap.add_argument("--fused-update", default="off", choices=["off", "keep", "nograd"],
                    help="AdamW of the weight matrices in the dW GEMM epilogue: off; on and the gradients still "
                         "stored (default: every output of the step as documented); on without storing them")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
