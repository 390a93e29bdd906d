#!/usr/bin/env python
"""Benchmark of the hybrid causal attention layer (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 1|2|4|5|6]

One step = one pass of the whole hot path over one synthetic batch: forward kernel, backward
preparation (delta, zero-fill) and backward kernel, for the GPT-2-124M-shaped layer
(batch 8, 12 heads of which 3 frozen, T = 4096, head dim 64, bf16).  Pattern normalisers are static
per layer (the method installs them once), so they are prepared once before the timed steps; the
time of that preparation is reported in `config`.

Prints ONE JSON line (rank 0).  `value` is TFLOP/s on the layer's algorithmic FLOPs
(B*D*T*(T+1)*(7*Ho + 2*Hf)), whole job over all ranks, inputs resident in HBM; `e2e` is the same
metric through the host-buffer entry point with every input copied to the device and every output
copied back inside the timed region.  `--impl reference` times the fp64 CPU oracle on a bounded
sample of the same workload.

The K-step region is timed `--repeats` times (default 5) and `ms_per_step` is the median region; the per-kernel
CUDA-event pairs that give the roofline's kernel duration cost a few microseconds per launch, so they are recorded
in one further K-step region of the same steps (`ms_per_step_with_kernel_events`), not in the headline regions.
`--config 4` is the forward-only long-prefill workload.  On config 1 the line carries `sweep`: the same step at 0,
25, 50, 75 and 100 % frozen heads.  With `--gpus N`, N > 1, and no torchrun environment, bench.py starts the N
ranks itself (one process per GPU, rendezvous on 127.0.0.1).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import saf_inputs as si  # noqa: E402

METRIC = "hybrid_attn_fwd_bwd_tflops"
UNIT = "TFLOP/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained"),
                "hbm_gbs": d["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm_sorted = sorted(sm)
        # "under load": the upper half of the samples (idle samples before/after the region drop out)
        load = sm_sorted[len(sm_sorted) // 2:] if sm_sorted else []
        return {"sm_mhz": (load[len(load) // 2] if load else None), "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(wl: si.Workload, budget_s: float = 12.0):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload: whole (b,h) units,
    alternating ordinary and frozen, until the budget is used.  Returns (TFLOP/s, description, threads)."""
    from oracle import saf_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    rng = np.random.default_rng(wl.seed)
    T, D = wl.T, wl.D
    scale = 1.0 / np.sqrt(D)
    ord_heads = [h for h in range(wl.H) if h not in wl.frozen_heads]
    kinds = []
    if ord_heads:
        kinds.append(False)
    if wl.frozen_heads:
        kinds.append(True)
    unit = D * T * (T + 1)
    flops, t_used, n_units, i = 0.0, 0.0, {False: 0, True: 0}, 0
    while t_used < budget_s:
        fr = kinds[i % len(kinds)]
        i += 1
        q, k, v, do = (si.bf16_bits_to_f64(si.f32_to_bf16_bits(rng.standard_normal((T, D), dtype=np.float32)))
                       for _ in range(4))
        alpha = rng.standard_normal(T)
        rho = wl.rho_slope * np.arange(T) + 0.1 * rng.standard_normal(T)
        t0 = time.perf_counter()
        orc.head_fwd_panels(fr, q, k, v, alpha, rho, scale, 1024)
        if wl.backward:
            orc.head_bwd_panels(fr, q, k, v, do, alpha, rho, scale, 1024)
        t_used += time.perf_counter() - t0
        n_units[fr] += 1
        flops += unit * ((2 if fr else 7) if wl.backward else (1 if fr else 2))
    desc = (f"{n_units[False]} ordinary + {n_units[True]} frozen (b,h) units of {wl.name} "
            f"(T={T}, D={D}), fwd{'+bwd' if wl.backward else ''}, dense fp64 numpy, of {wl.B * wl.H} units")
    return flops / t_used / 1e12, desc, threads, t_used


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    wl = si.config(args.config)
    vals, descs = [], None
    for _ in range(args.warmup):
        oracle_sample(wl, budget_s=1.0)
    t_all = 0.0
    for _ in range(args.steps):
        # keep the whole run within a few minutes whatever K is
        v, descs, threads, t = oracle_sample(wl, budget_s=min(args.ref_budget, 150.0 / max(args.steps, 1)))
        vals.append(v)
        t_all += t
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_all / max(args.steps, 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "B": wl.B, "H": wl.H, "Hf": len(wl.frozen_heads), "T": wl.T, "D": wl.D,
                       "note": "each step is a bounded sample of the workload run by the CPU oracle"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": descs},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- GPU arm
# --------------------------------------------------------------------------- the one-time fitter (extra leg)
def fit_leg(ctx, saf, wl, peaks, dev, steps=400):
    """Times the compact-pattern fitter on the heads one intervention of this model shape would fit: target marginals
    of synthetic mean attention maps, then `steps` Adam steps for all heads at once, then the oracle on a bounded
    sample of the same work.  Returns the dict reported under "fit"."""
    import torch
    from oracle import saf_fit_oracle as fo

    T = wl.T
    if T > 16384 or not len(wl.frozen_heads):
        return None
    Hf = max(1, min(12 * len(wl.frozen_heads), int(3.2e9 // (4 * T * T))))
    base = si.mean_attention_maps(min(3, Hf), T, seed=wl.seed + 77)
    A = torch.from_numpy(base).to(dev)
    A = A[torch.arange(Hf, device=dev) % A.shape[0]].contiguous()
    ea = torch.empty(Hf, T, dtype=torch.float64, device=dev)
    er = torch.empty_like(ea)
    pl = torch.empty(Hf, dtype=torch.float64, device=dev)
    fa, fr, fz = (torch.empty(Hf, T, device=dev) for _ in range(3))
    loss = torch.empty(Hf, dtype=torch.float64, device=dev)
    kl = torch.empty_like(loss)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    for _ in range(3):
        ctx.saf_fit_marginals(Hf, T, A, 1e-9, ea, er, pl)
    a, b = ev(), ev()
    a.record()
    for _ in range(5):
        ctx.saf_fit_marginals(Hf, T, A, 1e-9, ea, er, pl)
    b.record()
    torch.cuda.synchronize()
    marg_ms = a.elapsed_time(b) / 5
    ctx.saf_fit_compact(Hf, T, ea, er, pl, 20, 0.05, fa, fr, fz, T, loss, kl)       # warm-up
    a, b = ev(), ev()
    a.record()
    ctx.saf_fit_compact(Hf, T, ea, er, pl, steps, 0.05, fa, fr, fz, T, loss, kl)
    b.record()
    torch.cuda.synchronize()
    fit_ms = a.elapsed_time(b)
    code, detail = ctx.saf_last_device_status()
    if code != saf.SAF_OK:
        raise RuntimeError(f"fitter: device status {code} detail {detail:#x}")
    pairs = T * (T + 1) // 2
    # special-function-unit bound: 16 exp2 per clock per SM, 148 SMs, at the maximum SM clock
    mufu_peak = 16 * 148 * 1.965e9
    exps_min = 2 * pairs * Hf * steps            # one exponential per causal pair for the normalisers, one for the marginals
    exps_run = 3 * pairs * Hf * steps            # the marginal pass evaluates each pair twice (once per marginal)
    marg_bytes = 4 * pairs * Hf
    # the oracle on a bounded sample: one head, a few Adam steps at this T (dense fp64)
    t0 = time.perf_counter()
    P0 = fo.target_from_mean_attention(base[0])
    oea, oer, _ = fo.marginals(P0)
    t1 = time.perf_counter()
    osteps = 2
    fo.fit_compact(oea, oer, steps=osteps)
    t2 = time.perf_counter()
    kl_h = kl.cpu().numpy()
    return {
        "heads": Hf, "T": T, "adam_steps": steps, "fit_ms": fit_ms, "marginals_ms": marg_ms,
        "kappa_min_max": [float(kl_h.min()), float(kl_h.max())], "accepted": int((kl_h <= 0.2).sum()),
        "roofline_fit": {"bound": "alu", "kernel": "saf_fit_pass_kernel", "unit": "Gexp2/s",
                         "achieved": exps_min / (fit_ms * 1e-3) / 1e9, "executed": exps_run / (fit_ms * 1e-3) / 1e9,
                         "peak": mufu_peak / 1e9, "frac": exps_min / (fit_ms * 1e-3) / mufu_peak,
                         "peak_source": "16 exp2/clk/SM x 148 SMs x 1.965 GHz"},
        "roofline_marginals": {"bound": "hbm", "kernel": "saf_fit_marginals_kernel", "unit": "GB/s",
                               "achieved": marg_bytes / (marg_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                               "frac": marg_bytes / (marg_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "cpu_oracle": {"marginals_s_per_head": t1 - t0, "fit_s_per_head_per_step": (t2 - t1) / osteps,
                       "fit_s_extrapolated": (t2 - t1) / osteps * steps * Hf,
                       "sample": f"1 of {Hf} heads, {osteps} of {steps} Adam steps, dense fp64 numpy"},
    }


# --------------------------------------------------------------------------- calibration statistics (extra leg)
def calib_leg(ctx, saf, wl, prob, Q, K, LSE, peaks, dev):
    """Times the calibration statistics of this layer shape with every head ordinary: one streaming call over the
    batch's sequences (mean attention accumulator, variance and forward-KL sums), then the finalisation."""
    import torch

    H, T = wl.H, wl.T
    if wl.packed_qk or 4 * H * T * T > 8e9:
        return None
    mean = torch.zeros(H, T, T, device=dev)
    sumsq = torch.zeros(H, dtype=torch.float64, device=dev)
    plogp = torch.zeros_like(sumsq)
    s_var = torch.zeros_like(sumsq)
    s_kl = torch.zeros_like(sumsq)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    for _ in range(2):
        ctx.saf_calib_accumulate(prob, Q, K, LSE, mean, sumsq, plogp, 0)
    a, m, b, c = ev(), ev(), ev(), ev()
    reps = 5
    a.record()
    for r in range(reps):                      # first call of a layer: the accumulator tiles are written
        ctx.saf_calib_accumulate(prob, Q, K, LSE, mean, sumsq, plogp, 0)
    m.record()
    for r in range(reps):                      # later calls: added to what is there
        ctx.saf_calib_accumulate(prob, Q, K, LSE, mean, sumsq, plogp, 1)
    b.record()
    ctx.saf_calib_finalize(H, T, (reps + 1) * wl.B, mean, sumsq, plogp, s_var, s_kl)
    c.record()
    torch.cuda.synchronize()
    code, detail = ctx.saf_last_device_status()
    if code != saf.SAF_OK:
        raise RuntimeError(f"calibration: device status {code} detail {detail:#x}")
    first_ms = a.elapsed_time(m) / reps
    acc_ms = m.elapsed_time(b) / reps
    fin_ms = b.elapsed_time(c)
    pairs = T * (T + 1) // 2
    mufu_peak = 16 * 148 * 1.965e9
    exps = wl.B * H * pairs
    return {
        "sequences_per_call": wl.B, "heads": H, "T": T, "first_call_ms": first_ms, "accumulate_ms": acc_ms,
        "finalize_ms": fin_ms,
        "s_var_min_max": [float(s_var.min()), float(s_var.max())], "s_kl_min_max": [float(s_kl.min()), float(s_kl.max())],
        "roofline_accumulate": {"bound": "alu", "kernel": "saf_calib_kernel", "unit": "Gexp2/s",
                                "achieved": exps / (acc_ms * 1e-3) / 1e9, "peak": mufu_peak / 1e9,
                                "frac": exps / (acc_ms * 1e-3) / mufu_peak,
                                "peak_source": "16 exp2/clk/SM x 148 SMs x 1.965 GHz",
                                "tensor_tflops": 2.0 * exps * wl.D / (acc_ms * 1e-3) / 1e12},
        "roofline_finalize": {"bound": "hbm", "kernel": "saf_calib_mean_kernel", "unit": "GB/s",
                              "achieved": 8.0 * pairs * H / (fin_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                              "frac": 8.0 * pairs * H / (fin_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
    }


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2609_34650_b200 as saf
    from paper_2609_34650_b200 import dist as sd

    rank, local_rank, world = sd.env_world()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)

    wl = si.config(args.config, seed=sd.rank_seed(0, rank))
    bwd = wl.backward
    inp = si.generate(wl)

    def t16(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)

    hostQ, hostK, hostV, hostdO = (t16(x).pin_memory() for x in (inp.q, inp.k, inp.v, inp.do))
    Q, K, V = (x.to(dev) for x in (hostQ, hostK, hostV))
    dO = hostdO.to(dev) if bwd else None
    alpha_h, rho_h = torch.from_numpy(inp.alpha).pin_memory(), torch.from_numpy(inp.rho).pin_memory()
    alpha, rho = alpha_h.to(dev), rho_h.to(dev)
    logZ = torch.zeros_like(alpha)
    O = torch.empty_like(Q)
    LSE = torch.empty(wl.B, wl.H, wl.T, device=dev)
    dQ, dK, dV = (torch.empty(x.shape, device=dev, dtype=torch.float32) for x in (Q, K, V)) if bwd else (None,) * 3
    ctx = saf.Context(local_rank)
    prob = saf.make_problem(Q, wl.stored_len, k_like=K, v_like=V, kv_group=wl.kv_group)
    mask = inp.mask
    mask0 = np.zeros_like(mask)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # pattern preparation: once, timed on its own
    e0, e1 = ev(), ev()
    ctx.saf_pattern_prepare(mask, alpha, rho, logZ)
    torch.cuda.synchronize()
    e0.record()
    ctx.saf_pattern_prepare(mask, alpha, rho, logZ)
    e1.record()
    torch.cuda.synchronize()
    prepare_ms = e0.elapsed_time(e1)

    def step(m, c=ctx, al=alpha, rh=rho, lz=logZ):
        c.saf_hybrid_attn_fwd(prob, Q, K, V, m, al, rh, lz, O, LSE)
        if bwd:
            c.saf_hybrid_attn_bwd(prob, Q, K, V, O, dO, LSE, m, al, rh, lz, dQ, dK, dV)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(m, steps, **kw):
        barrier()
        a, b = ev(), ev()
        a.record()
        for _ in range(steps):
            step(m, **kw)
        b.record()
        barrier()
        return a.elapsed_time(b) / steps

    for _ in range(max(args.warmup, 3)):
        step(mask)
        step(mask0)
    torch.cuda.synchronize()

    # ---- headline: the K-step region, timed `repeats` times; clocks sampled while the regions run
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    flops_local = wl.flops()
    regions = []
    for _ in range(max(args.repeats, 1)):
        # an idle gap first: every region is then a burst measurement like a single K-step run (and like the burst
        # peak the roofline divides by); without it the later regions run into the board's power cap (~10 % slower)
        time.sleep(args.region_gap)
        regions.append(sd.max_over_ranks(timed(mask, args.steps), dev))       # slowest rank of each region
    time.sleep(args.region_gap)
    ms = float(np.median(regions))
    value = sd.sum_over_ranks(flops_local, dev) / (ms * 1e-3) / 1e12

    # ---- one more K-step region with an event pair around every kernel (the roofline's kernel durations)
    ctx.saf_set_profiling(True)
    kinds = (saf.SAF_KERNEL_FWD, saf.SAF_KERNEL_BWD, saf.SAF_KERNEL_BWD_PREP, saf.SAF_KERNEL_SCALE)
    for k in kinds:
        ctx.saf_get_kernel_time(k)
    ms_events = sd.max_over_ranks(timed(mask, args.steps), dev)
    k_fwd, k_bwd, k_prep, k_scale = (ctx.saf_get_kernel_time(k) for k in kinds)
    ctx.saf_set_profiling(False)
    code, detail = ctx.saf_last_device_status()
    if code != saf.SAF_OK:
        raise RuntimeError(f"device status {code} detail {detail:#x}")

    # optional extra outside the headline: gradients of the compact patterns (trainable-pattern control)
    pgrad_ms = None
    if bwd and len(wl.frozen_heads):
        da, dr = torch.empty_like(alpha), torch.empty_like(alpha)
        for _ in range(3):
            ctx.saf_pattern_grad(prob, V, O, dO, mask, alpha, rho, logZ, da, dr)
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record()
        for _ in range(10):
            ctx.saf_pattern_grad(prob, V, O, dO, mask, alpha, rho, logZ, da, dr)
        b.record()
        torch.cuda.synchronize()
        pgrad_ms = a.elapsed_time(b) / 10

    # extra: the same step recorded into a CUDA graph and replayed
    graph_ms = None
    try:
        gs = torch.cuda.Stream()
        gs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(gs):
            step(mask)
            cg = torch.cuda.CUDAGraph()
            with torch.cuda.graph(cg, stream=gs):
                step(mask)
            for _ in range(3):
                cg.replay()
            a, b = ev(), ev()
            a.record(gs)
            for _ in range(max(args.steps, 5)):
                cg.replay()
            b.record(gs)
        torch.cuda.synchronize()
        graph_ms = a.elapsed_time(b) / max(args.steps, 5)
    except Exception:                                                  # not part of the contract: report null
        graph_ms = None
        torch.cuda.synchronize()

    # ---- speedup vs the same library with zero frozen heads: interleaved A B B A, plus an A/A control that must
    # read 1.00 within 1 % or the comparison is discarded and taken again (the paper's rule; at most five times)
    reps = max(5, args.steps)
    for aa_attempt in range(1, 6):
        def burst(m):                                     # every region a burst after an idle gap, like the headline's
            time.sleep(args.region_gap)
            return timed(m, reps)
        a1 = burst(mask)
        b1 = burst(mask0)
        b2 = burst(mask0)
        a2 = burst(mask)
        c1 = burst(mask)
        c2 = burst(mask)
        speedup = (b1 + b2) / (a1 + a2)
        aa_control = c1 / c2
        if world > 1 or abs(aa_control - 1.0) <= 0.01:     # (ranks must take the same number of timed runs)
            break
    aa_ok = abs(aa_control - 1.0) <= 0.01

    # ---- frozen-rate sweep at this shape (config 1 only): nested frozen sets of one seeded permutation
    sweep = None
    if args.config == 1 and world == 1:
        sweep = []
        ctx_s = saf.Context(local_rank)
        full = si.generate(si.Workload("sweep-patterns", 1, wl.H, 8, wl.D, tuple(range(wl.H)), wl.rho_slope,
                                       Tp=wl.stored_len, seed=wl.seed + 1))
        al_s, rh_s = torch.from_numpy(full.alpha).to(dev), torch.from_numpy(full.rho).to(dev)
        lz_s = torch.zeros_like(al_s)
        for nf in (0, 3, 6, 9, 12):
            wls = si.config(3, nf)
            m = wls.mask
            ctx_s.saf_pattern_prepare(m, al_s, rh_s, lz_s)
            kw = dict(c=ctx_s, al=al_s, rh=rh_s, lz=lz_s)
            for _ in range(3):
                step(m, **kw)
            ts = []
            for _ in range(3):
                time.sleep(args.region_gap)                  # burst regions, as for the headline
                ts.append(timed(m, reps, **kw))
            t = float(np.median(ts))
            tf = wls.flops() / (t * 1e-3) / 1e12
            sweep.append({"frozen_heads": nf, "frozen_fraction": nf / wl.H, "ms_per_step": t, "tflops": tf})
        code, detail = ctx_s.saf_last_device_status()
        if code != saf.SAF_OK:
            raise RuntimeError(f"sweep: device status {code} detail {detail:#x}")
        t0 = sweep[0]["ms_per_step"]
        for r in sweep:
            r["speedup_vs_0pct_frozen"] = t0 / r["ms_per_step"]
        ctx_s.close()
        step(mask)                                           # leave the outputs consistent with `mask`

    # the sampler ran through the timed regions and the interleaved repeats of the same step
    clocks = sampler.stop() if rank == 0 else None
    fwd_only = None
    if bwd:
        barrier()
        a, b = ev(), ev()
        a.record()
        for _ in range(reps):
            ctx.saf_hybrid_attn_fwd(prob, Q, K, V, mask, alpha, rho, logZ, O, LSE)
        b.record()
        barrier()
        fwd_only = a.elapsed_time(b) / reps
    ctx.saf_hybrid_attn_fwd(prob, Q, K, V, mask, alpha, rho, logZ, O, LSE)   # leave O/LSE consistent with `mask`

    # ---- end to end through host buffers (pinned): inputs copied in, every output copied back
    hO = torch.empty_like(hostQ).pin_memory()
    hLSE = torch.empty(wl.B, wl.H, wl.T).pin_memory()
    nel = wl.B * wl.H * wl.T * wl.D
    if bwd:
        hdQ, hdK, hdV = (torch.empty(x.shape, dtype=torch.float32).pin_memory() for x in (Q, K, V))
        ctx2 = saf.Context(local_rank)
        probh = saf.make_problem(hostQ, wl.stored_len, k_like=hostK, v_like=hostV, kv_group=wl.kv_group)

        def step_host(prepare):
            ctx2.saf_hybrid_attn_step_host(probh, hostQ, hostK, hostV, hostdO, mask, alpha_h, rho_h, prepare, hO,
                                           hLSE, hdQ, hdK, hdV)
        h2d = (2 * nel + K.numel() + V.numel()) * 2
        d2h = nel * 2 + wl.B * wl.H * wl.T * 4 + (nel + K.numel() + V.numel()) * 4
    else:
        # forward-only workload: the device entry point between pinned-memory copies of Q, K, V in and O, LSE out
        def step_host(prepare):
            Q.copy_(hostQ, non_blocking=True)
            K.copy_(hostK, non_blocking=True)
            V.copy_(hostV, non_blocking=True)
            ctx.saf_hybrid_attn_fwd(prob, Q, K, V, mask, alpha, rho, logZ, O, LSE)
            hO.copy_(O, non_blocking=True)
            hLSE.copy_(LSE, non_blocking=True)
        h2d = (nel + K.numel() + V.numel()) * 2
        d2h = nel * 2 + wl.B * wl.H * wl.T * 4

    step_host(1)
    step_host(0)
    e2e_steps = max(2, min(args.steps, 5))
    barrier()
    a, b = ev(), ev()
    a.record()
    for _ in range(e2e_steps):
        step_host(0)
    b.record()
    barrier()
    e2e_ms_local = a.elapsed_time(b) / e2e_steps
    e2e_rate, e2e_ms = sd.whole_job_rate(flops_local, e2e_ms_local, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    hf = len(wl.frozen_heads)
    fwd_flops = wl.flops(backward=False)
    fwd_ms = k_fwd[0] / max(k_fwd[1], 1)
    fwd_name = "saf_fwd64_kernel" if wl.D == 64 else "saf_fwd_kernel<128>"
    fwd_entry = {"launch_ms": fwd_ms, "achieved": fwd_flops / (fwd_ms * 1e-3) / 1e12,
                 "frac": fwd_flops / (fwd_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    others = {}
    if k_scale[1]:
        others["saf_scale_rows_kernel"] = {"launch_ms": k_scale[0] / k_scale[1]}
    if bwd:
        dom_name = "saf_bwd_kernel" if wl.D == 64 else "saf_bwd128_kernel"
        dom_flops = wl.B * wl.D * wl.T * (wl.T + 1) * (5 * (wl.H - hf) + hf)
        dom_ms = k_bwd[0] / max(k_bwd[1], 1)
        others[fwd_name] = fwd_entry
        others["saf_bwd_prep_kernel"] = {"launch_ms": k_prep[0] / max(k_prep[1], 1)}
    else:
        dom_name, dom_flops, dom_ms = fwd_name, fwd_flops, fwd_ms
    kernel_sum_ms = (k_fwd[0] + k_bwd[0] + k_prep[0] + k_scale[0]) / max(k_fwd[1], 1)
    achieved = dom_flops / (dom_ms * 1e-3) / 1e12
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "roofline_traffic.json")
    if os.path.exists(tpath):
        with open(tpath) as f:
            traffic = json.load(f).get(f"{dom_name}@{wl.name}")
    roofline = {"bound": "tensor", "kernel": dom_name, "achieved": achieved, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "traffic": traffic,
                "peak_source": f"{peaks['source']} bf16 burst (MEASURED_PEAKS.json)" if peaks["source"] == "measured"
                else "fallback 1590 TFLOP/s",
                "launch_ms": dom_ms, "flops_per_launch": dom_flops,
                "timed_in": "a K-step region of the same steps with an event pair around every kernel",
                "kernel_sum_ms_per_step": kernel_sum_ms, "other_kernels": others}

    # context for the roofline's denominator: a library bf16 GEMM (8192^3) timed in this same process
    live_gemm = None
    try:
        n = 8192
        ga = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
        gb_ = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
        for _ in range(3):
            torch.matmul(ga, gb_)
        a, b = ev(), ev()
        a.record()
        for _ in range(10):
            torch.matmul(ga, gb_)
        b.record()
        torch.cuda.synchronize()
        live_gemm = 2.0 * n ** 3 * 10 / (a.elapsed_time(b) * 1e-3) / 1e12
        del ga, gb_
    except Exception:                                                  # context only
        live_gemm = None
        torch.cuda.synchronize()

    fit = None if (args.no_fit or not bwd) else fit_leg(ctx, saf, wl, peaks, dev)
    calib = None
    if not args.no_fit and bwd:
        # normalisers of the all-ordinary layer (calibration precedes replacement)
        ctx.saf_hybrid_attn_fwd(prob, Q, K, V, mask0, alpha, rho, logZ, O, LSE)
        calib = calib_leg(ctx, saf, wl, prob, Q, K, LSE, peaks, dev)
    cpu_v, cpu_desc, cpu_threads, _ = oracle_sample(si.config(args.config), budget_s=args.ref_budget)
    # forward kernel, the V staging kernel of the frozen heads, backward preparation and backward kernel
    launches_per_step = 1 + (1 if hf else 0) + (2 if bwd else 0)
    tensors_gb = ((4 * 2 + 3 * 4) if bwd else 4 * 2) * nel / 1e9
    line = {
        "metric": METRIC if bwd else "hybrid_attn_fwd_tflops", "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "B": wl.B, "H": wl.H, "kv_heads": wl.H // wl.kv_group, "Hf": hf, "T": wl.T, "D": wl.D,
                   "pass": "fwd+bwd" if bwd else "fwd only",
                   "grad_dtype": "f32", "frozen_fraction": hf / wl.H,
                   "flops_per_step_per_gpu": flops_local,
                   "l2": f"inputs+outputs per step ({tensors_gb:.2f} GB) exceed the 126 MB L2; no explicit flush",
                   "pattern_prepare": "once before the timed steps (static per layer)", "pattern_prepare_ms": prepare_ms,
                   "timed_regions": len(regions), "ms_per_step_regions": regions,
                   "region_gap_s": args.region_gap,
                   "parallelism": f"dp{world} (independent batches, no collective in the layer)"},
        "pct_of_bf16_peak": 100.0 * value / (peaks["bf16_tflops"] * world),
        # (context: the same against the sustained, power-capped peak, which long regions run into)
        "pct_of_bf16_peak_sustained": (100.0 * value / (peaks["bf16_tflops_sustained"] * world)
                                       if peaks.get("bf16_tflops_sustained") else None),
        "ms_per_step_with_kernel_events": ms_events,
        "speedup_vs_0pct_frozen": speedup, "aa_control": aa_control, "aa_attempts": aa_attempt,
        "aa_within_1pct": aa_ok,
        "ms_0pct_frozen": 0.5 * (b1 + b2), "ms_fwd_only": fwd_only, "ms_pattern_grad": pgrad_ms,
        "ms_per_step_cuda_graph": graph_ms,
        "sweep": sweep,
        "e2e": {"value": e2e_rate / 1e12, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        # per step: V scaling + forward kernel, backward preparation (which also stages w dO) + backward kernel;
        # counted over the timed regions that give ms_per_step
        "gpu_launches": launches_per_step * args.steps * len(regions),
        "gpu_launches_per_step": launches_per_step,
        "clocks": clocks,
        "roofline": roofline,
        "peak_context": {"library_bf16_gemm_8192_tflops_live": live_gemm,
                         "measured_peaks_file_bf16_tflops": peaks["bf16_tflops"]},
        "fit": fit,
        "calibration": calib,
        "cpu_baseline": {"value": cpu_v, "unit": UNIT, "cores": cpu_threads, "kind": "oracle", "sample": cpu_desc},
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launch_ranks(args, argv):
    """`--gpus N` without a torchrun environment: start the N ranks here, one process per GPU, with the
    environment torchrun would give them (rendezvous on 127.0.0.1), and pass rank 0's JSON line through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *argv], env=env,
                                      stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    rcs = [procs[0].returncode] + [p.wait() for p in procs[1:]]
    sys.stdout.write(out)
    sys.stdout.flush()
    if any(rcs):
        raise SystemExit(f"ranks exited with {rcs}")


def launcher_selftest(args):
    """What the ranks of `--gpus N` do around the timed steps, without a GPU: rendezvous (gloo), reduce a timing
    (max) and a unit count (sum), rank 0 prints one line.  Run by the CPU tests through the launcher above."""
    import torch.distributed as dist
    from paper_2609_34650_b200 import dist as sd
    rank, _, world = sd.env_world()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rate, ms = sd.whole_job_rate(100.0 * (rank + 1), 1.0 + rank)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"launcher_selftest": True, "n_gpus": world, "units_per_s": rate, "ms": ms}), flush=True)
    dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=5, help="how many times the K-step region is timed (median reported)")
    ap.add_argument("--region-gap", type=float, default=0.3, help="idle seconds before each timed region")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, choices=[1, 2, 4, 5, 6, 7])
    ap.add_argument("--no-fit", action="store_true", help="skip the extra legs that time the one-time fitter and the calibration statistics")
    ap.add_argument("--ref-budget", type=float, default=12.0, help="seconds of CPU-oracle work per sample")
    ap.add_argument("--launcher-selftest", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.impl == "ours" and args.gpus > 1 and "RANK" not in os.environ:
        launch_ranks(args, sys.argv[1:])
    elif args.launcher_selftest:
        launcher_selftest(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
