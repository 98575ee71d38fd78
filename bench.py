#!/usr/bin/env python
"""Benchmark of the ThinK hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic prompts:
  prefill  thinK_score_select + thinK_compact over all layers, then
  decode   `decode_steps` x (thinK_append + thinK_decode_attn) over all layers.
The headline `value` is the effective HBM bandwidth of that pass (algorithmic bytes of the
method / device time); `decode` and `prefill` carry the per-phase figures (us per decode step,
GB/s, fraction of the measured and of the nominal HBM peak).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl reference]

N > 1 runs N independent replicas (the path has no exchange step); launch with torchrun.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2407_21018_b200 import workloads as wl  # noqa: E402

NOMINAL_HBM_GBS = 8000.0
# DRAM bytes (read + write) of ONE launch of the decode kernel from an ncu capture of the current
# kernel (profiles/k_decode_mma_c2_ncu.md); configs without a capture report null.
NCU_DECODE_TRAFFIC_BYTES = {"c2": 879.9e6}
# DRAM bytes of the prefill kernels of one pass (score + compact; profiles/k_*_c2_ncu.md): K crosses HBM twice.
NCU_PREFILL_TRAFFIC_BYTES = {"c2": 1379.9e6}
FALLBACK_HBM_GBS = 6650.0


# --------------------------------------------------------------------------- byte accounting
def prefill_bytes(w: wl.Workload, T: int, Tv: int = 0) -> int:
    """Algorithmic bytes of score + select + compact: read K once, read the window queries, write
    the thinned prefix, the unpruned recent rows (keys and values) and the index list.  With value
    pruning (Tv > 0): V is read once as well and its thinned prefix and channel order are written."""
    e, G, R = w.elem_bytes, w.N_q // w.N_kv, w.recent
    tot = 0
    for S in w.seq_lens:
        S_p = S - R
        per_head = S * w.D * e + w.S_obs * G * w.D * e + S_p * T * e + 2 * R * w.D * e + R * w.D * e + T
        if Tv:
            per_head += S_p * w.D * e + S_p * Tv * e + w.D
        tot += per_head * w.L * w.N_kv
    return tot


def prefill_bytes_evicted(w: wl.Workload, T: int) -> int:
    """Same behind a token-eviction method (`w` = the workload after eviction, seq_lens = kept tokens):
    the kept key rows and their list are read once, the kept value rows are read and written once."""
    e = w.elem_bytes
    return prefill_bytes(w, T) + sum(S * 4 + 2 * (S - w.recent) * w.D * e for S in w.seq_lens) * w.L * w.N_kv


def decode_bytes(w: wl.Workload, T: int, t: int, Tv: int = 0) -> int:
    """Algorithmic bytes of decode step t (t tokens already appended before it): thinned prefix
    keys, unpruned tail keys, all values (prefix rows at Tv channels when values are pruned), index
    list, q in and out."""
    e, R = w.elem_bytes, w.recent
    tot = 0
    for S in w.seq_lens:
        S_p = S - R
        values = (S_p * Tv + (R + t + 1) * w.D) * e + w.D if Tv else (S + t + 1) * w.D * e
        per_head = S_p * T * e + (R + t + 1) * w.D * e + values + T
        tot += per_head * w.L * w.N_kv + 2 * w.L * w.N_q * w.D * e
    return tot


def append_bytes(w: wl.Workload) -> int:
    return 4 * w.B * w.L * w.N_kv * w.D * w.elem_bytes   # k_new, v_new read + written


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx = float(f[2])
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------- the GPU arm
def run_ours(args):
    from paper_2407_21018_b200 import binding as tk   # fails loudly when the CUDA library is missing

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    w = wl.get_config(args.config)
    import dataclasses
    if args.lam is not None:
        w = dataclasses.replace(w, lam=args.lam, name=f"{w.name}-lam{args.lam}")
    nsteps = args.decode_steps if args.decode_steps is not None else w.steps
    tok = None
    if args.kv_size:
        # Sec. 4.1 setting: an upstream eviction method kept kv_size tokens per head; the cache holds those
        src = w
        tok = wl.make_eviction(src, args.kv_size).to(dev)
        w = wl.evicted(src, args.kv_size)
        data = wl.make_prefill(src, device=dev, pad_nan=False)
    else:
        data = wl.make_prefill(w, device=dev, pad_nan=False)
    cfg = tk.make_config(w.B, w.L, w.N_q, w.N_kv, w.D, w.S_max, w.S_obs, w.recent, nsteps, w.lam, w.torch_dtype,
                         lam_v=args.lam_v)
    cache = tk.ThinKCache(cfg, w.seq_lens, device=dev, keep_scores=True)
    T = cache.T
    Tv = cache.T_v if args.lam_v > 0 else 0
    if Tv:
        w = dataclasses.replace(w, name=f"{w.name}-lamv{args.lam_v}")

    K, V, Q = data["K"], data["V"], data["Q_obs"]
    nvar = min(4, max(1, nsteps))
    steps_in = [wl.make_step(w, t, device=dev) for t in range(nvar)]
    out = torch.empty_like(steps_in[0]["q"])
    stream = torch.cuda.current_stream()

    def one_pass(ev=None):
        if ev is not None:
            ev["p0"].record(stream)
        if tok is not None:
            cache.prefill_evicted(Q, K, V, tok)
        elif Tv:
            cache.score_select_kv(Q, K, V)
            cache.compact(K, V)
        elif args.two_pass_prefill:
            cache.score_select(Q, K)
            cache.compact(K, V)
        else:
            cache.prefill(Q, K, V)
        if ev is not None:
            ev["p1"].record(stream)
        for t in range(nsteps):
            s = steps_in[t % nvar]
            if ev is not None:
                ev["s0"][t].record(stream)
            if args.fused_step:
                cache.append_decode(s["k_new"], s["v_new"], s["q"], out=out)   # one call, overlapped launches
                if ev is not None:
                    ev["d0"][t].record(stream)     # (no separate attention time in this mode)
                    ev["d1"][t].record(stream)
                continue
            cache.append(s["k_new"], s["v_new"])
            if args.reprune_every and (t + 1) % args.reprune_every == 0:
                cache.reprune_tail(w.recent)       # App. C.1 control flow: thin the oldest tail blocks
            if ev is not None:
                ev["d0"][t].record(stream)
            cache.decode_attn(s["q"], out=out)
            if ev is not None:
                ev["d1"][t].record(stream)

    def mk_events():
        E = lambda: torch.cuda.Event(enable_timing=True)
        return {"p0": E(), "p1": E(), "d0": [E() for _ in range(nsteps)], "d1": [E() for _ in range(nsteps)],
                "s0": [E() for _ in range(nsteps)]}

    n_warm = args.warmup if args.profile else max(3, args.warmup)
    for _ in range(n_warm):
        one_pass()
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    evs = [mk_events() for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    torch.cuda.synchronize()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(args.steps):
        one_pass(evs[k])
    t_end.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    from paper_2407_21018_b200 import replicas
    total_ms, _ = replicas.job_time_and_work(t_start.elapsed_time(t_end), 1.0, device=dev)   # slowest replica
    assert cache.device_error() == 0

    prefill_ms = [e["p0"].elapsed_time(e["p1"]) for e in evs]
    dec_ms = [[e["d0"][t].elapsed_time(e["d1"][t]) for t in range(nsteps)] for e in evs]
    # whole decode step (append + attention), whichever way it was launched
    step_us = 1e3 * sum(e["s0"][t].elapsed_time(e["d1"][t]) for e in evs for t in range(nsteps)) / max(1, args.steps * nsteps)
    if args.fused_step:
        dec_ms = [[e["s0"][t].elapsed_time(e["d1"][t]) for t in range(nsteps)] for e in evs]
    dec_mean_us = 1e3 * sum(sum(r) for r in dec_ms) / max(1, args.steps * nsteps)
    dec_all = sorted(1e3 * x for r in dec_ms for x in r) or [0.0]
    pre_all = sorted(1e3 * x for x in prefill_ms)
    dec_bytes = [decode_bytes(w, T, t, Tv) for t in range(nsteps)]
    dec_bytes_mean = sum(dec_bytes) / max(1, nsteps)
    pre_b = prefill_bytes_evicted(w, T) if tok is not None else prefill_bytes(w, T, Tv)
    pre_us = 1e3 * sum(prefill_ms) / len(prefill_ms)
    pass_bytes = pre_b + sum(dec_bytes) + nsteps * append_bytes(w)
    ms_per_step = total_ms / args.steps
    value = world * pass_bytes / (ms_per_step * 1e-3) / 1e9

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    dec_gbs = dec_bytes_mean / (dec_mean_us * 1e-6) / 1e9 if nsteps else 0.0
    pre_gbs = pre_b / (pre_us * 1e-6) / 1e9

    # ---- the same pass with thinK_append_decode (one call per decode step, attention overlapped with the append):
    # reported next to the headline, which keeps the two calls apart so that the attention kernel can be timed alone
    fused = None
    if not args.fused_step and nsteps > 0 and not args.reprune_every:
        saved, args.fused_step = args.fused_step, True
        one_pass()
        torch.cuda.synchronize()
        fa, fb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fev = [mk_events() for _ in range(3)]
        fa.record(stream)
        for e in fev:
            one_pass(e)
        fb.record(stream)
        torch.cuda.synchronize()
        args.fused_step = saved
        f_ms = fa.elapsed_time(fb) / len(fev)
        f_step = 1e3 * sum(e["s0"][t].elapsed_time(e["d1"][t]) for e in fev for t in range(nsteps)) / (len(fev) * nsteps)
        fused = {"ms_per_pass": f_ms, "value_GBps": pass_bytes / (f_ms * 1e-3) / 1e9, "step_us_append_plus_attn": f_step}

    # ---- end to end: inputs start in pinned host memory, results are read back every step
    e2e = None
    if not args.no_e2e:
        hK, hV, hQ = (x.cpu().pin_memory() for x in (K, V, Q))
        hs = [{k: v.cpu().pin_memory() for k, v in s.items()} for s in steps_in]
        hout = torch.empty_like(out, device="cpu").pin_memory()
        dq, dk, dv = (torch.empty_like(steps_in[0][k]) for k in ("q", "k_new", "v_new"))
        n_e2e = max(1, min(args.steps, 3))

        def e2e_pass():
            K.copy_(hK, non_blocking=True)
            V.copy_(hV, non_blocking=True)
            Q.copy_(hQ, non_blocking=True)
            if tok is not None:
                cache.prefill_evicted(Q, K, V, tok)
            else:
                cache.prefill(Q, K, V)
            for t in range(nsteps):
                s = hs[t % nvar]
                dq.copy_(s["q"], non_blocking=True)
                dk.copy_(s["k_new"], non_blocking=True)
                dv.copy_(s["v_new"], non_blocking=True)
                cache.append_decode(dk, dv, dq, out=out)
                hout.copy_(out, non_blocking=True)
        e2e_pass()
        torch.cuda.synchronize()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_pass()
        b.record(stream)
        torch.cuda.synchronize()
        e_ms, _ = replicas.job_time_and_work(a.elapsed_time(b) / n_e2e, 1.0, device=dev)
        h2d = sum(x.numel() * x.element_size() for x in (hK, hV, hQ)) + \
            nsteps * sum(v.numel() * v.element_size() for v in hs[0].values())
        d2h = nsteps * hout.numel() * hout.element_size()
        e2e = {"value": world * pass_bytes / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_sample(w, budget_s=args.cpu_budget)
        cpu.pop("sizing", None)

    if rank == 0:
        line = {
            "metric": "ThinK hot path effective HBM GB/s (prefill score+select+compact, then decode append+attn; "
                      "algorithmic bytes / device time)",
            "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": n_warm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": f"{w.name}: B={w.B} S={list(w.seq_lens) if len(set(w.seq_lens)) > 1 else w.seq_lens[0]} "
                                   f"L={w.L} heads={w.N_q}q/{w.N_kv}kv D={w.D} S_obs={w.S_obs} S_recent={w.recent} "
                                   f"lambda={w.lam} T={T}" + (f" lambda_v={args.lam_v} T_v={Tv}" if Tv else "") +
                                   f" decode_steps={nsteps}",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2 (K, V and the caches are each several L2 sizes)"},
            "decode": {"step_us_append_plus_attn": step_us, "fused_step": bool(args.fused_step),
                       "us_per_step": dec_mean_us, "us_median": dec_all[len(dec_all) // 2], "us_min": dec_all[0],
                       "GBps": dec_gbs, "frac_of_measured": dec_gbs / peak,
                       "frac_of_nominal_8TBps": dec_gbs / NOMINAL_HBM_GBS, "bytes_per_step": dec_bytes_mean},
            "prefill": {"us": pre_us, "us_median": pre_all[len(pre_all) // 2], "us_min": pre_all[0], "GBps": pre_gbs, "frac_of_measured": pre_gbs / peak,
                        "frac_of_nominal_8TBps": pre_gbs / NOMINAL_HBM_GBS, "bytes": pre_b,
                        "dram_bytes_ncu": NCU_PREFILL_TRAFFIC_BYTES.get(w.name),
                        "dram_GBps": (NCU_PREFILL_TRAFFIC_BYTES[w.name] / (pre_us * 1e-6) / 1e9
                                      if w.name in NCU_PREFILL_TRAFFIC_BYTES else None)},
            "roofline": {"kernel": "k_decode_mma" if w.dtype == "bf16" else "k_decode_generic", "bound": "hbm", "achieved": dec_gbs, "peak": peak,
                         "peak_source": f"of {peak_src}", "unit": "GB/s", "frac": dec_gbs / peak,
                         "traffic": NCU_DECODE_TRAFFIC_BYTES.get(w.name), "traffic_unit": "bytes per launch"},
            "fused_step_variant": fused,
            "clocks": clocks,
            "e2e": e2e,
            "gpu_launches": args.steps * (2 + (1 if w.recent > 0 else 0) + (1 if tok is not None else 0) + (2 if Tv else 0) + 2 * nsteps
                                          + (nsteps // args.reprune_every if args.reprune_every else 0)),
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# --------------------------------------------------------------------------- the oracle arm
def oracle_sample(w: wl.Workload, budget_s: float = 20.0, sizing=None):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: a few layers of
    the same prompts and a few decode steps, sized from a short probe so that it ends in about
    `budget_s` seconds.  Reported in the benchmark's unit (algorithmic bytes / wall time)."""
    import numpy as np
    from oracle import think_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = 1
    T = orc.kept_channels(w.lam, w.D)

    def run(L, B, steps):
        ws = wl.shrink(w, L=L, B=B, steps=steps)
        data = wl.make_prefill(ws, device="cpu")
        K64, V64, Q64 = (data[k].to(torch.float64).numpy() for k in ("K", "V", "Q_obs"))
        st = [wl.make_step(ws, t, device="cpu") for t in range(steps)]
        st = [{k: v.to(torch.float64).numpy() for k, v in s.items()} for s in st]
        o = orc.ThinKOracle(ws.B, ws.L, ws.N_q, ws.N_kv, ws.D, ws.seq_lens, ws.S_obs, ws.recent, ws.lam)
        t0 = time.perf_counter()
        o.score_select(Q64, K64)
        o.compact(K64, V64)
        t1 = time.perf_counter()
        for t in range(steps):
            o.append(st[t]["k_new"], st[t]["v_new"])
            o.decode_attn(st[t]["q"])
        t2 = time.perf_counter()
        nbytes = prefill_bytes(ws, T) + sum(decode_bytes(ws, T, t) for t in range(steps)) + steps * append_bytes(ws)
        return t2 - t0, t1 - t0, t2 - t1, nbytes, ws

    if sizing is None:
        run(1, 1, 1)                                 # warm-up of the numeric library's threads
        _, pre1, dec1, _, _ = run(1, 1, 1)           # one layer, one decode step: cost of either phase per layer
        steps = int(max(1, min(w.steps, 16)))
        if budget_s < 4 * (pre1 + steps * dec1):     # small budgets: fewer decode steps before fewer layers
            steps = int(max(1, min(steps, (budget_s / 2 - pre1) / max(dec1, 1e-6))))
        L = int(max(1, min(w.L, budget_s / max(pre1 + steps * dec1, 1e-3))))
    else:
        L, steps = sizing
    dt, dt_pre, dt_dec, nbytes, ws = run(L, 1, steps)
    return {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": f"{ws.name}: B=1 of {w.B}, L={L} of {w.L}, S={ws.seq_lens[0]}, {steps} decode steps; "
                      f"prefill {dt_pre:.2f} s, decode {dt_dec / steps * 1e3:.1f} ms/step",
            "seconds": dt, "sizing": (L, steps)}


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    w = wl.get_config(args.config)
    vals = []
    last = None
    # the whole run is held to about two minutes: one probe sizes the sample, every step then times that sample
    per = max(0.5, min(60.0, 120.0 / max(1, args.steps + args.warmup)))
    sizing = None
    for i in range(args.warmup + args.steps):
        last = oracle_sample(w, budget_s=per, sizing=sizing)
        sizing = last["sizing"]
        if i >= args.warmup:
            vals.append(last)
    v = sum(x["value"] for x in vals) / len(vals)
    ms = 1e3 * sum(x["seconds"] for x in vals) / len(vals)
    line = {"impl": "reference",
            "metric": "ThinK hot path effective HBM GB/s (prefill score+select+compact, then decode append+attn; "
                      "algorithmic bytes / device time)",
            "value": v, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", 1)), "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name} (bounded sample per step: {last['sample']})"},
            "cpu_baseline": {"value": v, "unit": "GB/s", "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2", choices=sorted(wl.CONFIGS))
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--reprune-every", type=int, default=0,
                    help="call thinK_reprune_tail(keep_recent=S_recent) every N decode steps (0 = never); byte "
                         "accounting stays that of the un-repruned path")
    ap.add_argument("--kv-size", type=int, default=0,
                    help="prefill behind a token-eviction method that kept this many tokens per head "
                         "(thinK_prefill_evicted on seeded kept-token lists); 0 = no eviction")
    ap.add_argument("--lam-v", type=float, default=0.0,
                    help="also prune the value channels with this ratio (App. D); 0 = values untouched")
    ap.add_argument("--fused-step", action="store_true",
                    help="decode steps through thinK_append_decode (append + attention in one call, the attention "
                         "launched as a programmatic dependent); decode.us_per_step is then the whole step")
    ap.add_argument("--lam", type=float, default=None, help="override the config's pruning ratio (c5 sweep)")
    ap.add_argument("--two-pass-prefill", action="store_true",
                    help="prefill through thinK_score_select + thinK_compact (two passes over K) instead of thinK_prefill")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--profile", action="store_true",
                    help="for runs under ncu: take --warmup literally (fewer launches before the captured ones)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
