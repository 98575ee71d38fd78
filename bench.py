#!/usr/bin/env python
"""Benchmark of the ThinK hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic prompts:
  prefill  thinK_prefill (score + select + compact) over all layers, then
  decode   `decode_steps` x (thinK_append + thinK_decode_attn) over all layers.
The headline `value` is the effective HBM bandwidth of that pass (algorithmic bytes of the
method / device time); `decode` and `prefill` carry the per-phase figures (us per decode step,
GB/s, fraction of the measured and of the nominal HBM peak).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config all|c2|c3|c4|c5|c1] [--impl reference]

With `--config all` (the default) the four bf16 configs run one after the other: the headline keys
describe the largest one (c4: 17-19 GB per decode step), `per_config` carries every config's figures.
N > 1 runs N independent replicas (the path has no exchange step): under torchrun as launched, or, when
started as a single process, by re-launching itself as N ranks.
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
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "c4"                       # the largest single-GPU configuration
ALL_CONFIGS = ("c2", "c3", "c5", "c4")
KERNEL_SOURCE = {"k_decode_mma": "k_decode_mma.cu", "k_decode_generic": "k_decode.cu", "k_colnorm_score_select": "k_score.cu",
                 "k_compact_bf16": "k_compact.cu"}


def ncu_traffic(config: str, kernel: str):
    """DRAM bytes (read + write) of ONE launch of `kernel` on `config` from the table of ncu captures
    (one line per capture: config, kernel, bytes, sha1 of the kernel's source file when it was taken).
    None without a capture, and None once the source file has changed since."""
    import hashlib
    table = os.path.join(ROOT, "profiles", "ncu_dram_bytes.txt")
    src = os.path.join(ROOT, "paper_2407_21018_b200", "csrc", KERNEL_SOURCE.get(kernel, ""))
    if not (os.path.exists(table) and os.path.isfile(src)):
        return None
    sha = hashlib.sha1(open(src, "rb").read()).hexdigest()
    for line in open(table):
        f = line.split()
        if len(f) >= 4 and not line.startswith("#") and f[0] == config and f[1] == kernel and f[3] == sha:
            return float(f[2])
    return None


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




# --------------------------------------------------------------------------- one config on this rank's GPU
def hbm_peak():
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        return float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def measure_config(args, name, passes, warm, dev, world, barrier, do_e2e, sample_clocks):
    """Runs `warm` untimed and `passes` timed passes of the whole path on config `name` and returns its
    figures (device times by CUDA events on the launching stream; job time = slowest replica)."""
    import dataclasses
    from paper_2407_21018_b200 import binding as tk   # fails loudly when the CUDA library is missing
    from paper_2407_21018_b200 import replicas

    w = wl.get_config(name)
    if args.layers:
        w = wl.shrink(w, L=args.layers)            # fewer layers of the same shape (profiler captures): not a bench workload
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

    def one_pass(ev=None, fused=False):
        if ev is not None:
            ev["p0"].record(stream)
        if tok is not None:
            cache.prefill_evicted(Q, K, V, tok)
        elif args.two_call_prefill:
            if Tv:
                cache.score_select_kv(Q, K, V)
            else:
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
            if fused:
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

    for _ in range(warm):
        one_pass(fused=args.fused_step)
    torch.cuda.synchronize()

    evs = [mk_events() for _ in range(passes)]
    sampler = ClockSampler(dev.index) if sample_clocks else None
    if sampler:
        sampler.start()
    barrier()
    torch.cuda.synchronize()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(passes):
        one_pass(evs[k], fused=args.fused_step)
    t_end.record(stream)
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop() if sampler else None
    total_ms, _ = replicas.job_time_and_work(t_start.elapsed_time(t_end), 1.0, device=dev)   # slowest replica
    assert cache.device_error() == 0

    prefill_ms = [e["p0"].elapsed_time(e["p1"]) for e in evs]
    dec_ms = [[e["d0"][t].elapsed_time(e["d1"][t]) for t in range(nsteps)] for e in evs]
    # whole decode step (append + attention), whichever way it was launched
    step_us = 1e3 * sum(e["s0"][t].elapsed_time(e["d1"][t]) for e in evs for t in range(nsteps)) / max(1, passes * nsteps)
    if args.fused_step:
        dec_ms = [[e["s0"][t].elapsed_time(e["d1"][t]) for t in range(nsteps)] for e in evs]
    dec_mean_us = 1e3 * sum(sum(r) for r in dec_ms) / max(1, passes * nsteps)
    dec_all = sorted(1e3 * x for r in dec_ms for x in r) or [0.0]
    pre_all = sorted(1e3 * x for x in prefill_ms)
    dec_bytes = [decode_bytes(w, T, t, Tv) for t in range(nsteps)]
    dec_bytes_mean = sum(dec_bytes) / max(1, nsteps)
    pre_b = prefill_bytes_evicted(w, T) if tok is not None else prefill_bytes(w, T, Tv)
    pre_us = 1e3 * sum(prefill_ms) / len(prefill_ms)
    pass_bytes = pre_b + sum(dec_bytes) + nsteps * append_bytes(w)
    ms_per_pass = total_ms / passes
    value = world * pass_bytes / (ms_per_pass * 1e-3) / 1e9

    peak, peak_src = hbm_peak()
    dec_gbs = dec_bytes_mean / (dec_mean_us * 1e-6) / 1e9 if nsteps else 0.0
    pre_gbs = pre_b / (pre_us * 1e-6) / 1e9
    dec_kernel = "k_decode_mma" if w.dtype == "bf16" else "k_decode_generic"
    base = name if (args.lam is None and not args.kv_size and not Tv) else None      # captures exist for the plain configs
    pre_traffic = None
    if base and w.dtype == "bf16":
        parts = [ncu_traffic(base, "k_colnorm_score_select"), ncu_traffic(base, "k_compact_bf16")]
        pre_traffic = sum(parts) if all(x is not None for x in parts) else None

    # ---- the same pass with thinK_append_decode (one call per decode step, attention overlapped with the append):
    # reported next to the headline, which keeps the two calls apart so that the attention kernel can be timed alone
    fused = None
    if not args.fused_step and nsteps > 0 and not args.reprune_every:
        one_pass(fused=True)
        torch.cuda.synchronize()
        fa, fb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fev = [mk_events() for _ in range(2)]
        fa.record(stream)
        for e in fev:
            one_pass(e, fused=True)
        fb.record(stream)
        torch.cuda.synchronize()
        f_ms = fa.elapsed_time(fb) / len(fev)
        f_step = 1e3 * sum(e["s0"][t].elapsed_time(e["d1"][t]) for e in fev for t in range(nsteps)) / (len(fev) * nsteps)
        fused = {"ms_per_pass": f_ms, "value_GBps": pass_bytes / (f_ms * 1e-3) / 1e9, "step_us_append_plus_attn": f_step}

    # ---- end to end: inputs start in pinned host memory, results are read back every step
    e2e = None
    if do_e2e:
        try:
            pin = lambda x: torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x)
            hK, hV, hQ = pin(K), pin(V), pin(Q)
            hs = [{k: pin(v) for k, v in s.items()} for s in steps_in]
            hout = torch.empty(out.shape, dtype=out.dtype, pin_memory=True)
            n_e2e = max(1, min(passes, 5))
            # Two sets of input tensors on the device: while pass i computes from one, the copy stream brings pass
            # i + 1's prompt and its per-step inputs into the other (what a server does with the next batch).  Every
            # pass still copies all its inputs -- the prompt tensors and every decode step's q, k_new, v_new -- from
            # pinned host memory inside the timed region; nothing but kernels and the read-back of each step's result
            # runs on the compute stream (host-to-device copies queued there would wait behind the next prompt on the
            # one copy engine).
            def step_buffers():
                return {k: torch.empty((nsteps,) + tuple(steps_in[0][k].shape), dtype=steps_in[0][k].dtype, device=dev)
                        for k in ("q", "k_new", "v_new")}
            sets = [(K, V, Q, step_buffers())]
            try:
                sets.append((torch.empty_like(K), torch.empty_like(V), torch.empty_like(Q), step_buffers()))
            except RuntimeError:
                pass                                   # no room for a second set: passes run back to back
            copy_stream = torch.cuda.Stream(device=dev)
            ready = [torch.cuda.Event() for _ in sets]
            free = [torch.cuda.Event() for _ in sets]

            def issue_copy(i):
                dK, dV, dQ, dS = sets[i]
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(free[i])    # the pass that used this set has finished
                    dK.copy_(hK, non_blocking=True)
                    dV.copy_(hV, non_blocking=True)
                    dQ.copy_(hQ, non_blocking=True)
                    for t in range(nsteps):
                        for k in ("q", "k_new", "v_new"):
                            dS[k][t].copy_(hs[t % nvar][k], non_blocking=True)
                    ready[i].record(copy_stream)

            def compute(i):
                dK, dV, dQ, dS = sets[i]
                stream.wait_event(ready[i])
                if tok is not None:
                    cache.prefill_evicted(dQ, dK, dV, tok)
                else:
                    cache.prefill(dQ, dK, dV)
                for t in range(nsteps):
                    cache.append_decode(dS["k_new"][t], dS["v_new"][t], dS["q"][t], out=out)
                    hout.copy_(out, non_blocking=True)
                free[i].record(stream)

            def e2e_run(n):
                for ev in free:
                    ev.record(stream)
                copy_stream.wait_stream(stream)        # the first copy starts inside the timed region
                issue_copy(0)
                for ps in range(n):
                    if ps + 1 < n and len(sets) > 1:
                        issue_copy((ps + 1) % len(sets))
                    compute(ps % len(sets))
                    if ps + 1 < n and len(sets) == 1:
                        issue_copy(0)
                stream.wait_stream(copy_stream)

            e2e_run(1)
            torch.cuda.synchronize()
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            e2e_run(n_e2e)
            b.record(stream)
            torch.cuda.synchronize()
            e_ms, _ = replicas.job_time_and_work(a.elapsed_time(b) / n_e2e, 1.0, device=dev)
            h2d = sum(x.numel() * x.element_size() for x in (hK, hV, hQ)) + \
                nsteps * sum(v.numel() * v.element_size() for v in hs[0].values())
            d2h = nsteps * hout.numel() * hout.element_size()
            e2e = {"value": world * pass_bytes / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "ms_per_step": e_ms,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e, "workload": w.name,
                   "pipelined": len(sets) > 1}
            del hK, hV, hQ
        except RuntimeError as ex:          # pinned host memory for the prompt tensors could not be had
            e2e = {"value": None, "unit": "GB/s", "unavailable": str(ex).splitlines()[0][:200]}

    launches = passes * ((3 if Tv else 2) + (1 if w.recent > 0 else 0) + (1 if tok is not None else 0) + (1 if Tv else 0)
                         + 2 * nsteps + (nsteps // args.reprune_every if args.reprune_every else 0))
    res = {
        "workload": f"{w.name}: B={w.B} S={list(w.seq_lens) if len(set(w.seq_lens)) > 1 else w.seq_lens[0]} "
                    f"L={w.L} heads={w.N_q}q/{w.N_kv}kv D={w.D} S_obs={w.S_obs} S_recent={w.recent} "
                    f"lambda={w.lam} T={T}" + (f" lambda_v={args.lam_v} T_v={Tv}" if Tv else "") +
                    f" decode_steps={nsteps}",
        "value": value, "unit": "GB/s", "passes": passes, "warmup": warm, "ms_per_pass": ms_per_pass, "dtype": w.dtype,
        "decode": {"step_us_append_plus_attn": step_us, "fused_step": bool(args.fused_step),
                   "us_per_step": dec_mean_us, "us_median": dec_all[len(dec_all) // 2], "us_min": dec_all[0],
                   "GBps": dec_gbs, "frac_of_measured": dec_gbs / peak,
                   "frac_of_nominal_8TBps": dec_gbs / NOMINAL_HBM_GBS, "bytes_per_step": dec_bytes_mean},
        "prefill": {"us": pre_us, "us_median": pre_all[len(pre_all) // 2], "us_min": pre_all[0], "GBps": pre_gbs,
                    "frac_of_measured": pre_gbs / peak, "frac_of_nominal_8TBps": pre_gbs / NOMINAL_HBM_GBS, "bytes": pre_b,
                    "call": "thinK_score_select + thinK_compact" if args.two_call_prefill else "thinK_prefill",
                    "dram_bytes_ncu": pre_traffic,
                    "dram_GBps": pre_traffic / (pre_us * 1e-6) / 1e9 if pre_traffic else None},
        "roofline": {"kernel": dec_kernel, "bound": "hbm", "achieved": dec_gbs, "peak": peak,
                     "peak_source": f"of {peak_src}", "unit": "GB/s", "frac": dec_gbs / peak,
                     "traffic": ncu_traffic(base, dec_kernel) if base else None, "traffic_unit": "bytes per launch"},
        "fused_step_variant": fused, "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
    }
    cache.close()
    del cache, data, K, V, Q, steps_in, out
    torch.cuda.empty_cache()
    return res, w


# --------------------------------------------------------------------------- the oracle on host cores
def _cuda_path_on_sample(ws, data, steps_in):
    """The CUDA path on the oracle's sample (outside any timed region): kept channels and attention outputs."""
    from paper_2407_21018_b200 import binding as tk
    dev = torch.device("cuda", torch.cuda.current_device())
    cfg = tk.make_config(ws.B, ws.L, ws.N_q, ws.N_kv, ws.D, ws.S_max, ws.S_obs, ws.recent, max(1, len(steps_in)),
                         ws.lam, ws.torch_dtype)
    cache = tk.ThinKCache(cfg, ws.seq_lens, device=dev)
    cache.prefill(data["Q_obs"].to(dev), data["K"].to(dev), data["V"].to(dev))
    outs = []
    for s in steps_in:
        outs.append(cache.append_decode(s["k_new"].to(dev), s["v_new"].to(dev), s["q"].to(dev)).to("cpu", torch.float64).numpy())
    idx = cache.idx_tensor().cpu().numpy().astype("int64")
    err = cache.device_error()
    cache.close()
    return idx, outs, err


def oracle_sample(w: wl.Workload, budget_s: float = 20.0, sizing=None, threads=None, check_gpu=False):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: a few layers of
    the same prompts and a few decode steps, sized from a short probe so that it ends in about
    `budget_s` seconds.  Reported in the benchmark's unit (algorithmic bytes / wall time).
    With `check_gpu` the CUDA path runs on the very same sample afterwards and is compared with what the
    oracle just computed: index mismatches (near-ties counted apart) and the max-abs attention error."""
    import contextlib
    import numpy as np
    from oracle import think_oracle as orc
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
        limit = threadpool_limits(limits=threads) if threads else contextlib.nullcontext()
        if threads:
            cores = min(cores, threads)
    except Exception:
        cores, limit = 1, contextlib.nullcontext()
    T = orc.kept_channels(w.lam, w.D)

    def run(L, B, steps, keep=False):
        ws = wl.shrink(w, L=L, B=B, steps=steps)
        data = wl.make_prefill(ws, device="cpu")
        K64, V64, Q64 = (data[k].to(torch.float64).numpy() for k in ("K", "V", "Q_obs"))
        st_in = [wl.make_step(ws, t, device="cpu") for t in range(steps)]
        st = [{k: v.to(torch.float64).numpy() for k, v in s.items()} for s in st_in]
        o = orc.ThinKOracle(ws.B, ws.L, ws.N_q, ws.N_kv, ws.D, ws.seq_lens, ws.S_obs, ws.recent, ws.lam)
        outs = []
        t0 = time.perf_counter()
        o.score_select(Q64, K64)
        o.compact(K64, V64)
        t1 = time.perf_counter()
        for t in range(steps):
            o.append(st[t]["k_new"], st[t]["v_new"])
            outs.append(o.decode_attn(st[t]["q"]))
        t2 = time.perf_counter()
        nbytes = prefill_bytes(ws, T) + sum(decode_bytes(ws, T, t) for t in range(steps)) + steps * append_bytes(ws)
        extra = (o, outs, data, st_in, st, K64, V64) if keep else None
        return t2 - t0, t1 - t0, t2 - t1, nbytes, ws, extra

    with limit:
        if sizing is None:
            run(1, 1, 1)                                 # warm-up of the numeric library's threads
            _, pre1, dec1, _, _, _ = run(1, 1, 1)        # one layer, one decode step: cost of either phase per layer
            steps = int(max(1, min(w.steps, 16)))
            if budget_s < 4 * (pre1 + steps * dec1):     # small budgets: fewer decode steps before fewer layers
                steps = int(max(1, min(steps, (budget_s / 2 - pre1) / max(dec1, 1e-6))))
            L = int(max(1, min(w.L, budget_s / max(pre1 + steps * dec1, 1e-3))))
        else:
            L, steps = sizing
        dt, dt_pre, dt_dec, nbytes, ws, extra = run(L, 1, steps, keep=check_gpu)
    res = {"value": nbytes / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
           "sample": f"{ws.name}: B=1 of {w.B}, L={L} of {w.L}, S={ws.seq_lens[0]}, {steps} decode steps; "
                     f"prefill {dt_pre:.2f} s, decode {dt_dec / steps * 1e3:.1f} ms/step",
           "seconds": dt, "sizing": (L, steps)}
    if check_gpu:
        o, outs, data, st_in, st, K64, V64 = extra
        idx_gpu, outs_gpu, dev_err = _cuda_path_on_sample(ws, data, st_in)
        mism = near = 0
        for b in range(ws.B):
            for l in range(ws.L):
                for h in range(ws.N_kv):
                    if not (idx_gpu[b, l, h] == o.idx[b, l, h]).all():
                        mism += 1
                        near += int(orc.near_tie(o.score[b, l, h], o.T, 1e-6))
        if mism:
            # the oracle continues with the CUDA path's (near-tie) choice so that the attention rows compare like with like
            o.idx = idx_gpu
            o.compact(K64, V64)
            outs = []
            for t in range(steps):
                o.append(st[t]["k_new"], st[t]["v_new"])
                outs.append(o.decode_attn(st[t]["q"]))
        # the max-abs bar applies where the output grid allows it: a bf16 output of magnitude >= 4 has half an ulp
        # of 0.0156 or more, those elements are counted and held to half an ulp + 1e-3 instead
        max_abs = worst_large = 0.0
        n_large = 0
        for a, b in zip(outs_gpu, outs):
            err = np.abs(a - b)
            small = np.abs(b) < 4.0 if w.dtype == "bf16" else np.ones(b.shape, dtype=bool)
            if small.any():
                max_abs = max(max_abs, float(err[small].max()))
            if (~small).any():
                n_large += int((~small).sum())
                ulp = 2.0 ** (np.floor(np.log2(np.abs(b[~small]))) - 7)
                worst_large = max(worst_large, float((err[~small] / (0.5 * ulp + 1e-3)).max()))
        res["parity"] = {"heads": ws.B * ws.L * ws.N_kv, "idx_mismatches": mism, "near_ties": near,
                         "attn_rows": steps * ws.B * ws.L * ws.N_q, "max_abs": max_abs,
                         "tolerance": 1e-2 if w.dtype == "bf16" else 1e-5, "outputs_ge_4": n_large,
                         "outputs_ge_4_worst_over_bar": worst_large, "device_error": dev_err,
                         "sample": res["sample"].split(";")[0]}
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    w = wl.get_config(HEADLINE if args.config == "all" else args.config)
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
            "metric": METRIC,
            "value": v, "unit": "GB/s", "n_gpus": int(os.environ.get("WORLD_SIZE", 1)), "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name} (bounded sample per step: {last['sample']})"},
            "cpu_baseline": {"value": v, "unit": "GB/s", "cores": last["cores"], "kind": "oracle",
                             "sample": last["sample"]},
            "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


METRIC = ("ThinK hot path effective HBM GB/s (prefill score+select+compact, then decode append+attn; "
          "algorithmic bytes / device time)")


# --------------------------------------------------------------------------- the GPU arm
def run_ours(args):
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    names = list(ALL_CONFIGS) if args.config == "all" else [args.config]
    head = HEADLINE if args.config == "all" else args.config
    n_warm = args.warmup if args.profile else max(3, args.warmup)
    # passes of the other configs: a second or two of device time each, never fewer than two
    side_passes = {"c1": 50, "c2": 20, "c3": 4, "c4": 2, "c5": 2}
    per, wls = {}, {}
    for name in names:
        is_head = name == head
        passes = args.steps if is_head else side_passes.get(name, 2)
        per[name], wls[name] = measure_config(args, name, passes, n_warm, dev, world, barrier,
                                              do_e2e=is_head and not args.no_e2e, sample_clocks=True)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle on this machine's cores, on a bounded sample of every config; the CUDA path is checked against
        # what the oracle computed on that sample (parity figures beside the timings)
        for name in names:
            share = args.cpu_budget if name == head else args.cpu_budget / 3
            c = oracle_sample(wls[name], budget_s=share, check_gpu=True)
            sizing = c.pop("sizing")
            one = oracle_sample(wls[name], budget_s=share / 2, sizing=(max(1, sizing[0] // 4), max(1, sizing[1] // 2)), threads=1)
            c["one_thread"] = {"value": one["value"], "unit": "GB/s", "cores": 1, "sample": one["sample"]}
            per[name]["parity"] = c.pop("parity")
            per[name]["cpu_baseline"] = c
        cpu = per[head]["cpu_baseline"]

    if rank == 0:
        h = per[head]
        line = {
            "metric": METRIC,
            "value": h["value"], "unit": "GB/s", "n_gpus": world, "steps": h["passes"], "warmup": n_warm,
            "ms_per_step": h["ms_per_pass"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": h["dtype"], "data": "synthetic",
            "config": {"workload": h["workload"], "configs_run": names,
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "l2": "inputs larger than L2 (K, V and the caches are each several L2 sizes)"},
            "decode": h["decode"], "prefill": h["prefill"], "roofline": h["roofline"],
            "fused_step_variant": h["fused_step_variant"], "clocks": h["clocks"], "e2e": h["e2e"],
            "gpu_launches": h["gpu_launches"], "parity": h.get("parity"), "cpu_baseline": cpu,
            "per_config": {n: {k: v for k, v in per[n].items() if k not in ("e2e",)} for n in names},
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5, help="timed passes of the headline config")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="all", choices=["all"] + sorted(wl.CONFIGS))
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
    ap.add_argument("--two-call-prefill", action="store_true",
                    help="prefill through thinK_score_select + thinK_compact instead of thinK_prefill")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--layers", type=int, default=0,
                    help="run the config with this many layers instead of its own (small case for ncu captures; the "
                         "workload label carries the changed layer count)")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under ncu: take --warmup literally (fewer launches before the captured ones)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as one process but asked for N replicas: start N ranks of this script, one per GPU
        from paper_2407_21018_b200 import replicas
        sys.exit(replicas.launch(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
