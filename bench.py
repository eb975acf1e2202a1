#!/usr/bin/env python
"""Benchmark of the D3ToM merge-layer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C2] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic input:
merge-layer attention + importance map, select, merge (similarity, aggregation,
compaction) and the post-merge layers (projection + ragged attention each).
The default workload is C2, the LLaDA-8B-shaped configuration with thousands of
visual tokens (4096 visual + 128 prompt + 64 response tokens, keep ratio 0.25,
3 post-merge layers).  One JSON line is printed by rank 0.  Beside the step time
of the chosen configuration it carries

  roofline      the dominant kernel (merge-layer attention) against the measured tensor peak
  kernels       every kernel of the step: device time inside running steps, algorithmic work,
                fraction of the nominal, measured-burst and measured-sustained peaks
  configs       step time, attention fraction and end-to-end time of the other configurations
  cpu_baseline  the CPU oracle timed on one whole step of the same workload
  e2e           the same step fed from pinned host memory, result copied back

With N > 1 every rank processes its own request batch of the same shape: the
path shards by request with no collective on the data path; the only
communication is the barrier and the max-over-ranks of the timing.  Launched
under torch.distributed.run the ranks come from the environment; launched
plainly with --gpus N > 1 this script starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD_TEXT = {
    "C0": "C0: tiny fp32 merge layer, 256 visual + 16 prompt + 16 response tokens, 4 heads x 64, keep 0.25",
    "C1": "C1: LLaDA-8B-shaped merge layer, 1024 visual + 64 prompt + 64 response tokens, 32 heads x 128, keep 0.10",
    "C2": "C2: LLaDA-8B-shaped, 4096 visual + 128 prompt + 64 response tokens, 32 heads x 128, keep 0.25, 3 post-merge layers",
    "C3": "C3: step schedule, 2048 visual + 64 prompt + 64 response tokens, 32 heads x 128, T = 64 denoising steps, "
          "one more decider per step, keep ratio 0.5 -> 0 (mean 0.25), 3 post-merge layers; a step = one denoising step",
    "C4": "C4: 8 ragged requests, 1024-4096 visual tokens each, 32 heads x 128, keep in {0.1,0.25,0.5}, 3 post-merge layers",
}
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel (the launch `roofline`
# times: attention alone at the merge-layer length) from the committed ncu capture, mean of two launches; null for
# configurations not captured, and null whenever attn_sk.cu / attn_tc.cu have changed since the capture
ATTN_TRAFFIC_BYTES = {"C2": 177.0e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
REFERENCE_BUDGET_S = 240.0          # the CPU arm stops adding steps once they would not fit this


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None
        self.path = None

    def __enter__(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def wait_started(self, keep_busy, limit_s=4.0):
        """Runs ``keep_busy`` until the sampler has written its first line (nvidia-smi takes a
        moment to start), so that the samples cover the timed region that follows."""
        t0 = time.time()
        while self.proc is not None and time.time() - t0 < limit_s:
            keep_busy()
            try:
                if os.path.getsize(self.path) > 0:
                    break
            except OSError:
                break

    def summary(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.path is None:
            return out
        try:
            rows = [l.strip().split(", ") for l in open(self.path) if l.strip()]
            os.unlink(self.path)
        except Exception:
            return out
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            # the median over the busiest half: the sampler also sees the idle edges of the region
            top = sorted(sm)[len(sm) // 2:]
            out.update(sm_mhz=float(np.median(top)), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------ oracle timing
def oracle_inputs(w, decider_pos=None):
    """The step's inputs as float64 arrays (conversion is not part of the timed oracle step)."""
    import torch
    decider_pos = w.decider_pos if decider_pos is None else decider_pos
    q = w.q_for(decider_pos).to(dtype=torch.float64).numpy()
    k = w.k.double().numpy()
    v = w.v.double().numpy()
    w_post = [x.double().numpy() for x in w.w_post]
    return q, k, v, w_post


def oracle_step(w, inputs, decider_pos=None, keep=None):
    """One WHOLE step of workload ``w`` on the CPU oracle as it stands, nothing sampled or extrapolated:
    attention over every head, importance, select, merge (MEAN) and every post-merge layer.
    Returns (seconds, seconds per part)."""
    from oracle import d3tom_oracle as orc
    q, k, v, w_post = inputs
    H, dh = w.H, w.dh
    scale = 1.0 / np.sqrt(dh)
    cu = w.cu_seqlens
    decider_pos = w.decider_pos if decider_pos is None else decider_pos
    dec = np.concatenate([np.asarray(d, np.int64) for d in decider_pos])
    t = {}
    t0 = time.perf_counter()
    hidden = orc.round_storage(orc.attention(q, k, v, cu, scale), w.dtype)
    t["attn"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    S = orc.importance(q, k, cu, w.n_visual, dec, w.cu_deciders(decider_pos), scale)
    t["importance"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    if keep is None:
        keep = [orc.keep_count(w.n_visual[b], w.keep_ratio[b]) if len(decider_pos[b]) else w.n_visual[b]
                for b in range(w.B)]
    kept = [orc.select(S[b].astype(np.float32), keep[b]) for b in range(w.B)]
    t["select"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    res = orc.merge(hidden, cu, w.n_visual, kept, orc.MEAN, w.dtype)
    t["merge"] = time.perf_counter() - t0
    t0 = time.perf_counter()
    x = res["hidden_out"]
    for wl_ in w_post:
        x = orc.post_layer(x, wl_, res["cu_seqlens_out"], H, w.dtype)
    t["post"] = time.perf_counter() - t0
    return sum(t.values()), t


ORACLE_SAMPLE_TEXT = ("one whole step of the workload on the NumPy/fp64 oracle as it stands: attention over all heads, "
                      "importance, select, merge (mean) and all post-merge layers; nothing sampled or extrapolated")


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def schedule_middle(w):
    """Schedule config: decider list and keep count of the middle denoising step (the oracle's sampled step)."""
    from oracle import d3tom_oracle as orc
    sm = w.T // 2
    a_min = 2.0 * (1.0 - w.mean_keep_ratio) - 1.0
    return sm, dict(decider_pos=w.step_deciders(sm),
                    keep=[orc.keep_count(w.n_visual[0], 1.0 - orc.schedule_alpha(sm, w.T, a_min, 1.0))])


def reference_arm(args, config):
    """The CPU oracle as the reference arm: every step is one whole oracle step of the workload."""
    from paper_2511_12280_b200 import workload as wl
    w = wl.config(args.config)
    config["requests_per_gpu"] = w.B
    kw = {}
    if w.T:        # the schedule config is timed at its middle step
        sm, kw = schedule_middle(w)
        config["sampled_step"] = sm
    inputs = oracle_inputs(w, kw.get("decider_pos"))
    times, parts = [], {}
    t_start = time.perf_counter()
    warm_left, steps_timed, warm_done = args.warmup, 0, 0
    while steps_timed < args.steps:
        sec, parts = oracle_step(w, inputs, **kw)
        if warm_left > 0:
            warm_left -= 1
            warm_done += 1
        else:
            times.append(sec)
            steps_timed += 1
        elapsed = time.perf_counter() - t_start
        per = elapsed / (warm_done + steps_timed)
        if elapsed + per > REFERENCE_BUDGET_S:          # the next step would not fit: stop here
            if not times:                               # not even one timed step yet: the last warm-up step is the sample
                times.append(sec)
                steps_timed = 1
                warm_done -= 1
            break
    us = float(np.mean(times)) * 1e6
    line = {"impl": "reference", "metric": "merge_layer_step_us", "value": us, "unit": "us", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "steps_timed": steps_timed, "warmup_done": warm_done,
            "step_us_median": float(np.median(times)) * 1e6, "step_us_min": float(np.min(times)) * 1e6,
            "cpu_baseline": {"value": us, "unit": "us", "cores": blas_threads(), "kind": "oracle",
                             "sample": ORACLE_SAMPLE_TEXT, "steps_timed": steps_timed, "extrapolated": False},
            "e2e": {"value": us, "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "breakdown_s": parts}
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------------ N ranks from a plain launch
def spawn_ranks(args):
    """`python bench.py --gpus N` with N > 1 and no launcher around it: start the N ranks (one per GPU, rendezvous on
    127.0.0.1) with torch.distributed.run and pass their output through."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


# ------------------------------------------------------------------------------------------ per-kernel device times
def step_kernel_labels(step):
    """Kernels of one run() in launch order, as (label, substring its kernel name must contain)."""
    seq = [("attn_merge_layer", "attn_"), ("importance_finish", "importance_finish"), ("select", "select"),
           ("prepare_rows", "prepare_rows")]
    if step.total_out < step.total:
        seq.append(("similarity_gemm", "gemm_"))
    seq += [("members", "members"), ("aggregate_compact", "aggregate")]
    for _ in range(step.n_post):
        seq += [("proj_qkv", "gemm_"), ("attn_post", "attn_")]       # gemm_tc_kernel, or gemm_pair_kernel for long layers
    return seq


def kernel_work(step, q):
    """Algorithmic work of every kernel of the step: ("tensor", flops) or ("hbm", bytes)."""
    D, H, es = step.D, step.H, q.element_size()
    V, K = step.n_visual_h, step.keep_h
    n_dec = [int(step.cu_dec_h[b + 1] - step.cu_dec_h[b]) for b in range(step.nB)]
    tv, tk = sum(V), sum(K)
    return {
        "attn_merge_layer": ("tensor", sum(4.0 * n * n * D for n in step.seqlens_h)),
        "importance_finish": ("hbm", sum(4.0 * H * d * v for d, v in zip(n_dec, V)) + 4.0 * tv),
        "select": ("hbm", 4.0 * tv + 4.0 * tk + tv),
        "prepare_rows": ("hbm", float(tv + tk) * D * es),
        "similarity_gemm": ("tensor", sum(2.0 * (v - k) * k * D for v, k in zip(V, K))),
        "members": ("hbm", 4.0 * tv + 4.0 * tv + 8.0 * tk),
        "aggregate_compact": ("hbm", float(step.total + step.total_out) * D * es),
        "proj_qkv": ("tensor", 2.0 * step.total_out * D * 3 * D),
        "attn_post": ("tensor", sum(4.0 * n * n * D for n in step.out_lens_h)),
    }


def kernel_profile(step, run_host, q, peaks, n_steps=10):
    """Device time of every kernel of the step while whole steps run back to back (CUDA profiling interface through
    torch.profiler, outside any timed region), with its algorithmic work and the fraction of each peak it reaches."""
    import torch
    from torch.profiler import ProfilerActivity, profile
    from paper_2511_12280_b200 import binding as B_
    try:
        # without launch overlap: otherwise a kernel's recorded time includes its wait for the drain of the one before
        B_.d3tom_set_launch_overlap(False)
        try:
            for _ in range(2):
                run_host()
            torch.cuda.synchronize()
            with profile(activities=[ProfilerActivity.CUDA]) as prof:
                for _ in range(n_steps):
                    run_host()
                torch.cuda.synchronize()
        finally:
            B_.d3tom_set_launch_overlap(True)
        evs = []
        for e in prof.events():
            if str(getattr(e, "device_type", "")).endswith("CUDA") and not e.name.lower().startswith(("memcpy", "memset")):
                evs.append((e.time_range.start, e.name, float(e.time_range.elapsed_us())))
        evs.sort()
        seq = step_kernel_labels(step)
        L = len(seq)
        # whole steps only: a step is L consecutive kernels whose names match the expected sequence (the profiler
        # now and then drops a record at the edge of its buffer; such a step is skipped)
        times, n_whole, i = {}, 0, 0
        while L and i + L <= len(evs):
            if all(must in evs[i + j][1] for j, (_, must) in enumerate(seq)):
                for j, (label, _) in enumerate(seq):
                    times.setdefault(label, []).append(evs[i + j][2])
                n_whole += 1
                i += L
            else:
                i += 1
        if n_whole < 2:
            return {"error": "expected %d kernels per step; the profiler saw %d kernels in %d steps and fewer than two "
                             "whole steps" % (L, len(evs), n_steps)}
        n_steps = n_whole
        work = kernel_work(step, q)
        out = {}
        per_step = 0.0
        for label, _ in dict.fromkeys(seq):
            ts = times[label]
            us = float(np.median(ts))
            calls = len(ts) // n_steps
            per_step += us * calls
            bound, amount = work[label]
            rate = amount / (us * 1e-6)
            entry = {"us": us, "launches_per_step": calls, "bound": bound}
            if bound == "tensor":
                tf = rate / 1e12
                entry.update(gflop=amount / 1e9, tflops=tf, frac_nominal=tf / NOMINAL_PEAKS["bf16_tflops"],
                             frac_measured_burst=tf / peaks["bf16_tflops"],
                             frac_measured_sustained=tf / peaks["bf16_tflops_sustained"])
            else:
                gbs = rate / 1e9
                entry.update(mbytes=amount / 1e6, gbs=gbs, frac_nominal=gbs / NOMINAL_PEAKS["hbm_gbs"],
                             frac_measured_copy=gbs / peaks["hbm_gbs"])
            out[label] = entry
        out["sum_us_per_step"] = per_step
        out["how"] = ("median device time over %d host-launched steps run back to back with the launch overlap "
                      "(programmatic dependent launch) switched off, so that each kernel's time is its own; the timed "
                      "step keeps the overlap, which hides most of every kernel's ramp-up and drain" % n_steps)
        return out
    except Exception as exc:                         # the profile is a report, never a reason to lose the bench line
        return {"error": "%s: %s" % (type(exc).__name__, exc)}


def block_timings(step, w, w_post0, q, dev, timed, reps):
    """The rest of a post-merge block (Algorithm 1, FFN_l; layer-cost equation of the FLOPs appendix): output
    projection and gated feed-forward network at the shortened length N_m, and the whole block at N_m and at the
    full length N, so that the measured saving of a post-merge layer can be set beside the FLOPs ratio.
    m = 3 d (12288 at d = 4096, the LLaDA-8B width)."""
    import torch
    from paper_2511_12280_b200 import workload as wl
    timed_cold = timed

    def timed(fn, iters):            # one untimed call first: these kernels have not run yet
        fn()
        return timed_cold(fn, iters)
    D, m = step.D, 3 * step.D
    t = wl.block_inputs(1000, 8, D, m, w.dtype)           # weights only; the rows come from the step's own tensors
    w_o, w_gu, w_dn = t["w_o"].to(dev), t["w_gate_up"].to(dev), t["w_down"].to(dev)
    ctx = step.ctx
    out = {}
    n_full, n_m = step.total, step.total_out
    act = torch.empty(n_full, m, dtype=q.dtype, device=dev)
    y = torch.empty(n_full, D, dtype=q.dtype, device=dev)
    z = torch.empty(n_full, D, dtype=q.dtype, device=dev)
    q3, k3, v3 = (torch.empty(n_full, D, dtype=q.dtype, device=dev) for _ in range(3))
    x_m, x_full = step.hidden_out, step.attn_out
    for tag, n, x, cu, mx in (("Nm", n_m, x_m, step.cu_out, step.max_out), ("N", n_full, x_full, step.cu_seqlens, step.max_seqlen)):
        parts = {
            "proj_qkv": timed(lambda: ctx.d3tom_proj_qkv(x, w_post0, n, D, q3, k3, v3), reps),
            "attn": timed(lambda: ctx.d3tom_attn_varlen(q3, k3, v3, cu, step.nB, n, mx, step.scale, y), reps),
            "proj_out": timed(lambda: ctx.d3tom_linear(y, w_o, x, n, D, D, z), reps),
            "ffn": timed(lambda: ctx.d3tom_ffn(z, w_gu, w_dn, z, n, D, m, act, y), reps),
        }
        parts["block"] = sum(parts.values())
        out[tag] = parts
    lens_m, lens_f = step.out_lens_h, step.seqlens_h
    macs = lambda lens: sum(4.0 * n * D * D + 2.0 * n * n * D + 3.0 * n * D * m for n in lens)      # layer-cost equation
    out["proj_out_tflops_Nm"] = 2.0 * n_m * D * D / (out["Nm"]["proj_out"] * 1e-6) / 1e12
    out["ffn_tflops_Nm"] = 6.0 * n_m * D * m / (out["Nm"]["ffn"] * 1e-6) / 1e12
    out["ffn_tflops_N"] = 6.0 * n_full * D * m / (out["N"]["ffn"] * 1e-6) / 1e12
    out["layer_time_ratio_Nm_over_N"] = out["Nm"]["block"] / out["N"]["block"]
    out["layer_flops_ratio_Nm_over_N"] = macs(lens_m) / macs(lens_f)
    out["m"] = m
    return out


def dense_ab(step, w, w_post, q, dev, reps=8, calls=6):
    """Dense layers of a post-merge block on CTA pairs against single-CTA tiles, alternating the two shapes quickly so
    that both see the same power state: median us per call of the projection, the output projection and the gated
    feed-forward network at the shortened length N_m and at the full length N."""
    import torch
    from paper_2511_12280_b200 import binding as B_
    from paper_2511_12280_b200 import workload as wl
    D, m = step.D, 3 * step.D
    t = wl.block_inputs(1000, 8, D, m, w.dtype)
    w_o, w_gu, w_dn = t["w_o"].to(dev), t["w_gate_up"].to(dev), t["w_down"].to(dev)
    ctx, out = step.ctx, {}
    n_full, n_m = step.total, step.total_out
    act = torch.empty(n_full, m, dtype=q.dtype, device=dev)
    y = torch.empty(n_full, D, dtype=q.dtype, device=dev)
    q3, k3, v3 = (torch.empty(n_full, D, dtype=q.dtype, device=dev) for _ in range(3))

    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(calls):
            fn(i)
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e3 / calls
    try:
        for tag, n, x in (("Nm", n_m, step.hidden_out), ("N", n_full, step.attn_out)):
            fns = {"proj_qkv": lambda i: ctx.d3tom_proj_qkv(x, w_post[i % len(w_post)], n, D, q3, k3, v3),
                   "proj_out": lambda i: ctx.d3tom_linear(x, w_o, x, n, D, D, y),
                   "ffn": lambda i: ctx.d3tom_ffn(x, w_gu, w_dn, x, n, D, m, act, y)}
            out[tag] = {"rows": n}
            for name, fn in fns.items():
                res = {0: [], 256: []}
                for _ in range(reps):
                    for width in (0, 256):
                        B_.d3tom_set_pair_tiles(width)
                        fn(0)
                        res[width].append(timed(fn))
                out[tag][name] = {"single_cta_us": float(np.median(res[0])), "cta_pairs_us": float(np.median(res[256]))}
    finally:
        B_.d3tom_set_pair_tiles(-1)
    return out


def make_kv_cache_case(step, w, k, v, dev):
    """Returns a callable that runs d3tom_merge_kv on the K/V rows of every request's [visual | prompt]
    prefix with the kept set that the step's select produced."""
    import torch
    D = step.D
    cu_full = step.cu_seqlens_h
    rows = np.concatenate([np.arange(cu_full[b], cu_full[b] + w.n_visual[b] + w.n_prompt[b]) for b in range(w.B)])
    idx = torch.as_tensor(rows, device=dev)
    k_c, v_c = k.reshape(-1, D)[idx].contiguous(), v.reshape(-1, D)[idx].contiguous()
    lens = [a + b for a, b in zip(w.n_visual, w.n_prompt)]
    cs = lambda a: np.concatenate([[0], np.cumsum(a)]).astype(np.int32)
    cu, cu_out = cs(lens), cs([n - vv + kk for n, vv, kk in zip(lens, w.n_visual, step.keep_h)])
    t = lambda a: torch.as_tensor(np.asarray(a, np.int32), device=dev)
    cu_d, cu_out_d = t(cu), t(cu_out)
    total, total_out = int(cu[-1]), int(cu_out[-1])
    k_o = torch.empty(total_out, D, dtype=k.dtype, device=dev); v_o = torch.empty_like(k_o)
    assign = torch.empty(step.total_vis, dtype=torch.int32, device=dev)
    mc = torch.empty(step.total_kept, dtype=torch.int32, device=dev)
    src = torch.empty(total_out, dtype=torch.int32, device=dev)
    nB, mode, ctx = step.nB, step.mode, step.ctx
    nv, cv, ki, ck, mv, mk = step.n_visual_d, step.cu_vis, step.kept_idx, step.cu_kept, step.max_visual, step.max_kept
    return lambda: ctx.d3tom_merge_kv(mode, k_c, v_c, cu_d, nv, cv, ki, ck, nB, D, total, total_out, mv, mk, k_o, v_o,
                                      cu_out_d, assign, mc, src)


# ------------------------------------------------------------------------------------------ one configuration on the GPU
def measure_config(name, args, dev, local_rank, world, full):
    """Times configuration ``name`` on this rank's GPU.  ``full`` adds the clock record, the per-kernel profile, the
    K/V-cache merge, the rest of a post-merge block and the serial end-to-end figure (the chosen configuration);
    without it only the step, its calls, the attention kernel alone and the overlapped end-to-end path are timed
    (the other configurations of the `configs` object)."""
    import torch
    import torch.distributed as dist
    from paper_2511_12280_b200 import binding as B_
    from paper_2511_12280_b200 import replicas, trajectory
    from paper_2511_12280_b200 import workload as wl
    from paper_2511_12280_b200.pipeline import HostFedStep, MergeLayerStep

    w = wl.config(name)
    total = int(w.cu_seqlens[-1])
    res = {"requests_per_gpu": w.B, "total_tokens": total}
    # one problem per schedule step (a single one for the constant-ratio configs)
    plan = plan_unmerged = None
    if w.T:
        a_min, a_max = 2.0 * (1.0 - w.mean_keep_ratio) - 1.0, 1.0
        T_steps = w.T // args.tokens_per_step
        kw_plan = dict(tokens_per_step=args.tokens_per_step, reversed_=args.reversed, deciders=args.deciders)
        plan = trajectory.plan_schedule(w.n_visual, w.n_prompt, [w.decode_order], T_steps, a_min, a_max, **kw_plan)
        plan_unmerged = trajectory.plan_schedule(w.n_visual, w.n_prompt, [w.decode_order], T_steps, a_min, a_max,
                                                 merged=False, **kw_plan)
        dec_steps = [p.decider_pos for p in plan]
        keep_steps = [p.keep_count for p in plan]
        res["schedule"] = {"T": T_steps, "alpha_min": a_min, "alpha_max": a_max, "tokens_per_step": args.tokens_per_step,
                           "reversed": bool(args.reversed), "deciders": args.deciders,
                           "keep_counts": [k[0] for k in keep_steps]}
    else:
        dec_steps = [w.decider_pos]
        keep_steps = [[B_.d3tom_keep_count(v, r) for v, r in zip(w.n_visual, w.keep_ratio)]]
    n_prob = len(dec_steps)
    mid = n_prob // 2
    step = MergeLayerStep(w.H, w.dh, w.torch_dtype, total, w.B, max(sum(len(d) for d in dec) for dec in dec_steps),
                          max(w.n_visual), n_post=len(w.w_post), mode=B_.AGG_MEAN, device=local_rank)
    probs = [step.make_problem(w.n_visual, w.n_prompt, w.n_resp, dec, keep) for dec, keep in zip(dec_steps, keep_steps)]
    step.use_problem(probs[mid])
    q_hs = [w.q_for(dec).contiguous().pin_memory() for dec in dec_steps]
    k_h, v_h = w.k.contiguous().pin_memory(), w.v.contiguous().pin_memory()
    qs = [t.to(dev) for t in q_hs]
    q = qs[mid]
    k, v = k_h.to(dev), v_h.to(dev)
    q_stage = torch.empty_like(q)               # where the serial end-to-end path lands the step's Q
    w_post = [x.to(dev) for x in w.w_post]
    out_h = torch.empty(total, step.D, dtype=w.torch_dtype).pin_memory()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3   # us

    def timed_each(fn, iters):
        """(mean over the whole region, per-iteration times): one event between consecutive iterations."""
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        ev[0].record()
        for i in range(iters):
            fn()
            ev[i + 1].record()
        ev[-1].synchronize()
        each = [ev[i].elapsed_time(ev[i + 1]) * 1e3 for i in range(iters)]
        return ev[0].elapsed_time(ev[-1]) / iters * 1e3, each

    counter = {"i": 0, "launches": 0}
    # one CUDA graph per problem: a step is then one graph launch (the kernels and their order are unchanged)
    graphs = None
    if not args.no_graph and args.only is None:
        graphs = []
        for i in range(n_prob):
            step.use_problem(probs[i])
            graphs.append(step.capture(qs[i], k, v, w_post))
        step.use_problem(probs[mid])
    res["launch"] = "cuda graph replay, one per step" if graphs is not None else "host launches"

    def run():
        i = counter["i"] % n_prob
        counter["i"] += 1
        step.use_problem(probs[i])
        counter["launches"] += step.launches_per_step()
        if graphs is not None:
            graphs[i].replay()
            return step.layer_out[-1] if step.n_post else step.hidden_out
        return step.run(qs[i], k, v, w_post)

    def run_host_mid():
        step.use_problem(probs[mid])
        return step.run(qs[mid], k, v, w_post)

    if args.only is not None:
        run()
        calls = {
            "attn_importance": lambda: step.attn_importance(q, k, v),
            # the launch that `roofline` times: attention alone at the merge-layer length, no importance side-work
            "attn_alone": lambda: step.ctx.d3tom_attn_varlen(q, k, v, step.cu_seqlens, step.nB, step.total,
                                                             step.max_seqlen, step.scale, step.attn_out),
            "select": lambda: step.select(),
            "merge": lambda: step.merge(),
            "step": run,
        }
        if step.n_post:
            calls["proj_qkv"] = lambda: step.ctx.d3tom_proj_qkv(step.hidden_out, w_post[0], step.total_out, step.D,
                                                                step.q2, step.k2, step.v2)
            calls["attn_varlen"] = lambda: step.ctx.d3tom_attn_varlen(step.q2, step.k2, step.v2, step.cu_out, step.nB,
                                                                      step.total_out, step.max_out, step.scale,
                                                                      step.layer_out[0])
        if args.only in ("proj_out", "ffn"):          # the rest of a post-merge block at the shortened length
            m_ff = 3 * step.D
            t = wl.block_inputs(1000, 8, step.D, m_ff, w.dtype)
            w_o, w_gu, w_dn = t["w_o"].to(dev), t["w_gate_up"].to(dev), t["w_down"].to(dev)
            act = torch.empty(step.total_out, m_ff, dtype=q.dtype, device=dev)
            y = torch.empty(step.total_out, step.D, dtype=q.dtype, device=dev)
            calls["proj_out"] = lambda: step.ctx.d3tom_linear(step.layer_out[0], w_o, step.hidden_out, step.total_out,
                                                              step.D, step.D, y)
            calls["ffn"] = lambda: step.ctx.d3tom_ffn(step.hidden_out, w_gu, w_dn, step.hidden_out, step.total_out,
                                                      step.D, m_ff, act, y)
        torch.cuda.synchronize()
        if args.only == "dense_ab":
            return {"only": args.only, "config": name, "dense_ab": dense_ab(step, w, w_post, q, dev)}
        us = timed(calls[args.only], args.steps)
        return {"only": args.only, "us": us, "config": name}

    n_steps = args.steps if full else max(n_prob, min(args.steps, 40))
    # ---- device-resident timing of the whole step
    for _ in range(max(3, args.warmup)):
        run()
    sync_all()
    clk_cm = ClockSampler(local_rank) if full else None
    if clk_cm is not None:
        clk_cm.__enter__()
        clk_cm.wait_started(run)          # keeps the GPU busy until the sampler delivers
    try:
        sync_all()
        counter["i"] = 0
        counter["launches"] = 0
        step_us, each = timed_each(run, n_steps)
        res["gpu_launches"] = counter["launches"]
        res["steps_timed"] = n_steps
        sync_all()
        # ---- per-step series of the schedule config: one event pair per denoising step, median of 3 trajectories
        if w.T:
            series = []
            for _ in range(3):
                counter["i"] = 0
                series.append([timed(run, 1) for _ in range(n_prob)])
            per_step = [float(x) for x in np.median(np.asarray(series), axis=0)]
            # the same trajectory without merging (every visual token kept), one graph per step as well
            traj_u = trajectory.Trajectory(step, plan_unmerged, w.n_visual, w.n_prompt, w.n_resp)
            traj_m = trajectory.Trajectory(step, plan, w.n_visual, w.n_prompt, w.n_resp)
            traj_u.capture(qs, k, v, w_post)
            traj_u.run()
            sync_all()
            unmerged_us = float(np.median([timed(traj_u.run, 1) for _ in range(3)]))
            res["per_step_us"] = per_step
            res["trajectory"] = {"T": len(plan), "total_us": float(sum(per_step)), "unmerged_total_us": unmerged_us,
                                 "time_ratio": float(sum(per_step)) / unmerged_us,
                                 "flops_ratio": traj_m.flops(step.D, step.n_post) / traj_u.flops(step.D, step.n_post)}
            del traj_u
        # ---- the same steps right after an idle second (boost clocks): the timed region above runs under the board's
        #      power cap, because the GPU has been busy for seconds by then; the difference is the cap, not the kernels
        if full and n_prob == 1:
            time.sleep(1.0)
            _, after_idle = timed_each(run, 10)
            res["step_us_after_idle"] = float(np.median(after_idle[4:]))
            sync_all()
        # the breakdown below is taken at the middle problem
        counter["i"] = mid
        run()
        sync_all()
        # ---- per-call breakdown (each call timed back to back on warm instruction caches;
        #      every call's working set is streamed from HBM or L2 as it would be inside the step)
        reps = min(100, max(10, args.steps))
        # the dominant kernel alone (no importance side-work): the attention kernel at the merge-layer length; taken
        # first, before the long GEMM timings below pull the board into its power cap
        time.sleep(0.5)      # the burst peak it is compared with was measured on an idle board: let the power state settle
        attn_alone = lambda: step.ctx.d3tom_attn_varlen(q, k, v, step.cu_seqlens, step.nB, step.total,
                                                        step.max_seqlen, step.scale, step.attn_out)
        for _ in range(5):   # the first launches after an idle spell run while the SM clock is still ramping up
            attn_alone()     # (384, 283, 274, 270, 268 us, then 262 - 266 us per launch at 4288 rows)
        attn_kernel_us, attn_each = timed_each(attn_alone, reps)
        br = {}
        br["attn_importance"] = timed(lambda: step.attn_importance(q, k, v), reps)
        br["select"] = timed(lambda: step.select(), reps)
        br["merge"] = timed(lambda: step.merge(), reps)
        if step.n_post:
            br["proj_qkv"] = timed(lambda: step.ctx.d3tom_proj_qkv(step.hidden_out, w_post[0], step.total_out, step.D,
                                                                     step.q2, step.k2, step.v2), reps)
            br["attn_varlen"] = timed(lambda: step.ctx.d3tom_attn_varlen(step.q2, step.k2, step.v2, step.cu_out, step.nB,
                                                                        step.total_out, step.max_out, step.scale,
                                                                        step.layer_out[0]), reps)
        block = None
        if full:
            # the same routing applied to the cached K/V prefix (Sec. 4.4): caches = K, V rows of [visual | prompt]
            kv = make_kv_cache_case(step, w, k, v, dev)
            br["merge_kv"] = timed(kv, reps)
            # the rest of a post-merge block at N_m and at N (tensor-core path: bf16, widths in multiples of 128)
            if step.n_post and w.dtype == "bf16" and step.D % 128 == 0 and not args.no_block:
                block = block_timings(step, w, w_post[0], q, dev, timed, max(5, reps // 4))
                br["proj_out"] = block["Nm"]["proj_out"]
                br["ffn"] = block["Nm"]["ffn"]
        sync_all()
    finally:
        if clk_cm is not None:
            clk_cm.__exit__(None, None, None)
    if clk_cm is not None:
        res["clocks"] = clk_cm.summary()
    assert step.ctx.device_status() == 0, "device status word reports a kernel-side problem"

    peaks, peak_kind = load_peaks()
    # ---- every kernel of the step inside running steps (outside the timed regions)
    if w.dtype == "bf16":
        for _ in range(3):
            run_host_mid()
        torch.cuda.synchronize()
        res["kernels"] = kernel_profile(step, run_host_mid, q, peaks, n_steps=10 if full else 5)
        # what a plain device copy of the aggregation's bytes takes when issued back to back (same launch cost,
        # source resident in L2 when it fits): the practical bound for that kernel at this size
        agg = res["kernels"].get("aggregate_compact") if isinstance(res["kernels"], dict) else None
        if agg is not None:
            half = int(agg["mbytes"] * 1e6 / 2) // 2
            src = torch.empty(half, dtype=torch.bfloat16, device=dev)
            dst = torch.empty_like(src)
            for _ in range(3):
                dst.copy_(src)
            agg["plain_copy_same_bytes_us"] = timed(lambda: dst.copy_(src), 20)
            del src, dst

    # ---- end to end through the C ABI with host buffers: H2D of Q,K,V, the step, D2H of the result.
    #      HostFedStep overlaps the input copy of the next step and the result copy of the previous one with the
    #      running step (two input slots, three streams); the serial figure (copy, run, copy on one stream) is
    #      reported beside it.
    e2e_bytes = {"h2d": 0, "d2h": 0, "n": 0}
    # (graphs only with a single problem: with one graph per schedule step and slot on top of the graphs above, replay
    #  was measured slower than host launches, 1.8 against 1.0 ms per step; the copies bound this path either way)
    feed = HostFedStep(step, q, w_post, use_graphs=graphs is not None and n_prob == 1)

    def e2e():
        i = counter["i"] % n_prob
        counter["i"] += 1
        n_out = feed.submit(q_hs[i], k_h, v_h, out_h, probs[i], key=i)
        e2e_bytes["h2d"] += 3 * q.numel() * q.element_size()
        e2e_bytes["d2h"] += n_out * step.D * q.element_size()
        e2e_bytes["n"] += 1

    def e2e_serial():
        i = counter["i"] % n_prob
        counter["i"] += 1
        step.use_problem(probs[i])
        q_stage.copy_(q_hs[i], non_blocking=True); k.copy_(k_h, non_blocking=True); v.copy_(v_h, non_blocking=True)
        y = step.run(q_stage, k, v, w_post)
        out_h[:step.total_out].copy_(y[:step.total_out], non_blocking=True)

    def timed_fed(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            e2e()
        feed.wait()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / iters * 1e3
    for _ in range(4):                                                   # warm-up; records the graph of either slot
        e2e()
    feed.wait()
    sync_all()
    counter["i"] = 0
    e2e_bytes.update(h2d=0, d2h=0, n=0)
    e2e_us = timed_fed(max(n_prob, min(50, max(5, args.steps // 2))))
    sync_all()
    e2e_serial_us = None
    if full:
        for _ in range(3):
            e2e_serial()
        sync_all()
        counter["i"] = 0
        e2e_serial_us = timed(e2e_serial, max(n_prob, min(20, max(5, args.steps // 4))))
        sync_all()
    step.use_problem(probs[mid])

    step_us_max = replicas.max_over_ranks(step_us, dev)
    e2e_us_max = replicas.max_over_ranks(e2e_us, dev)

    # ---- roofline of the dominant kernel (merge-layer attention): 4 N^2 D flops per request
    attn_flops = sum(4.0 * n * n * step.D for n in step.seqlens_h)
    achieved = attn_flops / (attn_kernel_us * 1e-6) / 1e12
    res["roofline"] = {"bound": "tensor", "kernel": "attn_sk_kernel / attn_tc_kernel (merge-layer attention, timed alone; one request with uneven rounds takes the balanced walk)",
                       "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                       "frac": achieved / peaks["bf16_tflops"], "traffic": ATTN_TRAFFIC_BYTES.get(name),
                       "algorithmic_bytes": 4.0 * step.total * step.D * q.element_size(),
                       "peak_kind": peak_kind + " burst",
                       "frac_nominal": achieved / NOMINAL_PEAKS["bf16_tflops"],
                       "frac_measured_sustained": achieved / peaks["bf16_tflops_sustained"],
                       "us": attn_kernel_us, "us_median": float(np.median(attn_each)), "us_min": float(min(attn_each)),
                       "launches_timed": len(attn_each), "warmup_launches": 5}
    merge_bytes = (step.total + step.total_out) * step.D * q.element_size()
    sim_flops = sum(2.0 * (v_ - k_) * k_ * step.D for v_, k_ in zip(step.n_visual_h, step.keep_h))
    post_attn_flops = sum(4.0 * n * n * step.D for n in step.out_lens_h)
    derived = {
        "attn_importance_tflops": attn_flops / (br["attn_importance"] * 1e-6) / 1e12,
        "attn_importance_frac_of_burst": attn_flops / (br["attn_importance"] * 1e-6) / 1e12 / peaks["bf16_tflops"],
        "merge_call_gbs": merge_bytes / (br["merge"] * 1e-6) / 1e9,
        "merge_call_frac_of_hbm_peak": merge_bytes / (br["merge"] * 1e-6) / 1e9 / peaks["hbm_gbs"],
        "similarity_gflop": sim_flops / 1e9,
    }
    if step.n_post:
        derived["attn_varlen_tflops"] = post_attn_flops / (br["attn_varlen"] * 1e-6) / 1e12
        derived["proj_qkv_tflops"] = 2.0 * step.total_out * step.D * 3 * step.D / (br["proj_qkv"] * 1e-6) / 1e12
    res.update(step_us=step_us_max, step_us_this_rank=step_us, step_us_median=float(np.median(each)),
               step_us_min=float(np.min(each)), breakdown_us=br, derived=derived, dtype=w.dtype,
               e2e={"value": e2e_us_max / world, "unit": "us",
                    "h2d_bytes_per_step": int(e2e_bytes["h2d"] // max(1, e2e_bytes["n"])),
                    "d2h_bytes_per_step": int(e2e_bytes["d2h"] // max(1, e2e_bytes["n"])),
                    "how": "copies of neighbouring steps overlap the running step (two input slots, three streams)"})
    if e2e_serial_us is not None:
        res["e2e"]["serial_us"] = e2e_serial_us / world
    if block is not None:
        res["block"] = block
    res["peaks"] = dict(peaks, kind=peak_kind)
    res["_workload"] = w
    res["_mid"] = (dec_steps[mid], keep_steps[mid], mid)
    step.ctx.close()
    return res


# ------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="C2", choices=sorted(WORKLOAD_TEXT))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-block", action="store_true", help="skip the timing of the rest of a post-merge block")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--tokens-per-step", type=int, default=1,
                    help="schedule config: response tokens revealed per denoising step (2 gives T = 32 for 64 tokens)")
    ap.add_argument("--reversed", action="store_true", help="schedule config: the high->low ablation of the schedule")
    ap.add_argument("--deciders", default="all", choices=["all", "recent"],
                    help="schedule config: every token revealed so far, or only those of the previous step")
    ap.add_argument("--no-graph", action="store_true", help="enqueue every kernel of a step from the host instead of replaying a CUDA graph")
    ap.add_argument("--only", default=None, choices=["attn_importance", "attn_alone", "select", "merge", "proj_qkv", "attn_varlen", "proj_out", "ffn", "step", "dense_ab"],
                    help="profiling aid: after one full step, run just this call --steps times and exit")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        return spawn_ranks(args)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    config = {"workload": WORKLOAD_TEXT[args.config], "requests_per_gpu": None, "aggregation": "mean",
              "l2": "inputs larger than L2 (per-step working set > 126 MB)",
              "parallelism": "request-sharded replicas x%d" % world,
              "unit_of_work": "one merge-layer step of one request batch of the workload; every GPU runs its own batch, "
                              "value = slowest rank's time per step / number of GPUs"}

    if args.impl == "reference":
        if rank != 0:
            return 0
        return reference_arm(args, config)

    import torch
    import torch.distributed as dist
    from paper_2511_12280_b200 import binding as B_

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the merge-layer path has no CPU fallback")
    if local_rank >= torch.cuda.device_count():
        raise SystemExit("rank %d has no GPU: %d visible" % (local_rank, torch.cuda.device_count()))
    B_.load()           # fails loudly if the CUDA library has not been built
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    res = measure_config(args.config, args, dev, local_rank, world, full=True)
    if args.only is not None:
        print(json.dumps(res))
        return 0
    w = res.pop("_workload")
    mid_dec, mid_keep, mid = res.pop("_mid")
    config["requests_per_gpu"] = res.pop("requests_per_gpu")
    config["launch"] = res.pop("launch")
    if "schedule" in res:
        config["schedule"] = res.pop("schedule")
    step_us = res.pop("step_us")
    line = {
        "metric": "merge_layer_step_us", "value": step_us / world, "unit": "us", "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": step_us / 1e3,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if res.pop("dtype") == "bf16" else "f32", "data": "synthetic", "config": config,
        "steps_per_s": world / (step_us * 1e-6),
        "step_us_median": res.pop("step_us_median"), "step_us_min": res.pop("step_us_min"),
        "step_us_after_idle": res.pop("step_us_after_idle", None),
        "e2e": res.pop("e2e"), "gpu_launches": int(res.pop("gpu_launches")),
        "roofline": res.pop("roofline"), "breakdown_us": res.pop("breakdown_us"), "derived": res.pop("derived"),
        "clocks": res.pop("clocks"), "peaks": res.pop("peaks"),
    }
    res.pop("step_us_this_rank", None); res.pop("steps_timed", None); res.pop("total_tokens", None)
    if "per_step_us" in res:
        line["per_step_us"] = res["per_step_us"]
        line["trajectory_total_us"] = float(sum(res.pop("per_step_us")))
    line.update(res)                       # kernels, block, trajectory

    # ---- the other configurations, briefly (one GPU; the chosen configuration is the one the metric is quoted on)
    if world == 1 and not args.no_configs:
        others = {}
        for name in ("C1", "C3", "C4"):
            if name == args.config:
                continue
            r = measure_config(name, args, dev, local_rank, world, full=False)
            o = {"workload": WORKLOAD_TEXT[name], "step_us": r["step_us"], "step_us_median": r["step_us_median"],
                 "step_us_min": r["step_us_min"], "steps_timed": r["steps_timed"],
                 "attn_kernel_us": r["roofline"]["us"], "attn_tflops": r["roofline"]["achieved"],
                 "attn_frac": r["roofline"]["frac"], "attn_frac_nominal": r["roofline"]["frac_nominal"],
                 "e2e_us": r["e2e"]["value"], "h2d_bytes_per_step": r["e2e"]["h2d_bytes_per_step"],
                 "d2h_bytes_per_step": r["e2e"]["d2h_bytes_per_step"], "breakdown_us": r["breakdown_us"],
                 "kernels": r.get("kernels")}
            if "trajectory" in r:
                o["trajectory"] = r["trajectory"]
            others[name] = o
        line["configs"] = others

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        kw = {}
        if w.T:
            kw = dict(decider_pos=mid_dec, keep=mid_keep)
            config["cpu_baseline_step"] = mid
        sec, parts = oracle_step(w, oracle_inputs(w, kw.get("decider_pos")), **kw)
        line["cpu_baseline"] = {"value": sec * 1e6, "unit": "us", "cores": blas_threads(), "kind": "oracle",
                                "sample": ORACLE_SAMPLE_TEXT, "steps_timed": 1, "extrapolated": False,
                                "breakdown_s": parts}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
