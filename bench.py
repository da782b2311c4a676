#!/usr/bin/env python
"""Benchmark of the HyperAttention forward pass (one step = one whole forward: hash, sample,
sort, attention tiles, merge) on synthetic inputs of the baseline's shapes.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3|c2|c4|c5|c1] [--impl reference]

The default workload is the causal 131072-row configuration (c3); the 32768-row configuration (c2) is
measured in the same run and reported under `also`.  With --gpus N > 1 and no torchrun environment the
script starts the N ranks itself.

Prints ONE JSON line.  `value` is tokens/s with inputs resident in HBM; `e2e` is the same
metric through the host-buffer entry point (pinned host memory, copies inside the timed
region); `roofline` describes the dominant kernel (the attention tiles); `kernels` lists every
stage with its own bound; `cpu_baseline` is the NumPy oracle timed on the host cores on a
bounded sample of the same workload (a reported baseline, not a target), together with the
GPU-vs-oracle error on that sample.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2310_05869_b200 import workloads as WL  # noqa: E402

WORKLOADS = {"c1": 0, "c2": 1, "c3": 2, "c4": 3, "c5": 4}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the attention kernel,
# from the ncu captures summarised under profiles/ (taken on 4 / 8 heads and scaled to the
# workload's 32 heads: the traffic is proportional to the number of segments).
NCU_TRAFFIC_BYTES = {"c3_n131k_causal": 8 * 0.9292e9, "c2_n32k_d128": 4 * 0.2453e9}
# sm__pipe_tensor_cycles_active (% of peak sustained active) of the attention kernel in the same captures
NCU_TENSOR_PIPE_PCT = {"c3_n131k_causal": 26.0, "c2_n32k_d128": 27.1}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return dict(FALLBACK_PEAKS, source="fallback")


# ---------------------------------------------------------------- algorithmic work per forward
def work_model(w: WL.Workload):
    """Algorithmic flops / bytes of each stage for one forward (what the method itself has to
    compute or move, not what a particular kernel happens to do)."""
    G, n, d, e = w.G, w.n, w.d, (2 if w.dtype == "bf16" else 4)
    nodes = []  # (count per segment, size)
    leaves = []
    if not w.causal:
        if w.b < n:
            nodes.append((1, n))
        else:
            leaves.append((1, n, False))
    elif n <= w.n0:
        leaves.append((1, n, True))
    else:
        L = 0
        while (n >> L) > w.n0:
            L += 1
        for l in range(L):
            nodes.append((1 << l, n >> (l + 1)))
        leaves.append((1 << L, n >> L, True))
    flops = 0.0
    sorted_rows = 0
    for cnt, s in nodes:
        if w.b < s:
            flops += cnt * 4.0 * s * (w.b + w.m) * d
            sorted_rows += cnt * s
        else:
            flops += cnt * 4.0 * s * s * d
    for cnt, s, causal in leaves:
        flops += cnt * (4.0 * d * s * (s + 1) / 2 if causal else 4.0 * s * s * d)
    flops *= G
    any_sorted = sorted_rows > 0
    hash_bytes = 2.0 * G * n * (d * e + 1) if any_sorted else 0.0
    sort_bytes = G * sorted_rows * (2 * 1 + 4 + 4 + 4)        # ids of Q and K rows, perm_q, perm_k, rank_k
    merge_bytes = 0.0
    if w.causal and n > w.n0:
        L = 0
        while (n >> L) > w.n0:
            L += 1
        # partial rows travel in the output's type (bf16 here), their log-sum-exp in fp32
        merge_bytes = G * n * ((1 + L / 2.0) * (e * d + 4) + d * e + 4)
    dense_flops = G * (4.0 * n * n * d) * (0.5 if w.causal else 1.0)
    return {"attention_flops": flops, "hash_bytes": hash_bytes, "sort_bytes": float(sort_bytes),
            "merge_bytes": merge_bytes, "dense_attention_flops": dense_flops}


# ---------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------- oracle leg
def oracle_sample_plan(w: WL.Workload, leg: str):
    """Which part of the workload the oracle is timed on: whole segments, and for causal
    workloads a bounded set of query rows per segment (hashing and sorting always cover the
    whole segment).  leg "baseline" (run once, ~10-30 s of CPU work) or "step" (one step of the
    reference arm, ~1-2 s)."""
    def spread(k):
        k = min(k, w.G)
        return sorted({(i * (w.G - 1)) // max(k - 1, 1) for i in range(k)})
    if w.n <= 2048:
        return {"segments": spread(w.G), "rows": None}
    if w.causal:
        return {"segments": spread(8 if leg == "baseline" else 2), "rows": 16384 if leg == "baseline" else 4096}
    per_seg_cost = w.n / 32768.0
    k = max(1, int((32 if leg == "baseline" else 4) / per_seg_cost))
    return {"segments": spread(k), "rows": None}


def run_oracle_sample(w: WL.Workload, arrs, plan, ids=None):
    """Runs the oracle on the planned sample.  Returns (seconds, {seg: (rows, out, lse)})."""
    from oracle import hyperattn_oracle as O
    res = {}
    t0 = time.perf_counter()
    W = O.directions(w.d, w.r, w.seed)
    rng = np.random.default_rng(12345)
    for g in plan["segments"]:
        Q, K, V = (WL.as_f64(x[g]) for x in arrs)
        rows = None
        if plan["rows"] is not None and plan["rows"] < w.n:
            rows = np.sort(rng.choice(w.n, size=plan["rows"], replace=False))
        iq = ik = None
        if ids is not None:
            iq, ik = ids[0][g], ids[1][g]
        o, l = O.segment_forward(Q, K, V, W, w.b, w.m, w.causal, w.n0, w.seed, g, scale=1.0 / math.sqrt(w.d),
                                 rows=rows, ids_q=iq, ids_k=ik)
        res[g] = (np.arange(w.n) if rows is None else rows, o, l)
    return time.perf_counter() - t0, res


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def sample_tokens(w, plan):
    per_seg = w.n if plan["rows"] is None else min(plan["rows"], w.n)
    return per_seg * len(plan["segments"]) / w.H          # tokens = rows of one head set / H heads


def warmup_steps(args):
    """Warm-up steps actually run (the timing rules ask for at least three); the same for both arms."""
    return max(args.warmup, 3)


def reference_arm(args, w):
    """The oracle timed on the host cores: each step is the bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    arrs = make_sample_inputs(w)
    plan = oracle_sample_plan(w, "step")
    for _ in range(warmup_steps(args)):
        run_oracle_sample(w, arrs, plan)
    times = []
    for _ in range(args.steps):
        dt, _ = run_oracle_sample(w, arrs, plan)
        times.append(dt)
    tot = sum(times)
    toks = sample_tokens(w, plan) * args.steps
    value = toks / tot
    desc = describe_sample(w, plan)
    line = {"impl": "reference", "metric": "forward tokens/s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": warmup_steps(args), "ms_per_step": 1e3 * tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w),
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": host_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def describe_sample(w, plan):
    rows = "all rows" if plan["rows"] is None else f"{plan['rows']} random rows per segment (hash and sort of the whole segment)"
    return f"segments {plan['segments']} of {w.G} of workload {w.name}, {rows}; tokens counted as rows/H"


def make_sample_inputs(w):
    return WL.make_inputs(w)


def config_dict(w):
    return {"workload": w.name, "B": w.B, "H": w.H, "n": w.n, "d": w.d, "block": w.b, "samples": w.m,
            "hash_bits": w.r, "causal": w.causal, "n0": w.n0, "input_kind": w.kind,
            "l2": "inputs exceed L2 (no flush)" if w.G * w.n * w.d * 2 * 3 > 126e6 else "inputs fit L2; 256 MB flush buffer written between steps"}


# ---------------------------------------------------------------- GPU arm
def stage_report(w, peaks, stage_ms):
    """Per-stage roofline figures from the stages' mean launch times (ms)."""
    wm = work_model(w)
    burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    att_ms = stage_ms["attention"]
    att_tflops = wm["attention_flops"] / (att_ms * 1e-3) / 1e12 if att_ms > 0 else 0.0
    # The timed region is milliseconds long and runs at the maximum SM clock, so the like-for-like
    # denominator is the burst GEMM peak; the fraction of the sustained (power-capped) peak is given too.
    roofline = {"kernel": "attention tiles (block + sampled + causal leaves)", "bound": "tensor", "achieved": att_tflops,
                "peak": burst, "unit": "TFLOP/s", "frac": att_tflops / burst,
                "peak_source": f"bf16_tflops (burst) of {peaks['source']}",
                "frac_of_sustained_peak": att_tflops / sustained, "sustained_peak": sustained,
                "ms_per_launch": att_ms, "traffic": NCU_TRAFFIC_BYTES.get(w.name),
                "tensor_pipe_active_pct": NCU_TENSOR_PIPE_PCT.get(w.name),
                "counters_from": "ncu capture on a reduced-head slice, see profiles/"}
    kernels = {}
    for s_, key in (("hash", "hash_bytes"), ("merge", "merge_bytes")):
        if stage_ms.get(s_, 0) > 0:
            gbs = wm[key] / (stage_ms[s_] * 1e-3) / 1e9
            kernels[s_] = {"bound": "hbm", "ms": stage_ms[s_], "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                           "frac": gbs / peaks["hbm_gbs"]}
    sort_ms = stage_ms.get("sort_scan", 0) + stage_ms.get("sort_scatter", 0)
    if sort_ms > 0:
        gbs = wm["sort_bytes"] / (sort_ms * 1e-3) / 1e9
        kernels["sort"] = {"bound": "hbm", "ms": sort_ms, "ms_scan": stage_ms["sort_scan"], "ms_scatter": stage_ms["sort_scatter"],
                           "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"]}
    kernels["attention"] = {"bound": "tensor", "ms": att_ms, "achieved": att_tflops, "peak": burst, "unit": "TFLOP/s",
                            "frac": att_tflops / burst, "frac_of_sustained_peak": att_tflops / sustained}
    kernels["sample"] = {"ms": stage_ms.get("sample", 0.0), "note": "drawn by extra blocks of the sort_scan launch"}
    return wm, roofline, kernels


def measure_device(w, args, ha, RK, info, dev, peaks, steps):
    """Whole forwards on device-resident inputs: W warm-up steps, `steps` timed steps between barriers
    (CUDA events on the call's stream, max over ranks), then a per-call pass that times every stage."""
    import torch
    arrs = WL.make_inputs(RK.rank_workload(w, info.rank))

    def dev_tensor(x):
        if x.dtype == np.uint16:
            return torch.from_numpy(x.view(np.int16)).to(dev).view(torch.bfloat16).view(w.B, w.H, w.n, w.d)
        return torch.from_numpy(x).to(dev).view(w.B, w.H, w.n, w.d)

    q, k, v = (dev_tensor(x) for x in arrs)
    small = w.G * w.n * w.d * 2 * 3 <= 126e6
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None
    stream = torch.cuda.current_stream(dev)

    def step():
        if flush is not None:
            flush.fill_(1)
        return ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)

    def barrier():
        RK.barrier(info)
        torch.cuda.synchronize(dev)

    for _ in range(warmup_steps(args)):
        out, lse = step()
    barrier()
    # ---- timed region: K whole forwards, device time; the dominant kernel (attention) is bracketed
    # by events inside it, the other stages are timed in the per-call pass below (an event pair
    # around every small kernel would put gaps between them) ------------------------------------
    ha.profile_reset()
    ha.profile_enable(True, stages=["attention"])
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    flush_ms = 0.0
    barrier()
    e0.record(stream)
    for _ in range(steps):
        out, lse = step()
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    prof = ha.profile_read()
    ha.profile_enable(False)
    ha.profile_reset()
    if flush is not None:   # subtract the flush writes (timed separately)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for _ in range(steps):
            flush.fill_(1)
        f1.record(stream)
        torch.cuda.synchronize(dev)
        flush_ms = f0.elapsed_time(f1)
    ms_total = max(ms_total - flush_ms, 1e-6)
    ms_total = RK.max_over_ranks(info, ms_total, dev)
    value = RK.job_throughput(info, w.B * w.n, steps, ms_total)

    # ---- per-call latency distribution (outside the timed region: one event pair per call) ------
    lat_steps = max(5, min(steps, 30))
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(lat_steps)]
    ha.profile_enable(True)
    for a0, a1 in evs:
        if flush is not None:
            flush.fill_(1)
        a0.record(stream)
        ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
        a1.record(stream)
    torch.cuda.synchronize(dev)
    prof_all = ha.profile_read()
    ha.profile_enable(False)
    ha.profile_reset()
    lat = sorted(a0.elapsed_time(a1) for a0, a1 in evs)
    latency = {"median_ms": lat[len(lat) // 2], "min_ms": lat[0], "calls": lat_steps}

    calls = max(prof["calls"], 1)
    calls_all = max(prof_all["calls"], 1)
    # every stage from the per-call pass; the attention kernel from the timed region itself
    stage_ms = {s_: prof_all["ms"][s_] / calls_all for s_ in prof_all["ms"]}
    launches = {s_: prof_all["launches"][s_] // calls_all for s_ in prof_all["launches"]}
    stage_ms["attention"] = prof["ms"]["attention"] / calls
    wm, roofline, kernels = stage_report(w, peaks, stage_ms)
    ms_step = ms_total / steps
    dense_ms = wm["dense_attention_flops"] / (peaks["bf16_tflops"] * 1e12) * 1e3
    rec = {"value": value, "ms_per_step": ms_step, "steps": steps, "latency_per_call": latency,
           "dense_attention_roofline_ms": dense_ms, "speedup_vs_dense_roofline": dense_ms / ms_step,
           "launches_per_step": launches, "roofline": roofline, "kernels": kernels}
    return rec, (arrs, q, k, v, out, lse)


def gpu_arm(args, w):
    import torch
    import paper_2310_05869_b200 as ha
    from paper_2310_05869_b200 import ranks as RK

    info = RK.rank_env()
    world, rank, local = info.world, info.rank, info.local_rank
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    RK.init(info, "nccl", dev)
    peaks = load_peaks()
    stream = torch.cuda.current_stream(dev)

    def barrier():
        RK.barrier(info)
        torch.cuda.synchronize(dev)

    sampler = ClockSampler(local) if rank == 0 else None
    # every rank owns its own B*H segments (weak scaling: no exchange between segments)
    main_rec, (arrs, q, k, v, out, lse) = measure_device(w, args, ha, RK, info, dev, peaks, args.steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- backward pass (on request): the derivative of the same call, timed on its own ------------
    backward = None
    if args.backward and w.dtype == "bf16":
        out_b, lse_b = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
        dout = torch.randn(q.shape, device=dev, dtype=torch.float32).to(torch.bfloat16)
        for _ in range(2):
            ha.backward(q, k, v, out_b, lse_b, dout, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
        bsteps = max(3, min(args.steps, 10))
        barrier()
        e0.record(stream)
        for _ in range(bsteps):
            ha.backward(q, k, v, out_b, lse_b, dout, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
        e1.record(stream)
        barrier()
        bms = RK.max_over_ranks(info, e0.elapsed_time(e1), dev) / bsteps
        bflops = 2.5 * work_model(w)["attention_flops"]          # five contractions per tile instead of two
        backward = {"ms_per_call": bms, "flops": bflops, "achieved_tflops": bflops / (bms * 1e-3) / 1e12,
                    "frac_of_bf16_burst": bflops / (bms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "frac_of_bf16_sustained": bflops / (bms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                    "path": "tcgen05 / TMEM, fp32 global reductions", "steps": bsteps}
        del out_b, lse_b, dout

    # ---- end to end through the host-buffer entry point ---------------------------------------
    hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
    ho = torch.empty(q.shape, dtype=q.dtype).pin_memory()
    hl = torch.empty((w.B, w.H, w.n), dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    for _ in range(2):
        ha.forward_host(hq, hk, hv, ho, hl, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        ha.forward_host(hq, hk, hv, ho, hl, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed)
    e1.record(stream)
    barrier()
    e2e_ms = RK.max_over_ranks(info, e0.elapsed_time(e1), dev)
    es = q.element_size()
    h2d = 3 * q.numel() * es
    d2h = ho.numel() * ho.element_size() + hl.numel() * 4
    e2e = {"value": RK.job_throughput(info, w.B * w.n, e2e_steps, e2e_ms), "unit": "tokens/s", "ms_per_step": e2e_ms / e2e_steps,
           "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    assert torch.equal(ho.to(dev), out), "host-buffer entry point disagrees with the device entry point"
    del hq, hk, hv, ho, hl
    clocks = sampler.stop() if sampler else None

    # ---- the other half of the metric: the 32768-row configuration in the same run ----------------
    also = {}
    if args.also and w.name == WL.CONFIGS[WORKLOADS["c3"]].name:
        w2 = WL.CONFIGS[WORKLOADS["c2"]]
        rec2, keep = measure_device(w2, args, ha, RK, info, dev, peaks, args.steps)
        del keep
        rec2["config"] = config_dict(w2)
        rec2["unit"] = "tokens/s"
        also["c2"] = rec2

    if rank != 0:
        RK.shutdown(info)
        return

    # ---- oracle on the host cores: bounded sample, plus the error of the GPU result on it -----
    cpu = None
    if not args.no_cpu_baseline:
        from oracle import hyperattn_oracle as O
        plan = oracle_sample_plan(w, "baseline")
        out32, lse32, inter = ha.forward(q, k, v, w.b, w.m, w.r, causal=w.causal, n0=w.n0, seed=w.seed,
                                         out_dtype=torch.float32, debug=True)
        torch.cuda.synchronize(dev)
        any_sorted = w.b < (w.n if not w.causal else w.n // 2) and not (w.causal and w.n <= w.n0)
        # timed: the oracle's own whole forward (its own hash included) on the sample
        secs, res = run_oracle_sample(w, arrs, plan, None)
        # bucket ids of the sampled segments, oracle against GPU: rows whose ids differ (hash bits with a
        # projection next to zero, decided in fp32 on the GPU); if there are any, the comparison of the
        # outputs is repeated (untimed) with the GPU's ids given to the oracle
        mism = 0
        if any_sorted:
            Wd = O.directions(w.d, w.r, w.seed)
            gq, gk = inter["q_ids"].cpu().numpy(), inter["k_ids"].cpu().numpy()
            for g in plan["segments"]:
                mism += int((O.bucket_ids(WL.as_f64(arrs[0][g]), Wd)[0] != gq[g]).sum())
                mism += int((O.bucket_ids(WL.as_f64(arrs[1][g]), Wd)[0] != gk[g]).sum())
            if mism:
                _, res = run_oracle_sample(w, arrs, plan, (gq, gk))
        o_np = out32.view(w.G, w.n, w.d)
        l_np = lse32.view(w.G, w.n)
        errs, lerrs = [], []
        for g, (rows, ro, rl) in res.items():
            idx = torch.from_numpy(rows).to(dev)
            errs.append(np.abs(o_np[g][idx].cpu().numpy() - ro).reshape(-1))
            lerrs.append(np.abs(l_np[g][idx].cpu().numpy() - rl) / np.maximum(np.abs(rl), 1.0))
        err = np.concatenate(errs)
        lerr = np.concatenate(lerrs)
        cpu = {"value": sample_tokens(w, plan) / secs, "unit": "tokens/s", "cores": host_threads(), "kind": "oracle",
               "sample": describe_sample(w, plan), "seconds": secs,
               "gpu_vs_oracle": {"out_max_abs": float(err.max()), "out_max_abs_bound": 2e-2, "out_mean_abs": float(err.mean()),
                                 "out_mean_abs_bound": 2e-3, "lse_max_rel": float(lerr.max()), "lse_rel_bound": 1e-3,
                                 "rows": int(lerr.size), "rows_with_different_bucket_id": mism,
                                 "ids_given_to_oracle": bool(mism),
                                 "near_zero_hash_bits": int(inter["near_zero_bits"].item())}}

    line = {"metric": "forward tokens/s", "value": main_rec["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": warmup_steps(args), "ms_per_step": main_rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic", "config": config_dict(w),
            "latency_per_call": main_rec["latency_per_call"], "latency_ms": main_rec["ms_per_step"],
            "dense_attention_roofline_ms": main_rec["dense_attention_roofline_ms"],
            "speedup_vs_dense_roofline": main_rec["speedup_vs_dense_roofline"],
            "e2e": e2e, "gpu_launches": sum(main_rec["launches_per_step"].values()) * args.steps,
            "launches_per_step": main_rec["launches_per_step"],
            "roofline": main_rec["roofline"], "kernels": main_rec["kernels"], "cpu_baseline": cpu, "clocks": clocks,
            "peaks": peaks}
    if also:
        line["also"] = also
    if backward is not None:
        line["backward"] = backward
    print(json.dumps(line))
    RK.shutdown(info)


def free_port():
    import socket
    with socket.socket() as s_:
        s_.bind(("127.0.0.1", 0))
        return s_.getsockname()[1]


def spawn_ranks(n, argv):
    """Starts this script as n ranks of one node (one process per GPU) through torch.distributed.run and
    returns its exit code; used when --gpus N > 1 is asked for outside a torchrun environment."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--no-also", dest="also", action="store_false", help="with the default workload: skip the c2 sub-record")
    ap.add_argument("--n", type=int, default=0, help="override the sequence length (c4 sweep)")
    ap.add_argument("--heads", type=int, default=0, help="override H (smaller cases for profiler captures)")
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--backward", action="store_true", help="also time the backward pass (an extra key of the JSON line)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    w = WL.CONFIGS[WORKLOADS[args.workload]]
    if args.n:
        w = w.scaled(n=args.n, name=f"{w.name}_n{args.n}")
    if args.heads:
        w = w.scaled(H=args.heads, name=f"{w.name}_h{args.heads}")
    if args.impl == "reference":
        reference_arm(args, w)
    else:
        gpu_arm(args, w)


if __name__ == "__main__":
    main()
