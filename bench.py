#!/usr/bin/env python
"""Benchmark of the chunked-prefill attention path on B200.

A "step" is one pass of the whole hot path (work decomposition -> attention -> merge when split) over
one batch of synthetic input: the GQA long-context chunk (64 q-heads, 4 kv-heads, head_dim 128, chunk of
8192 tokens, 128-token pages with a shuffled block table) evaluated once at each of its prefix lengths
0, 8K, 32K, 64K and 128K.  The reported value is the aggregate TFLOP/s of a step (exact causal flop
count); the per-prefix latency / TFLOP/s curve -- the cost curve the paper's V-shaped layout is built
around -- is reported beside it in "curve".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload ...]

One JSON line on stdout (rank 0).  With --impl reference the CPU oracle is timed on the host cores on a
bounded sample of the same workload.  The default run (one GPU) also times the other four benchmark
configurations, each with its own clock sample and oracle baseline, and reports them under "configs".
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2608_26523_b200 import dist as D, workloads as W

METRIC = "chunk-attn TFLOP/s and % dense BF16 peak vs prefix length (1 B200)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        res = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return res
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
                except ValueError:
                    continue
                for n, v in zip(names, parts[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
        os.unlink(self.path)
        if sm:
            res.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return res


def oracle_sample_rate(prob_cpu, target_seconds, rng):
    """Time the fp64 oracle (as it stands) on random (request, row, head) samples of the workload.

    Returns (flops done, seconds, rows, threads)."""
    import oracle
    c = prob_cpu.chunk_len.numpy().astype(np.int64)
    pre = prob_cpu.prefix_len.numpy().astype(np.int64)
    req_of_row = np.repeat(np.arange(len(c)), c)             # packed row -> request
    row_in_req = np.concatenate([np.arange(x) for x in c]) if len(c) else np.zeros(0, np.int64)
    hq = prob_cpu.num_q_heads
    per_row = 2.0 * (prob_cpu.head_dim_qk + prob_cpu.head_dim_v)

    def run(n):
        pick = rng.integers(0, len(req_of_row), n)
        rows = np.stack([req_of_row[pick], row_in_req[pick], rng.integers(0, hq, n)], axis=1).astype(np.int32)
        t0 = time.perf_counter()
        oracle.ref_chunk_attn_rows(prob_cpu.q, prob_cpu.k_cache, prob_cpu.v_cache,
                                   prob_cpu.k_cache.stride()[:3], prob_cpu.v_cache.stride()[:3],
                                   None if prob_cpu.block_table is None else prob_cpu.block_table.numpy(),
                                   prob_cpu.block_size, prob_cpu.prefix_len.numpy(), prob_cpu.chunk_len.numpy(),
                                   hq, prob_cpu.num_kv_heads, prob_cpu.head_dim_qk, prob_cpu.head_dim_v,
                                   prob_cpu.scale, rows)
        dt = time.perf_counter() - t0
        fl = float(((pre[rows[:, 0]] + rows[:, 1].astype(np.int64) + 1) * per_row).sum())
        return fl, dt

    threads = oracle.num_threads()
    fl, dt = run(4 * threads)                       # calibration batch
    n = int(max(threads, min(4 * threads * target_seconds / max(dt, 1e-3), 200000)))
    fl, dt = run(n)
    return fl, dt, n, threads


# Nominal dense bf16 tensor rate of a B200 (2.25 PFLOP/s; the vendor's doubled figures are with 2:4 sparsity): context beside the
# measured peaks, never the denominator of a claim.
NOMINAL_BF16_TFLOPS = 2250.0


def cpu_baseline_entry(prob_cpu, seconds, what):
    fl, dt, n, threads = oracle_sample_rate(prob_cpu, seconds, np.random.default_rng(0))
    rate = fl / dt
    return {"value": round(rate / 1e12, 6), "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%d random (row, head) pairs of %s (%.1f s of CPU time)" % (n, what, dt),
            "extrapolated_full_s": round(prob_cpu.flops() / rate, 1)}   # the whole launch at the sampled rate (not run)


def read_traffic_record(name):
    """DRAM bytes per launch of a kernel, as recorded beside its ncu summary (profiles/<name>): key = value lines."""
    path = os.path.join(ROOT, "profiles", name)
    rec = {}
    if os.path.exists(path):
        with open(path) as f:
            for line in f:
                if "=" in line and not line.lstrip().startswith("#"):
                    k, v = line.split("=", 1)
                    rec[k.strip()] = v.strip()
    return rec


def fit_cost_curve(prefixes, ms):
    """The paper's linear latency model (its Eq. 2) fitted to a measured curve, and its balance identity (its Eq. 3,
    tau(k-1) + tau(k+1) = 2 tau(k)) on the evenly spaced points of the curve."""
    x = np.array(prefixes, dtype=np.float64); y = np.array(ms, dtype=np.float64)
    if len(x) < 3:
        return None
    b, a = np.polyfit(x, y, 1)
    r2 = 1.0 - float(((y - (a + b * x)) ** 2).sum() / max(((y - y.mean()) ** 2).sum(), 1e-30))
    out = {"fit_ms": {"a": round(float(a), 5), "b_per_token": float(b), "r2": round(r2, 6)},
           "fit_residual_max_rel": round(float((np.abs(y - (a + b * x)) / y).max()), 5)}
    # every triple (i, j, k) of measured points with x_j - x_i == x_k - x_j is an instance of Eq. 3
    res = []
    for j in range(1, len(x) - 1):
        for i in range(j):
            for k in range(j + 1, len(x)):
                if x[j] - x[i] == x[k] - x[j]:
                    res.append(abs(y[i] + y[k] - 2 * y[j]) / (2 * y[j]))
    if res:
        out["eq3_residual_max"] = round(float(max(res)), 5)
        out["eq3_triples"] = len(res)
    return out


def time_points(runners, stream, steps, warmup, sampler=None):
    """warmup untimed passes over the runners, then `steps` timed ones; per-runner median ms (CUDA events on the launching
    stream), the whole region's ms per step, launches per step and the clock record."""
    from paper_2608_26523_b200 import api
    with torch.cuda.stream(stream):
        for _ in range(warmup):
            for r in runners:
                r.run(stream.cuda_stream)
        launches = 0
        for r in runners:
            r.run(stream.cuda_stream)
            launches += api.vpp_last_launch_count()
        stream.synchronize()
        for r in runners:
            assert int(r.status.item()) == 0, "device status %d" % int(r.status.item())
        if sampler is not None:
            sampler.start()
            time.sleep(0.25)
        ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in runners]
              for _ in range(steps)]
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record(stream)
        for s_ in range(steps):
            for i, r in enumerate(runners):
                ev[s_][i][0].record(stream)
                r.run(stream.cuda_stream)
                ev[s_][i][1].record(stream)
        t1.record(stream)
        stream.synchronize()
    clocks = sampler.stop() if sampler is not None else None
    per = [statistics.median(ev[s_][i][0].elapsed_time(ev[s_][i][1]) for s_ in range(steps)) for i in range(len(runners))]
    time_points.last_min = [min(ev[s_][i][0].elapsed_time(ev[s_][i][1]) for s_ in range(steps)) for i in range(len(runners))]
    return per, t0.elapsed_time(t1) / steps, launches, clocks


def sweep_other_configs(dev, peaks, steps, warmup, with_cpu):
    """The four benchmark configurations beside cfg 2, each timed by itself (own warm-up, own clock sample)."""
    from paper_2608_26523_b200 import api
    burst, sustained = float(peaks["bf16_tflops"]), float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    stream = torch.cuda.Stream(device=dev)
    out = {}

    def curve_of(prefixes, per_ms, flops):
        rows = []
        for P, ms, ms_min, fl in zip(prefixes, per_ms, time_points.last_min, flops):
            tf = fl / (ms * 1e-3) / 1e12
            rows.append({"prefix": P, "ms": round(ms, 4), "ms_min": round(ms_min, 4), "tflops": round(tf, 2),
                         "frac_of_burst": round(tf / burst, 4), "frac_of_sustained": round(tf / sustained, 4),
                         "frac_of_nominal": round(tf / NOMINAL_BF16_TFLOPS, 4)})
        return rows

    plans = [("cfg3", W.cfg3, W.CFG3_PREFIXES, 8192, 0, "absorbed MLA Hq=128 (576/512), chunk 8192, 64-token pages", 65536),
             ("cfg4", W.cfg4, [16384 * k for k in (0, 21, 42, 63)], 16384, 4,
              "GQA Hq=64 Hkv=8 d=128, chunk 16384, 128-token pages, split-KV S=4 + merge; 4 evenly spaced points of the 16", 65536)]
    for name, make, prefixes, chunk, splits, desc, cpu_prefix in plans:
        base = make(prefix=max(prefixes), max_prefix=max(prefixes), device=dev)
        runners = [api.ChunkAttn(base.with_chunk([P], [chunk], base.q), num_kv_splits=splits) for P in prefixes]
        per, step_ms, launches, clocks = time_points(runners, stream, steps, warmup, ClockSampler(dev.index or 0))
        flops = [r.prob.flops() for r in runners]
        entry = {"workload": "%s: %s" % (name, desc), "num_kv_splits": splits, "steps": steps, "warmup": warmup,
                 "curve": curve_of(prefixes, per, flops), "cost_curve": fit_cost_curve(prefixes, per),
                 "tflops": round(sum(flops) / (step_ms * 1e-3) / 1e12, 2), "gpu_launches": launches * steps, "clocks": clocks}
        del runners, base
        torch.cuda.empty_cache()
        if with_cpu:
            small = make(prefix=cpu_prefix, device=dev).to("cpu")
            entry["cpu_baseline"] = cpu_baseline_entry(small, 4.0, "the chunk at prefix %d" % cpu_prefix)
            del small
        out[name] = entry

    # cfg 5: one launch
    prob = W.cfg5(device=dev)
    runners = [api.ChunkAttn(prob, num_kv_splits=0)]
    per, step_ms, launches, clocks = time_points(runners, stream, max(steps, 5), warmup, ClockSampler(dev.index or 0))
    tf = prob.flops() / (per[0] * 1e-3) / 1e12
    kv_tokens = int((prob.prefix_len + prob.chunk_len).sum().item())
    out["cfg5"] = {"workload": "cfg5: 32 requests, 16384 packed query tokens, lengths log-uniform 1K-256K, Hq=64 Hkv=8 d=128, "
                               "128-token pages, one launch", "ms": round(per[0], 4), "tflops": round(tf, 2),
                   "frac_of_burst": round(tf / burst, 4), "frac_of_sustained": round(tf / sustained, 4),
                   "frac_of_nominal": round(tf / NOMINAL_BF16_TFLOPS, 4), "ms_min": round(time_points.last_min[0], 4),
                   "kv_tokens": kv_tokens, "gpu_launches": launches * max(steps, 5), "clocks": clocks}
    if with_cpu:
        out["cfg5"]["cpu_baseline"] = cpu_baseline_entry(prob.to("cpu"), 4.0, "the batch")
    del runners, prob
    torch.cuda.empty_cache()

    # cfg 1: four launches of 512 rows against one contiguous 2048-token cache (latency-bound: no roofline claimed)
    runners = [api.ChunkAttn(W.cfg1(k, device=dev), num_kv_splits=0) for k in range(4)]
    per, step_ms, launches, clocks = time_points(runners, stream, max(steps, 20), max(warmup, 5), ClockSampler(dev.index or 0))
    rows = []
    for k, (r, ms) in enumerate(zip(runners, per)):
        P = 512 * k
        byts = (P + 512) * 1 * 256 * 2 + 512 * 4 * 128 * 2 * 2 + 512 * 4 * 4      # K/V read once, q in, out + lse out
        rows.append({"prefix": P, "us": round(ms * 1e3, 2), "tflops": round(r.prob.flops() / (ms * 1e-3) / 1e12, 2),
                     "GB/s": round(byts / ms / 1e6, 1)})
    out["cfg1"] = {"workload": "cfg1: Hq=4 Hkv=1 d=128, 2048 tokens as 4 chunks of 512, contiguous cache; the whole problem is "
                               "L2-resident and 16 work items cannot fill 148 SMs: latency-bound, no roofline claimed",
                   "curve": rows, "us_per_chunk_mean": round(step_ms * 1e3 / 4, 2), "gpu_launches": launches * max(steps, 20),
                   "clocks": clocks}
    if with_cpu:
        import oracle
        full = W.cfg1(0, device="cpu").extra["full"]
        rows_all = oracle.all_rows(full.chunk_len.numpy(), 4)
        t0 = time.perf_counter()
        oracle.ref_chunk_attn_rows(full.q, full.k_cache, full.v_cache, full.k_cache.stride()[:3], full.v_cache.stride()[:3],
                                   None, full.block_size, full.prefix_len.numpy(), full.chunk_len.numpy(), 4, 1, 128, 128,
                                   full.scale, rows_all)
        dt = time.perf_counter() - t0
        out["cfg1"]["cpu_baseline"] = {"value": round(full.flops() / dt / 1e12, 6), "unit": UNIT, "cores": oracle.num_threads(),
                                       "kind": "oracle", "sample": "all 2048 rows x 4 heads (the four chunks; %.2f s)" % dt}
    return out


def bench_groups(args):
    """Group sizes: the same chunk (8192 rows at prefix 32768, d = 128, 128-token pages) with MHA, an odd group and an even
    group -- work items are two q-heads of a kv-head over 128 rows (even groups) or two 128-row tiles of one q-head (odd
    groups, MHA included); both run the pipelined kernel."""
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    prefix, chunk = (int(args.prefixes.split(",")[0]) if args.prefixes else 32768), 8192
    cases = [("MHA: Hq=32 Hkv=32", 32, 32), ("odd group: Hq=24 Hkv=8 (G=3)", 24, 8), ("even group: Hq=32 Hkv=8 (G=4)", 32, 8),
             ("MQA-like: Hq=32 Hkv=1 (G=32)", 32, 1)]
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    launches = 0
    for desc, hq, hkv in cases:
        prob = W.make_problem(W.BASE_SEED + 500 + hkv, [prefix], [chunk], hq, hkv, 128, 128, block_size=128, device=dev)
        runner = api.ChunkAttn(prob, num_kv_splits=args.splits)
        per, step_ms, nl, _ = time_points([runner], stream, max(args.steps, 5), max(args.warmup, 3))
        launches += nl * max(args.steps, 5)
        tf = prob.flops() / (per[0] * 1e-3) / 1e12
        rows.append({"case": desc, "ms": round(per[0], 4), "tflops": round(tf, 1), "frac_of_burst": round(tf / peaks["bf16_tflops"], 4)})
        del prob, runner
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = rows[0]
    print(json.dumps({"metric": "chunk attention TFLOP/s by group size (1 B200)", "value": top["tflops"], "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": top["ms"], "higher_is_better": True, "dtype": "bf16",
                      "data": "synthetic", "vs_baseline": None,
                      "config": {"workload": "groups; chunk %d at prefix %d, d=128, 128-token pages; %s" % (chunk, prefix, top["case"]),
                                 "l2": "K/V of the MHA case (%d MB) exceeds the L2" % ((prefix + chunk) * 32 * 512 // 1000000)},
                      "cases": rows,
                      "roofline": {"bound": "tensor", "achieved": top["tflops"], "peak": peaks["bf16_tflops"], "unit": UNIT,
                                   "frac": top["frac_of_burst"], "traffic": None,
                                   "peak_source": "%s (burst bf16 matmul)" % peaks["_source"], "kernel": "attn128_ws_kernel<same head>, " + top["case"]},
                      "gpu_launches": launches, "clocks": clocks}))
    return 0


def bench_pages(args):
    """Cache page sizes: the cfg 2 chunk (8192 rows at prefix 32768) over caches of 256- to 16-token pages, and the cfg 3 chunk
    (absorbed MLA) over 64- to 16-token pages.  A KV tile of 128 keys takes one copy per operand with pages of 128 tokens or
    more and 2 x 128 / B copies with smaller ones."""
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    prefix, chunk = (int(args.prefixes.split(",")[0]) if args.prefixes else 32768), 8192
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    launches = 0
    cases = [("d=128 (Hq=64 Hkv=4)", bs, (W.BASE_SEED + 2, 64, 4, 128, 128, 1.0, None, False)) for bs in (256, 128, 64, 32, 16)]
    cases += [("absorbed MLA (Hq=128, 576/512)", bs, (W.BASE_SEED + 3, 128, 1, 576, 512, 0.5, 1.0 / math.sqrt(192.0), True))
              for bs in (64, 32, 16)]
    for desc, bs, (seed, hq, hkv, dqk, dv, std, scale, alias) in cases:
        prob = W.single_request_cache(seed, prefix, chunk, hq, hkv, dqk, dv, bs, std, scale, alias, dev, "pages", prefix)
        runner = api.ChunkAttn(prob, num_kv_splits=args.splits)
        per, step_ms, nl, _ = time_points([runner], stream, max(args.steps, 5), max(args.warmup, 3))
        launches += nl * max(args.steps, 5)
        tf = prob.flops() / (per[0] * 1e-3) / 1e12
        rows.append({"case": "%s, pages of %d tokens" % (desc, bs), "ms": round(per[0], 4), "tflops": round(tf, 1),
                     "frac_of_burst": round(tf / peaks["bf16_tflops"], 4)})
        del prob, runner
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = rows[1]
    print(json.dumps({"metric": "chunk attention TFLOP/s by cache page size (1 B200)", "value": top["tflops"], "unit": UNIT, "n_gpus": 1,
                      "steps": args.steps, "warmup": args.warmup, "ms_per_step": top["ms"], "higher_is_better": True, "dtype": "bf16",
                      "data": "synthetic", "vs_baseline": None,
                      "config": {"workload": "pages; chunk %d at prefix %d; %s" % (chunk, prefix, top["case"]),
                                 "l2": "K/V of the d=128 cases is 84 MB, Q and out 134 MB each: larger than the L2 together"},
                      "cases": rows,
                      "roofline": {"bound": "tensor", "achieved": top["tflops"], "peak": peaks["bf16_tflops"], "unit": UNIT,
                                   "frac": top["frac_of_burst"], "traffic": None,
                                   "peak_source": "%s (burst bf16 matmul)" % peaks["_source"], "kernel": "attn128_ws_kernel, " + top["case"]},
                      "gpu_launches": launches, "clocks": clocks}))
    return 0


def bench_merge(args):
    """vpp_lse_merge against the HBM roofline: S*(4*Dv+4) bytes read + (2*Dv+4) written per (row, head), CUDA-event timed,
    cycling through enough distinct buffers that no launch finds its inputs in the L2."""
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    cases = [("cfg4 partials: S=2, T=16384, Hq=64, Dv=128", 2, 16384, 64, 128),
             ("cfg4 partials: S=4, T=16384, Hq=64, Dv=128", 4, 16384, 64, 128),
             ("cfg4 partials: S=8, T=16384, Hq=64, Dv=128", 8, 16384, 64, 128),
             ("MLA partials: S=2, T=8192, Hq=128, Dv=512", 2, 8192, 128, 512),
             ("MLA partials: S=4, T=8192, Hq=128, Dv=512", 4, 8192, 128, 512)]
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    total_launches = 0
    for desc, S, T, Hq, Dv in cases:
        bytes_call = S * T * Hq * (4 * Dv + 4) + T * Hq * (2 * Dv + 4)
        sets = max(2, int(math.ceil(400e6 / bytes_call)))
        o_parts = [torch.randn(S, T, Hq, Dv, device=dev) for _ in range(sets)]
        l_parts = [torch.randn(S, T, Hq, device=dev) for _ in range(sets)]
        out = [torch.empty(T, Hq, Dv, dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        lse = [torch.empty(T, Hq, device=dev) for _ in range(sets)]
        n = max(args.steps, 5) * sets
        with torch.cuda.stream(stream):
            for i in range(max(args.warmup, 3)):
                api.vpp_lse_merge(o_parts[i % sets], l_parts[i % sets], out[i % sets], lse[i % sets], stream.cuda_stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(n):
                api.vpp_lse_merge(o_parts[i % sets], l_parts[i % sets], out[i % sets], lse[i % sets], stream.cuda_stream)
            e1.record(stream)
        e1.synchronize()
        ms = e0.elapsed_time(e1) / n
        total_launches += n
        rows.append({"case": desc, "us": round(ms * 1e3, 2), "GB/s": round(bytes_call / ms / 1e6, 1),
                     "frac_of_hbm_peak": round(bytes_call / ms / 1e6 / peaks["hbm_gbs"], 4), "bytes": bytes_call,
                     "launches_timed": n})
        del o_parts, l_parts, out, lse
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = rows[1]
    print(json.dumps({"metric": "lse-merge GB/s (read + written) vs HBM peak (1 B200)", "value": top["GB/s"], "unit": "GB/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "dtype": "f32",
                      "data": "synthetic", "vs_baseline": None,
                      "config": {"workload": "merge; " + top["case"], "l2": "distinct buffers of 400 MB or more per case"},
                      "cases": rows,
                      "roofline": {"bound": "hbm", "achieved": top["GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": top["frac_of_hbm_peak"], "traffic": None,
                                   "peak_source": "%s (copy bandwidth)" % peaks["_source"], "kernel": "lse_merge_kernel, " + top["case"]},
                      "gpu_launches": total_launches, "clocks": clocks}))
    return 0


def bench_append(args):
    """The KV-cache append kernel (the step before attention) against the HBM roofline: bytes read + written per call
    divided by the CUDA-event time.  Small chunks cycle through enough distinct buffers to exceed the L2."""
    import torch
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    gen = torch.Generator(device="cpu").manual_seed(W.BASE_SEED + 77)
    cases = [("cfg2 chunk: T=8192 Hkv=4 d=128, 128-token pages", 8192, 4, 128, 128, 128, False),
             ("cfg4 chunk: T=16384 Hkv=8 d=128, 128-token pages", 16384, 8, 128, 128, 128, False),
             ("cfg3 chunk: T=8192 latent 576 (values alias keys), 64-token pages", 8192, 1, 576, 512, 64, True),
             ("large: T=262144 Hkv=8 d=128, 128-token pages", 262144, 8, 128, 128, 128, False)]
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    for desc, T, hkv, dqk, dv, bs, alias in cases:
        bytes_call = T * hkv * (dqk + (0 if alias else dv)) * 2 * 2           # read + written
        sets = max(1, int(math.ceil(400e6 / bytes_call)))                       # distinct buffers > 126 MB L2
        nblk = T // bs
        k_new = [torch.randn(T, hkv, dqk, generator=gen).to(torch.bfloat16).to(dev) for _ in range(min(sets, 4))]
        v_new = None if alias else [x[..., :dv].contiguous() for x in k_new]
        k_cache = [torch.zeros(nblk, bs, hkv, dqk, dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        v_cache = [kc[..., :dv] for kc in k_cache] if alias else [torch.zeros_like(kc) for kc in k_cache]
        bt = torch.randperm(nblk, generator=gen).to(torch.int32).view(1, nblk).to(dev)
        pre = torch.zeros(1, dtype=torch.int32, device=dev)
        cl = torch.full((1,), T, dtype=torch.int32, device=dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        def call(i):
            api.vpp_kv_append(k_new[i % len(k_new)], None if alias else v_new[i % len(k_new)], k_cache[i % sets],
                              v_cache[i % sets], bt, pre, cl, bs, T, status=status, stream=stream.cuda_stream)
        n = max(args.steps, 5) * max(1, sets // 4)
        with torch.cuda.stream(stream):
            for i in range(max(args.warmup, 3)):
                call(i)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(n):
                call(i)
            e1.record(stream)
        e1.synchronize()
        assert int(status.item()) == 0
        ms = e0.elapsed_time(e1) / n
        rows.append({"case": desc, "us": round(ms * 1e3, 2), "GB/s": round(bytes_call / ms / 1e6, 1),
                     "frac_of_hbm_peak": round(bytes_call / ms / 1e6 / peaks["hbm_gbs"], 4), "bytes": bytes_call,
                     "launches_timed": n})
        del k_new, v_new, k_cache, v_cache
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = rows[-1]
    print(json.dumps({"metric": "kv-append GB/s (read + written) vs HBM peak (1 B200)", "value": top["GB/s"], "unit": "GB/s",
                      "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "dtype": "bf16 (bytes moved)",
                      "data": "synthetic", "config": {"workload": "kv-append; " + top["case"], "l2": "distinct buffers of 400 MB or more per case"},
                      "cases": rows, "vs_baseline": None,
                      "roofline": {"bound": "hbm", "achieved": top["GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": top["frac_of_hbm_peak"], "traffic": None,
                                   "peak_source": "%s (copy bandwidth)" % peaks["_source"], "kernel": "kv_append_kernel, " + top["case"]},
                      "gpu_launches": sum(r["launches_timed"] for r in rows), "clocks": clocks}))
    return 0


def bench_decode(args):
    """Decode rows (one query token per request) through the same attention entry point: HBM-bound, judged by the
    bytes of K/V that have to be read once (context x Hkv x (Dqk + Dv) x 2 B) per second."""
    import torch
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    cases = [("64 decode rows, context 32768, Hq=64 Hkv=8 d=128", [32768] * 64, [1] * 64, 64, 8, 128),
             ("64 decode rows, context 32768, Hq=64 Hkv=4 d=128", [32768] * 64, [1] * 64, 64, 4, 128),
             ("256 decode rows, context 8192, Hq=64 Hkv=8 d=128", [8192] * 256, [1] * 256, 64, 8, 128),
             ("16 decode rows (context 32768) + one 8192-token chunk at prefix 32768, Hq=64 Hkv=4", [32768] * 17,
              [1] * 16 + [8192], 64, 4, 128),
             ("64 decode rows, context 32768, absorbed MLA Hq=128 (576/512), 64-token pages", [32768] * 64, [1] * 64, 128, 1, 576),
             ("256 decode rows, context 8192, absorbed MLA Hq=128 (576/512), 64-token pages", [8192] * 256, [1] * 256, 128, 1, 576),
             ("32 decode rows, context 8192, Hq=64 Hkv=8 d=128 (1 GB of K/V: the profiler-sized case)", [8192] * 32, [1] * 32, 64, 8, 128)]
    if args.case >= 0:
        cases = [cases[args.case]]
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    launches = 0
    for desc, prefix, chunk, hq, hkv, dqk in cases:
        if dqk == 128:
            prob = W.make_problem(W.BASE_SEED + 91, prefix, chunk, hq, hkv, 128, 128, block_size=128, std=1.0, device=dev)
            kv_bytes = sum(p + c for p, c in zip(prefix, chunk)) * hkv * 256 * 2
        else:
            prob = W.make_problem(W.BASE_SEED + 92, prefix, chunk, hq, 1, 576, 512, block_size=64, std=0.5,
                                  scale=1.0 / 192 ** 0.5, v_aliases_k=True, device=dev)
            kv_bytes = sum(p + c for p, c in zip(prefix, chunk)) * 576 * 2
        runner = api.ChunkAttn(prob, num_kv_splits=args.splits)
        n = max(args.steps, 5)
        with torch.cuda.stream(stream):
            for _ in range(max(args.warmup, 3)):
                runner.run(stream.cuda_stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n):
                runner.run(stream.cuda_stream)
            e1.record(stream)
        e1.synchronize()
        assert int(runner.status.item()) == 0
        ms = e0.elapsed_time(e1) / n
        launches += n * api.vpp_last_launch_count()
        rows.append({"case": desc, "ms": round(ms, 4), "kv_GB/s": round(kv_bytes / ms / 1e6, 1),
                     "frac_of_hbm_peak": round(kv_bytes / ms / 1e6 / peaks["hbm_gbs"], 4),
                     "tflops": round(prob.flops() / ms / 1e9, 1), "kv_bytes": kv_bytes})
        del prob, runner
        torch.cuda.empty_cache()
    clocks = sampler.stop()
    top = rows[0]
    print(json.dumps({"metric": "decode rows through chunk attention: K/V GB/s vs HBM peak (1 B200)", "value": top["kv_GB/s"],
                      "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic", "vs_baseline": None,
                      "config": {"workload": "decode; " + top["case"], "l2": "K/V of every case exceeds the L2 (1 GB or more)"},
                      "cases": rows,
                      "roofline": {"bound": "hbm", "achieved": top["kv_GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": top["frac_of_hbm_peak"], "traffic": None,
                                   "peak_source": "%s (copy bandwidth)" % peaks["_source"],
                                   "kernel": "attn128_ws_kernel, packed single-token items; " + top["case"]},
                      "gpu_launches": launches, "clocks": clocks}))
    return 0


def bench_sparse(args):
    """Index-selected (sparse) attention over the cfg3 latent cache: 8192-token chunk, Hq = 128, 2048 listed keys per
    token, at several prefix lengths and for two list structures.  The cost per chunk should not depend on the prefix
    (the paper's remark that sparse attention flattens the latency curve); the flop count is that of the listed keys."""
    import torch
    from paper_2608_26523_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    chunk, topk, hq = 8192, args.topk, 128
    prefixes = [int(x) for x in args.prefixes.split(",")] if args.prefixes else [8192, 65536, 262144, 516096]
    base = W.cfg3(prefix=prefixes[0], max_prefix=max(max(prefixes), args.max_prefix), device=dev)
    stream = torch.cuda.Stream()
    rows = []
    sampler = ClockSampler(0)
    sampler.start()
    launches = 0
    for kind in ("clustered", "scattered"):
        for i, pre in enumerate(prefixes):
            q = W.random_q(W.BASE_SEED + 300 + i, chunk, hq, 576, std=0.5, device=dev)
            prob = base.with_chunk([pre], [chunk], q)
            idx_cpu = W.make_sparse_indices_strata(W.BASE_SEED + 400 + i, [pre], [chunk], topk, kind=kind)
            listed = int((idx_cpu >= 0).sum())
            idx = idx_cpu.to(dev)
            runner = api.SparseAttn(prob, idx)
            n = max(args.steps, 3)
            with torch.cuda.stream(stream):
                for _ in range(max(args.warmup, 3)):
                    runner.run(stream.cuda_stream)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(n):
                    runner.run(stream.cuda_stream)
                e1.record(stream)
            e1.synchronize()
            assert int(runner.status.item()) == 0
            ms = e0.elapsed_time(e1) / n
            launches += 2 * n
            flops = 2.0 * hq * (576 + 512) * listed
            row_bytes = listed * 576 * 2                       # every listed row once (the value pass re-reads it on chip)
            io_bytes = chunk * hq * (576 + 512) * 2 + idx.numel() * 4
            rows.append({"lists": kind, "prefix": pre, "ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1),
                         "frac_of_bf16_peak": round(flops / ms / 1e9 / peaks["bf16_tflops"], 4),
                         "listed_rows_GB/s": round(row_bytes / ms / 1e6, 1),
                         "frac_of_hbm_peak_if_no_reuse": round((row_bytes + io_bytes) / ms / 1e6 / peaks["hbm_gbs"], 4)})
            del runner, idx, prob, q
    clocks = sampler.stop()
    cpu = None
    if not args.no_cpu_baseline:
        # the oracle as it stands on a bounded sample of the first case's tokens
        import numpy as np
        from oracle.ref_sparse_attn import ref_sparse_chunk_attn
        pre = prefixes[0]
        q = W.random_q(W.BASE_SEED + 300, chunk, hq, 576, std=0.5, device="cpu")
        idx_cpu = W.make_sparse_indices_strata(W.BASE_SEED + 400, [pre], [chunk], topk, kind="clustered").numpy()
        toks = list(range(0, chunk, 3))          # about 15 s of CPU work
        bits = lambda t: t.view(torch.int16).numpy().view(np.uint16)
        k_cpu = base.k_cache.cpu()
        bt = base.block_table.cpu().numpy()
        t0 = time.perf_counter()
        ref_sparse_chunk_attn(bits(q), bits(k_cpu), idx_cpu, bt, base.block_size, np.array([pre], np.int32),
                              np.array([chunk], np.int32), 512, base.scale, toks)
        dt = time.perf_counter() - t0
        fl = 2.0 * hq * (576 + 512) * float((idx_cpu[toks] >= 0).sum())
        cpu = {"value": round(fl / dt / 1e12, 6), "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
               "sample": "%d tokens of the chunk at prefix %d, all heads (%.1f s of wall time; numpy, threads as the BLAS takes them)"
                         % (len(toks), pre, dt)}
    top = rows[len(prefixes) - 1]          # clustered lists at the longest prefix
    ms_all = [r["ms"] for r in rows if r["lists"] == "clustered"]
    print(json.dumps({"metric": "sparse (index-selected) MLA chunk attention TFLOP/s over listed keys (1 B200)",
                      "value": top["tflops"], "unit": "TFLOP/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step": top["ms"], "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                      "vs_baseline": None,
                      "config": {"workload": "sparse: cfg3 cache (Hq=128, latent 576/512, 64-token pages), chunk %d, %d listed "
                                             "keys per token, lists = recent window of %d + stratified earlier positions "
                                             "(clustered: shared by 64 consecutive tokens; scattered: independent)"
                                             % (chunk, topk, topk // 4),
                                 "l2": "the cache at the longer prefixes (75 MB - 604 MB) exceeds or fills the L2; Q and out "
                                       "stream (2.3 GB per chunk)"},
                      "cases": rows,
                      "latency_flatness": {"ms_min": min(ms_all), "ms_max": max(ms_all),
                                           "note": "clustered lists: ms per chunk across the prefixes; dense cfg3 grows "
                                                   "2.1 us per prefix token"},
                      "roofline": {"bound": "tensor", "achieved": top["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                   "frac": top["frac_of_bf16_peak"], "traffic": None,
                                   "peak_source": "%s (dense bf16 matmul, burst)" % peaks["_source"],
                                   "kernel": "dsa_attn_kernel, clustered lists, prefix %d" % top["prefix"]},
                      "cpu_baseline": cpu, "gpu_launches": launches, "clocks": clocks}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5", "append", "decode", "sparse", "merge", "groups", "pages"],
                    help="cfg2 is the benchmark the metric is quoted on; the others are the parity configurations")
    ap.add_argument("--prefixes", default="")
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--max-prefix", type=int, default=0,
                    help="size the KV cache (and its page pool) for this prefix even if the run uses shorter ones")
    ap.add_argument("--topk", type=int, default=2048, help="listed keys per token (--workload sparse)")
    ap.add_argument("--case", type=int, default=-1, help="run only this case of --workload decode")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="cfg2 only: skip the other four configurations")
    ap.add_argument("--e2e-slices", default="auto",
                    help="the end-to-end leg streams the chunk in slices: auto (planned), a count of equal slices, or lengths a,b,c,...")
    args = ap.parse_args()
    if args.workload == "append":
        return bench_append(args)
    if args.workload == "decode":
        return bench_decode(args)
    if args.workload == "sparse":
        return bench_sparse(args)
    if args.workload == "merge":
        return bench_merge(args)
    if args.workload == "pages":
        return bench_pages(args)
    if args.workload == "groups":
        return bench_groups(args)
    WL = {"cfg1": dict(prefixes=[0, 512, 1024, 1536], chunk=512, hq=4, hkv=1,
                       desc="cfg1: Hq=4 Hkv=1 d=128, 2048 tokens as 4 chunks of 512, contiguous cache"),
          "cfg2": dict(prefixes=W.CFG2_PREFIXES, chunk=8192, hq=64, hkv=4,
                       desc="cfg2: GQA Hq=64 Hkv=4 d=128, chunk 8192, 128-token pages, shuffled block_table"),
          "cfg3": dict(prefixes=W.CFG3_PREFIXES, chunk=8192, hq=128, hkv=1,
                       desc="cfg3: absorbed MLA Hq=128, one latent kv-head, Dqk=576 Dv=512, chunk 8192, 64-token pages"),
          "cfg4": dict(prefixes=W.CFG4_PREFIXES, chunk=16384, hq=64, hkv=8,
                       desc="cfg4: GQA Hq=64 Hkv=8 d=128, chunk 16384, 128-token pages, split-KV + merge"),
          "cfg5": dict(prefixes=[-1], chunk=16384, hq=64, hkv=8,
                       desc="cfg5: 32 requests, 16384 packed query tokens, lengths log-uniform 1K-256K, Hq=64 Hkv=8 d=128")}[args.workload]
    prefixes = [int(x) for x in args.prefixes.split(",")] if args.prefixes else list(WL["prefixes"])
    chunk = WL["chunk"]
    if args.workload == "cfg4" and args.splits == 0:
        args.splits = 4
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    peaks = load_peaks()
    config = {"workload": "%s, prefixes %s" % (WL["desc"], prefixes), "prefixes": prefixes, "chunk": chunk,
              "num_kv_splits": args.splits,
              "l2": "inputs larger than L2: each step cycles through %d MB of KV plus %d MB of Q per prefix point"
              % (int((max(prefixes) + chunk) * (1152 if args.workload == "cfg3" else WL["hkv"] * 512) / 1e6),
                 int(chunk * WL["hq"] * (1152 if args.workload == "cfg3" else 256) / 1e6))
              if args.workload in ("cfg2", "cfg3", "cfg4") else
              ("whole problem is L2-resident: latency-bound case, no roofline claimed" if args.workload == "cfg1"
               else "inputs larger than L2 (about 3 GB of KV)")}

    # ------------------------------------------------------------------------------------------
    if args.impl == "reference":
        if rank != 0:
            return
        rng = np.random.default_rng(0)
        budget = 20.0
        steps_total = args.steps + args.warmup
        per_step = min(budget, 120.0 / max(steps_total, 1))
        # a smaller cache is enough for the sample: rows of the 64K point
        prob = W.cfg2(prefix=65536, device="cpu")
        times, flops, rows_n = [], [], 0
        for s in range(steps_total):
            fl, dt, n, threads = oracle_sample_rate(prob, per_step, rng)
            if s >= args.warmup:
                times.append(dt); flops.append(fl); rows_n += n
        val = sum(flops) / sum(times) / 1e12
        line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": config,
                "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                                 "sample": "%d random (row, head) pairs of the chunk at prefix 65536 over %d steps"
                                 % (rows_n, args.steps)},
                "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line), flush=True)
        return

    # ------------------------------------------------------------------------------------------
    from paper_2608_26523_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        D.init("nccl", dev)
    api.load_library()

    max_prefix = max(max(prefixes), args.max_prefix)
    stream = torch.cuda.Stream(device=dev)
    runners = []
    if args.workload == "cfg5":
        runners.append(api.ChunkAttn(W.cfg5(device=dev), num_kv_splits=args.splits))
    elif args.workload == "cfg1":
        for P in prefixes:
            runners.append(api.ChunkAttn(W.cfg1(P // 512, device=dev), num_kv_splits=args.splits))
    else:
        base = {"cfg2": W.cfg2, "cfg3": W.cfg3, "cfg4": W.cfg4}[args.workload](prefix=max_prefix, max_prefix=max_prefix,
                                                                              device=dev)
        for P in prefixes:
            prob = base.with_chunk([P], [chunk], base.q)
            runners.append(api.ChunkAttn(prob, num_kv_splits=args.splits))
    flops_pt = [r.prob.flops() for r in runners]
    flops_step = float(sum(flops_pt))
    launches_per_step = 0

    def one_step(events=None):
        for i, r in enumerate(runners):
            if events is not None:
                events[i][0].record(stream)
            r.run(stream.cuda_stream)
            if events is not None:
                events[i][1].record(stream)

    def barrier():
        D.barrier(dev)

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            one_step()
        launches_per_step = 0
        for r in runners:
            r.run(stream.cuda_stream)
            launches_per_step += api.vpp_last_launch_count()
        barrier()
        for r in runners:
            assert int(r.status.item()) == 0, "device status %d" % int(r.status.item())

        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
            time.sleep(0.3)
        ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in runners]
              for _ in range(args.steps)]
        t_beg = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
        barrier()
        t_beg.record(stream)
        for s in range(args.steps):
            one_step(ev[s])
        t_end.record(stream)
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        total_ms = t_beg.elapsed_time(t_end)
        per_pt_ms = [statistics.median(ev[s][i][0].elapsed_time(ev[s][i][1]) for s in range(args.steps))
                     for i in range(len(runners))]
        per_pt_min = [min(ev[s][i][0].elapsed_time(ev[s][i][1]) for s in range(args.steps)) for i in range(len(runners))]

        # ---- end to end: host buffers in, host buffers out, copies inside the timed region ----
        e2e = None
        if not args.no_e2e and args.workload == "cfg2":
            i_main = prefixes.index(65536) if 65536 in prefixes else len(prefixes) - 1
            r = runners[i_main]
            P = prefixes[i_main]
            # The public call for host-resident inputs, vpp_chunk_attn_host_fwd: q and the chunk's own K/V rows come from
            # pinned host memory, out and lse go back to it; the library streams the chunk in slices, the copies of one
            # slice overlapping the append + attention of its neighbours.  Every step copies all inputs in and all
            # results out, and no step starts before the previous one's last copy has finished.
            slices = None if args.e2e_slices == "auto" else [int(x) for x in args.e2e_slices.split(",")]
            pipe = api.HostChunkPipeline(r.prob, slices=slices, num_kv_splits=args.splits)
            e2e_plan = pipe.slices
            q_host = r.prob.q.cpu().pin_memory()
            k_host = pipe.chunk_rows(r.prob.k_cache).cpu().contiguous().pin_memory()
            v_host = pipe.chunk_rows(r.prob.v_cache).cpu().contiguous().pin_memory()
            out_host = torch.empty(r.out.shape, dtype=r.out.dtype).pin_memory()
            lse_host = torch.empty(r.lse.shape, dtype=r.lse.dtype).pin_memory()
            h2d = (q_host.numel() + k_host.numel() + v_host.numel()) * 2
            d2h = out_host.numel() * 2 + lse_host.numel() * 4

            def e2e_step():
                pipe.run(q_host, k_host, v_host, out_host, lse_host, stream)

            for _ in range(2):
                e2e_step()
            barrier()
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            n_e2e = max(args.steps, 3)
            for _ in range(n_e2e):
                e2e_step()
            t1.record(stream)
            barrier()
            e2e_ms = t0.elapsed_time(t1) / n_e2e
            e2e = (flops_pt[i_main], e2e_ms, h2d, d2h, P)
            # the streamed result is the resident launch's result
            assert int(pipe.status.item()) == 0
            r.run(stream.cuda_stream)
            stream.synchronize()
            diff = (out_host[::7].float() - r.out[::7].float().cpu()).abs().max().item()
            assert diff <= 1e-2, "streamed chunk differs from the resident launch by %g" % diff

    # ---- (cfg2, one GPU) the 96K point that makes 0 / 32K / 64K / 96K / 128K evenly spaced, outside the timed step ----
    extra_pt = None
    if args.workload == "cfg2" and world == 1 and not args.prefixes and max_prefix >= 98304:
        r96 = api.ChunkAttn(base.with_chunk([98304], [chunk], base.q), num_kv_splits=args.splits)
        per96, _, _, _ = time_points([r96], stream, max(args.steps, 3), 2)
        extra_pt = (98304, per96[0])
        del r96

    # ---- max over ranks ----
    if world > 1:
        t = D.max_over_ranks([total_ms, e2e[1] if e2e else 0.0], dev)
        total_ms = t[0]
        if e2e:
            e2e = (e2e[0], t[1], e2e[2], e2e[3], e2e[4])
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12
    burst, sustained = float(peaks["bf16_tflops"]), float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    curve = []
    for P, ms, ms_min, fl in zip(prefixes, per_pt_ms, per_pt_min, flops_pt):
        tf = fl / (ms * 1e-3) / 1e12
        curve.append({"prefix": P, "ms": round(ms, 4), "ms_min": round(ms_min, 4), "tflops": round(tf, 2),
                      "frac_of_burst_peak": round(tf / burst, 4), "frac_of_sustained_peak": round(tf / sustained, 4),
                      "frac_of_nominal_peak": round(tf / NOMINAL_BF16_TFLOPS, 4)})
    cost_curve = None
    if len(prefixes) >= 3 and args.workload in ("cfg2", "cfg3", "cfg4"):
        cost_curve = fit_cost_curve(prefixes, per_pt_ms)
        if extra_pt is not None:
            # the paper's balance identity on evenly spaced points: the 96K point (timed outside the step) completes
            # 0 / 32K / 64K / 96K / 128K
            xs = sorted(set(prefixes) | {extra_pt[0]})
            ys = [extra_pt[1] if x == extra_pt[0] else per_pt_ms[prefixes.index(x)] for x in xs]
            even = fit_cost_curve(xs, ys)
            cost_curve["eq3_residual_max"] = even.get("eq3_residual_max")
            cost_curve["eq3_triples"] = even.get("eq3_triples")
            cost_curve["eq3_points"] = "evenly spaced triples among %s (prefix %d timed outside the step: %.4f ms)" % (xs, extra_pt[0], extra_pt[1])
    # dominant kernel = the attention kernel at the longest prefix; its launch is timed together with the
    # ~10 us work-decomposition kernel that precedes it on the same stream
    i_top = int(np.argmax(flops_pt))
    ach = flops_pt[i_top] / (per_pt_ms[i_top] * 1e-3) / 1e12
    # DRAM bytes of that launch: from the record written beside the ncu summary of the same command (never a literal here)
    traffic, traffic_source = None, None
    if args.workload == "cfg2":
        rec = read_traffic_record("attn128_ws_cfg2_traffic.txt")
        if rec.get("prefix") == str(prefixes[i_top]) and args.splits == int(rec.get("num_kv_splits", "0")):
            traffic = float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"])
            traffic_source = "profiles/attn128_ws_cfg2_traffic.txt (ncu capture at commit %s)" % rec.get("commit", "?")
    roofline = {"bound": "tensor", "achieved": round(ach, 2), "peak": burst, "unit": "TFLOP/s",
                "frac": round(ach / burst, 4), "traffic": traffic, "traffic_source": traffic_source,
                "algorithmic_bytes": int((prefixes[i_top] + chunk) * WL["hkv"] * 512 + chunk * WL["hq"] * (256 + 256 + 4))
                if args.workload in ("cfg2", "cfg4") else None, "peak_source": "%s (burst bf16 matmul)" % peaks["_source"],
                "frac_of_sustained": round(ach / sustained, 4), "kernel": "attention kernel, prefix %d" % prefixes[i_top]}
    line = {"metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config, "curve": curve, "cost_curve": cost_curve,
            "roofline": roofline, "gpu_launches": launches_per_step * args.steps, "clocks": clocks}
    if e2e:
        line["e2e"] = {"value": round(world * e2e[0] / (e2e[1] * 1e-3) / 1e12, 3), "unit": UNIT,
                       "h2d_bytes_per_step": int(e2e[2]), "d2h_bytes_per_step": int(e2e[3]),
                       "ms_per_step": round(e2e[1], 4),
                       "workload": "vpp_chunk_attn_host_fwd on the chunk at prefix %d: q and the chunk's K/V rows host->device, "
                                   "appended to the cache, out and lse device->host, streamed in slices of %s query rows whose "
                                   "copies overlap the neighbouring slices' append + attention" % (e2e[4], e2e_plan)}
    if not args.no_cpu_baseline and world == 1 and args.workload == "cfg2":
        prob_cpu = runners[prefixes.index(65536) if 65536 in prefixes else -1].prob.to("cpu")
        fl, dt, n, threads = oracle_sample_rate(prob_cpu, 15.0, np.random.default_rng(0))
        line["cpu_baseline"] = {"value": round(fl / dt / 1e12, 6), "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": "%d random (row, head) pairs of the chunk at prefix %d (%.1f s of CPU time)"
                                % (n, int(prob_cpu.prefix_len[0]), dt),
                                "extrapolated_full_s": round(prob_cpu.flops() / (fl / dt), 1)}   # that whole chunk at the sampled rate (not run)
    if args.workload == "cfg2" and world == 1 and not args.no_sweep and not args.prefixes:
        del runners
        if e2e:
            del pipe, q_host, out_host, lse_host, k_host, v_host
        base = None
        torch.cuda.empty_cache()
        line["configs"] = sweep_other_configs(dev, peaks, max(3, min(args.steps, 5)), max(3, args.warmup), not args.no_cpu_baseline)
    if world > 1:
        dist.destroy_process_group()
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
