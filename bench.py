#!/usr/bin/env python
"""Benchmark of the SubNet query stream (ResNet-50-shaped SuperNet, batch 1, 224x224, bf16).

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --steps K --warmup W    # the CPU checker on the host cores

A step is one pass of the whole hot path over the query stream: `--queries` SubNet queries, each a
different uniformly sampled SubNet config, through sgs_stream_run with inputs resident in HBM.
Prints one JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
# many streams in flight need more than the default 8 hardware work queues; must be set before CUDA starts
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

from paper_2306_17266_b200 import workload as wl  # noqa: E402

RES, BATCH = 224, 1
METRIC, UNIT = "subnet_queries_per_s", "queries/s"
WORKLOAD = "ResNet-50-shaped SuperNet, 1000-query stream at batch 1, 224x224x3, SubNets sampled uniformly (seed 2)"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 6:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def cpu_oracle_qps(n_queries: int):
    """Times the CPU checker, as it stands, on the first queries of the same workload."""
    import oracle
    blob = wl.make_blob(wl.RESNET, seed=0, bf16_weights=True)
    net = oracle.Net(wl.RESNET, blob)
    cfgs = wl.uniform_stream(wl.RESNET, 1000, seed=2)[:n_queries]
    xs = wl.make_inputs(n_queries, BATCH, RES, seed=1, bf16=True)
    t0 = time.perf_counter()
    for c, x in zip(cfgs, xs):
        net.forward(c, x, oracle.BF16_STORE)
    dt = time.perf_counter() - t0
    return n_queries / dt, dt, oracle.num_threads()


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    per_step = max(1, args.ref_queries)
    import oracle
    blob = wl.make_blob(wl.RESNET, seed=0, bf16_weights=True)
    net = oracle.Net(wl.RESNET, blob)
    cfgs = wl.uniform_stream(wl.RESNET, 1000, seed=2)
    xs = wl.make_inputs(per_step, BATCH, RES, seed=1, bf16=True)
    k = 0
    for _ in range(args.warmup):
        net.forward(cfgs[k % 1000], xs[0], oracle.BF16_STORE)
        k += 1
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for i in range(per_step):
            net.forward(cfgs[k % 1000], xs[i], oracle.BF16_STORE)
            k += 1
    dt = time.perf_counter() - t0
    qps = args.steps * per_step / dt
    sample = f"{per_step} queries per step of the same stream (a whole step is 1000 queries)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": qps, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------------------------
# Other configurations (not part of the default line): each prints one JSON line of its own.
# ----------------------------------------------------------------------------------------------
def _stream_pool(net, sgs, torch, cfgs, batch, res, opts, stream, pool_groups, family):
    """Runs `cfgs` as consecutive sgs_stream_run calls over a pool of `pool_groups` resident inputs."""
    n_cls = 1000
    x = torch.from_numpy(wl.make_inputs(pool_groups, batch, res, seed=1, bf16=True).reshape(pool_groups * batch, res, res, 3))
    x = x.cuda().to(torch.bfloat16).contiguous()
    logits = torch.zeros((pool_groups * batch, n_cls), dtype=torch.float32, device="cuda")
    tot = {"ms": 0.0, "q": 0, "flops": 0.0, "wbytes": 0.0, "miss": 0.0, "hit": 0.0, "launches": 0, "p50": []}
    for i in range(0, len(cfgs), pool_groups):
        part = cfgs[i:i + pool_groups]
        st = net.stream_run(wl.cfg_array(part), x.data_ptr(), batch, res, logits.data_ptr(), opts, stream.cuda_stream)
        tot["ms"] += st.total_ms; tot["q"] += len(part); tot["flops"] += st.useful_flops; tot["wbytes"] += st.weight_bytes
        tot["miss"] += st.hbm_weight_bytes; tot["hit"] += st.hit_ratio * len(part); tot["launches"] += st.kernel_launches
        tot["p50"].append(st.p50_ms)
    return tot


SWEEP_WORKLOAD = ("ResNet-50-shaped SuperNet throughput sweep: batches of 64 = 4 SubNet configs x 16 images in one grouped launch per layer, "
                  "configs uniform (seed 5)")


def measure_sweep(net, sgs, torch, stream, peaks, n_groups=1250, resolutions=(160, 192, 224), cache=1, window=4, concurrency=4):
    """Throughput sweep (waves of 4 members x 16 images): images/s, useful TFLOP/s and fractions of the bf16 peaks."""
    cfgs = wl.uniform_stream(wl.RESNET, n_groups, seed=5)
    rows = []
    for res in resolutions:
        opts = sgs.StreamOpts(cache_enabled=cache, window_q=window, cache_budget_bytes=0, use_graphs=1, record_latency=0,
                              concurrency=concurrency, wave=4)
        _stream_pool(net, sgs, torch, cfgs[:64], 16, res, opts, stream, 64, wl.RESNET)  # warm-up: workspaces
        t = _stream_pool(net, sgs, torch, cfgs, 16, res, opts, stream, 64, wl.RESNET)
        tf = t["flops"] / (t["ms"] * 1e-3) / 1e12
        rows.append({"res": res, "images": t["q"] * 16, "images_per_s": t["q"] * 16 / (t["ms"] * 1e-3), "useful_tflops": tf,
                     "frac_of_bf16_sustained_peak": tf / peaks["bf16_tflops_sustained"], "frac_of_bf16_burst_peak": tf / peaks["bf16_tflops"],
                     "gflop_per_image": t["flops"] / (t["q"] * 16) / 1e9, "ms": t["ms"]})
    return rows


EXTRA_OPTIONS = []  # (name, value) pairs of --option: library tuning aids, applied to every SuperNet the run creates


def apply_options(net):
    for name, value in EXTRA_OPTIONS:
        net.set_option(name, value)
    return net


def measure_mbv3(sgs, torch, stream, queries=1000, wave=32, concurrency=4, cache=1, window=4, profile=False, persistent_only=False):
    """The MobileNetV3-shaped stream (1000 queries, batch 1, 224x224, configs uniform seed 3): layer by layer in waves,
    and as ONE launch of the persistent SubNet kernel (every SM serves whole queries)."""
    net = apply_options(sgs.SuperNet(wl.MBV3, wl.make_blob(wl.MBV3, seed=0, bf16_weights=True), sgs.SGS_BF16))
    cfgs = wl.uniform_stream(wl.MBV3, queries, seed=3)
    popt = sgs.StreamOpts(cache_enabled=cache, window_q=window, cache_budget_bytes=0, record_latency=0, persistent=1)
    for _ in range(2):
        _stream_pool(net, sgs, torch, cfgs, 1, 224, popt, stream, len(cfgs), wl.MBV3)
    tp = _stream_pool(net, sgs, torch, cfgs, 1, 224, popt, stream, len(cfgs), wl.MBV3)
    persistent = {"queries_per_s": tp["q"] / (tp["ms"] * 1e-3), "ms_per_launch": tp["ms"], "kernel_launches": tp["launches"],
                  "useful_tflops": tp["flops"] / (tp["ms"] * 1e-3) / 1e12, "weight_hit_ratio_on_chip": tp["hit"] / tp["q"],
                  "execution": "one launch of the persistent SubNet kernel; every SM takes the next query and runs all of its layers"}
    if persistent_only:
        net.close()
        return {"persistent": persistent}
    opts = sgs.StreamOpts(cache_enabled=cache, window_q=window, cache_budget_bytes=0, use_graphs=1, record_latency=1,
                          concurrency=concurrency, wave=wave)
    for _ in range(2):
        _stream_pool(net, sgs, torch, cfgs, 1, 224, opts, stream, len(cfgs), wl.MBV3)
    t = _stream_pool(net, sgs, torch, cfgs, 1, 224, opts, stream, len(cfgs), wl.MBV3)
    out = {"queries_per_s": t["q"] / (t["ms"] * 1e-3), "p50_ms": float(np.median(t["p50"])), "gflop_per_query": t["flops"] / t["q"] / 1e9,
           "kernel_launches_per_query": t["launches"] / t["q"],
           "execution": f"waves of {wave}, {concurrency} in flight" if wave > 0 else f"one stream per query, {concurrency} in flight",
           "persistent": persistent}
    if profile:
        net.set_option("profile", 2)
        popts = sgs.StreamOpts(cache_enabled=cache, window_q=window, cache_budget_bytes=0, use_graphs=0, record_latency=0, wave=wave)
        _stream_pool(net, sgs, torch, cfgs, 1, 224, popts, stream, len(cfgs), wl.MBV3)
        prof = [net.profile_read(c) for c in range(4)]
        net.set_option("profile", 0)
        out["kernel_time_ms_by_class"] = {"conv_tc": prof[0]["total_ms"], "conv_cuda_core": prof[1]["total_ms"],
                                          "depthwise": prof[2]["total_ms"], "other": prof[3]["total_ms"]}
        out["depthwise_gbs_at_batch1"] = prof[2]["alg_bytes"] / (prof[2]["total_ms"] * 1e-3) / 1e9 if prof[2]["total_ms"] else None
    net.close()
    return out


def measure_depthwise(sgs, peaks, fma_tflops):
    """Depthwise kernels on working sets larger than L2 (64 x 56 x 56 x 480 bf16 in, same or a quarter out): GB/s of
    algorithmic bytes (input + output), fraction of the HBM peak, and for the 5x5 / 7x7 windows the fraction of the
    measured fp32 FMA rate (2 * k * k FLOP per output element)."""
    from paper_2306_17266_b200 import microbench
    rows = []
    for shape in microbench.DW_PRESETS["large"][:6]:
        r = microbench.bench_dw(shape)
        N, H, W, K, k, stride = shape
        outs = N * (H // stride) * (W // stride) * K
        tf = 2.0 * k * k * outs / r["us"] / 1e6
        rows.append({"k": k, "stride": stride, "shape": f"{N}x{H}x{W}x{K}", "us": r["us"], "gbs": r["gbs"], "frac_of_hbm_peak": r["gbs"] / peaks["hbm_gbs"],
                     "fma_tflops": tf, "frac_of_fma_peak": tf / fma_tflops if fma_tflops else None})
    return rows


def measure_plan_miss(net, sgs, torch, stream, x_dev, logits, opts, n=1000):
    """What a never-seen config costs: the plan cache is emptied, a stream of `n` fresh configs (uniform, seed 99) runs
    once cold and once warm; the difference per planned query is host planning + tensor-map encoding."""
    cfgs = wl.cfg_array(wl.uniform_stream(wl.RESNET, n, seed=99))
    net.set_option("drop_plans", 1)
    cold = net.stream_run(cfgs, x_dev.data_ptr(), BATCH, RES, logits.data_ptr(), opts, stream.cuda_stream)
    warm = net.stream_run(cfgs, x_dev.data_ptr(), BATCH, RES, logits.data_ptr(), opts, stream.cuda_stream)
    misses = max(1, cold.plan_misses)
    return {"fresh_configs": n, "plan_misses_cold": cold.plan_misses, "plan_misses_warm": warm.plan_misses,
            "cold_queries_per_s": cold.queries_per_s, "warm_queries_per_s": warm.queries_per_s,
            "us_per_never_seen_config": (cold.total_ms - warm.total_ms) * 1e3 / misses,
            "note": "device-timed stream with the plan cache emptied first (cold) against the same stream again (warm)"}


def run_suite(args):
    import torch
    import paper_2306_17266_b200 as sgs
    peaks = measured_peaks()
    stream = torch.cuda.Stream()
    out = {"suite": args.suite, "data": "synthetic", "dtype": "bf16", "n_gpus": 1}
    if args.suite == "sweep":
        # throughput sweep: 20k images as groups of 16 images sharing a config (4 groups = one batch of 64)
        net = sgs.SuperNet(wl.RESNET, wl.make_blob(wl.RESNET, seed=0, bf16_weights=True), sgs.SGS_BF16)
        n_groups = args.queries // 16 if args.queries != 1000 else 1250
        rows = measure_sweep(net, sgs, torch, stream, peaks, n_groups, resolutions=(args.res,) if args.res else (160, 192, 224), cache=args.cache,
                             window=args.window, concurrency=args.concurrency)
        out.update({"metric": "subnet_images_per_s", "unit": "images/s", "value": rows[-1]["images_per_s"], "rows": rows,
                    "config": {"workload": SWEEP_WORKLOAD + ", 20k images per resolution", "peaks": peaks}})
    elif args.suite == "sgs":
        # locality stream: Markov chain of configs; cache on / off, window Q in {1, 4, 8}, batch 1 (waves of 32) and
        # batch 16 (waves of 4 configs x 16 images), the execution modes of the stream and sweep benchmarks
        net = sgs.SuperNet(wl.RESNET, wl.make_blob(wl.RESNET, seed=0, bf16_weights=True), sgs.SGS_BF16)
        n = args.queries if args.queries != 1000 else 5000
        cfgs = wl.markov_stream(n, seed=4)
        rows = []
        for batch, nq, wave in ((1, n, 32), (16, max(64, n // 8), 4)):
            pool = 512 if batch == 1 else 32
            warm = sgs.StreamOpts(cache_enabled=0, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=0, weights_evict_first=0,
                                  concurrency=args.concurrency, wave=wave)
            _stream_pool(net, sgs, torch, cfgs[:nq], batch, 224, warm, stream, pool, wl.RESNET)  # builds every plan
            for cache, q, ef, mech in ((0, 4, 0, 0), (0, 4, 1, 0), (1, 1, 0, 0), (1, 4, 0, 0), (1, 8, 0, 0), (1, 4, 0, 1), (1, 4, 0, 2)):
                net.set_option("cache_mechanism", mech)
                opts = sgs.StreamOpts(cache_enabled=cache, window_q=q, cache_budget_bytes=0, use_graphs=1, record_latency=1, weights_evict_first=ef,
                                      concurrency=args.concurrency, wave=wave)
                _stream_pool(net, sgs, torch, cfgs[:pool], batch, 224, opts, stream, pool, wl.RESNET)
                t = _stream_pool(net, sgs, torch, cfgs[:nq], batch, 224, opts, stream, pool, wl.RESNET)
                rows.append({"batch": batch, "wave": wave, "cache": cache, "window_q": q, "weights_evict_first": ef,
                             "mechanism": ["tile hints", "launch window", "both"][mech] if cache else None, "queries": t["q"],
                             "queries_per_s": t["q"] / (t["ms"] * 1e-3), "p50_ms": float(np.median(t["p50"])),
                             "weight_mb_per_query": t["wbytes"] / t["q"] / 1e6, "hbm_weight_mb_per_query": t["miss"] / t["q"] / 1e6,
                             "hit_ratio": t["hit"] / t["q"]})
            net.set_option("cache_mechanism", 0)
        out.update({"metric": "hbm_weight_bytes_per_query", "unit": "MB/query (analytic)", "value": rows[3]["hbm_weight_mb_per_query"], "rows": rows,
                    "config": {"workload": "SGS locality stream on the ResNet-50-shaped SuperNet: Markov chain of configs (p=0.9 one stage's depth or width changes), seed 4, 224x224",
                               "note": "the cached SubGraph restarts at every pool boundary (512 queries at batch 1, 32 at batch 16)"}})
    elif args.suite == "sgs-probe":
        # one short locality stream, one variant, one wave (or query) at a time: meant to be run under a profiler that
        # sums DRAM bytes over the convolution kernels of the measured part (its launch range is printed)
        net = sgs.SuperNet(wl.RESNET, wl.make_blob(wl.RESNET, seed=0, bf16_weights=True), sgs.SGS_BF16)
        n = args.queries if args.queries != 1000 else 48
        warm_n = 16
        cfgs = wl.markov_stream(warm_n + n, seed=4)
        net.set_option("cache_mechanism", args.mechanism)
        opts = sgs.StreamOpts(cache_enabled=args.cache, window_q=args.window, cache_budget_bytes=args.budget_mb << 20, use_graphs=0, record_latency=0,
                              weights_evict_first=args.evict_first, concurrency=1, wave=args.wave)
        before = net.get_counter("kernel_launches")
        _stream_pool(net, sgs, torch, cfgs[:warm_n], args.batch, 224, opts, stream, warm_n, wl.RESNET)
        skip = net.get_counter("kernel_launches") - before
        tcs = net.get_counter("tc_convs")
        t = _stream_pool(net, sgs, torch, cfgs[warm_n:], args.batch, 224, opts, stream, n, wl.RESNET)
        out.update({"metric": "hbm_weight_bytes_per_query", "unit": "MB/query (analytic)", "value": t["miss"] / t["q"] / 1e6,
                    "weight_mb_per_query": t["wbytes"] / t["q"] / 1e6, "hit_ratio": t["hit"] / t["q"], "queries": t["q"],
                    "launches_before_measured_part": skip, "launches_in_measured_part": t["launches"],
                    "config": {"batch": args.batch, "wave": args.wave, "cache": args.cache, "window_q": args.window, "weights_evict_first": args.evict_first,
                               "mechanism": args.mechanism, "budget_mb": args.budget_mb,
                               "note": "load-time kernels precede the warm-up launches; count them with the profiler's launch list"}})
    elif args.suite == "sched":
        # caching decision of Algorithm 1 (nearest candidate SubGraph to the running average) beside the
        # intersection of the window, over the window length Q, the size of the candidate set and the budget
        fam = wl.MBV3 if args.family == "mbv3" else wl.RESNET
        net = sgs.SuperNet(fam, wl.make_blob(fam, seed=0, bf16_weights=True), sgs.SGS_BF16)
        n = args.queries
        cfgs = wl.markov_stream(n, seed=4, family=fam)
        rows = []
        warm = sgs.StreamOpts(cache_enabled=0, window_q=4, record_latency=0, concurrency=args.concurrency, wave=args.wave)
        _stream_pool(net, sgs, torch, cfgs, 1, 224, warm, stream, n, fam)
        # budgets: the device maximum, and about a quarter of the SuperNet's weights
        for budget_mb in ((0, 24) if fam == wl.RESNET else (0, 4)):
            for n_cand in (0, 16, 64, 256):
                net.cache_set_candidates(wl.candidate_cfgs(fam, n_cand, seed=6) if n_cand else [])
                for q in (1, 2, 4, 8, 16):
                    opts = sgs.StreamOpts(cache_enabled=1, window_q=q, cache_budget_bytes=budget_mb << 20, record_latency=0,
                                          concurrency=args.concurrency, wave=args.wave,
                                          policy=sgs.SGS_POLICY_AVGNET if n_cand else sgs.SGS_POLICY_INTERSECTION)
                    t = _stream_pool(net, sgs, torch, cfgs, 1, 224, opts, stream, n, fam)
                    rows.append({"policy": "avgnet" if n_cand else "intersection", "candidates": n_cand, "window_q": q,
                                 "budget_mb": net.cache_stats().budget_bytes / 2**20, "hit_ratio": t["hit"] / t["q"],
                                 "weight_mb_per_query": t["wbytes"] / t["q"] / 1e6, "hbm_weight_mb_per_query": t["miss"] / t["q"] / 1e6,
                                 "queries_per_s": t["q"] / (t["ms"] * 1e-3)})
        net.cache_set_candidates([])
        best = max(rows, key=lambda r: r["hit_ratio"])
        out.update({"metric": "cache_hit_ratio", "unit": "mean ||SN ∩ G|| / ||SN|| (analytic)", "value": best["hit_ratio"], "best": best, "rows": rows,
                    "config": {"workload": f"SGS locality stream on the {'MobileNetV3' if fam == wl.MBV3 else 'ResNet-50'}-shaped SuperNet: {n} queries, Markov chain of configs (p=0.9 one elastic choice changes), seed 4, 224x224, batch 1",
                               "candidates": "smallest and largest SubNet plus uniform draws (seed 6), each clipped to the budget",
                               "execution": f"waves of {args.wave}, {args.concurrency} in flight" if args.wave > 0 else f"one stream per query, {args.concurrency} in flight"}})
    elif args.suite == "table":
        # the latency table of Section 3.2 measured on this device (rows SubNets, columns cached SubGraphs, last
        # column = nothing cached) and Algorithm 1 driven by it; accuracies are a FLOPs-monotone stand-in
        import time
        net = sgs.SuperNet(wl.RESNET, wl.make_blob(wl.RESNET, seed=0, bf16_weights=True), sgs.SGS_BF16)
        batch, res, n_sub, n_cand = args.batch, 224, 8, 8
        subnets = wl.candidate_cfgs(wl.RESNET, n_sub, seed=11)
        acc = wl.proxy_accuracy([net.subnet_cost(c, batch, res)[0] for c in subnets])
        x = torch.from_numpy(wl.make_inputs(1, batch, res, seed=1, bf16=True).reshape(batch, res, res, 3)).cuda().to(torch.bfloat16).contiguous()
        logits = torch.zeros((batch, 1000), dtype=torch.float32, device="cuda")
        rows = []
        for budget_mb in (0, 24):
            net.cache_set_candidates(wl.candidate_cfgs(wl.RESNET, n_cand, seed=6))
            net.cache_configure(True, budget_mb << 20, args.window)
            sched = sgs.Scheduler(net, subnets, acc, args.window)
            sched.measure(x.data_ptr(), batch, res, logits.data_ptr(), reps=9, flush_bytes=256 << 20, stream=stream.cuda_stream)
            table = sched.get_table()
            none = table[:, -1]
            gain = (none[:, None] - table[:, :-1]) / none[:, None]
            n = 100000
            policy, a_t, l_t = wl.sched_queries(n, seed=8, accuracy=acc, latency=table.reshape(-1))
            t0 = time.perf_counter()
            served, state = sched.step(policy, a_t, l_t)
            lookup_ns = (time.perf_counter() - t0) / n * 1e9
            lat = table[served, state]
            met = np.where(policy == 0, acc[served] >= a_t, lat <= l_t)
            rows.append({"budget_mb": net.cache_stats().budget_bytes / 2**20, "table_ms": np.round(table, 4).tolist(),
                         "best_column_gain_mean": float(gain.max(axis=1).mean()), "best_column_gain_max": float(gain.max()),
                         "column_spread_mean": float(((table[:, :-1].max(axis=1) - table[:, :-1].min(axis=1)) / none).mean()),
                         "step_ns": lookup_ns, "hard_constraint_met": float(met.mean()),
                         "served_histogram": np.bincount(served, minlength=n_sub).tolist(),
                         "cache_state_histogram": np.bincount(state, minlength=n_cand + 1).tolist()})
            sched.close()
        net.cache_set_candidates([])
        out.update({"metric": "latency_table_best_column_gain", "unit": "mean over SubNets of (L[i][none] - min_j L[i][j]) / L[i][none]",
                    "value": rows[0]["best_column_gain_mean"], "rows": rows, "accuracy_proxy": np.round(acc, 4).tolist(),
                    "config": {"workload": f"ResNet-50-shaped SuperNet, {n_sub} SubNets x ({n_cand} candidate SubGraphs + empty cache), batch {batch}, 224x224; one query at a time, 256 MB overwritten before every timed run, median of 9",
                               "scheduler": f"Algorithm 1 with Q = {args.window} on 100000 synthetic (policy, A_t, L_t) queries (seed 8); step_ns includes the caching decision every Q queries"}})
    elif args.suite == "mbv3":
        r = measure_mbv3(sgs, torch, stream, args.queries, args.wave, args.concurrency, args.cache, args.window, profile=not args.persistent,
                         persistent_only=args.persistent)
        head = r["persistent"] if args.persistent else r
        out.update({"metric": METRIC, "unit": UNIT, "value": head["queries_per_s"], **r,
                    "config": {"workload": f"MobileNetV3-shaped SuperNet, {args.queries}-query stream at batch 1, 224x224, configs uniform (seed 3)",
                               "execution": head["execution"]}})
    elif args.suite == "dw":
        fma = sgs.measure_fma_peak(stream.cuda_stream)
        rows = measure_depthwise(sgs, peaks, fma)
        out.update({"metric": "depthwise_gbs", "unit": "GB/s (input + output bytes)", "value": rows[0]["gbs"], "rows": rows, "fp32_fma_tflops_measured": fma,
                    "config": {"workload": "depthwise k x k (centre window of the stored 7x7), 64 x 56 x 56 x 480 bf16, h-swish, working set beyond L2", "peaks": peaks}})
    print(json.dumps(out))


def ncu_record(name):
    """Counters taken under the profiler cannot be measured inside a timed run; they are read from the `key: value`
    lines of a small record kept beside the profile summaries.  A record carries the hash of the kernel source it was
    taken on: once that source changes the figures are reported as null."""
    import hashlib
    path = os.path.join(ROOT, "profiles", name)
    rec = {}
    try:
        with open(path) as f:
            for line in f:
                if ":" in line and not line.startswith("#"):
                    k, v = line.split(":", 1)
                    rec[k.strip()] = v.strip()
        with open(os.path.join(ROOT, "paper_2306_17266_b200", "csrc", rec["kernel_source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest()[:16] != rec["kernel_source_sha256_16"]:
                return None
    except (OSError, KeyError):
        return None
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="sgs", choices=["sgs", "reference"])
    ap.add_argument("--queries", type=int, default=1000, help="queries per step")
    ap.add_argument("--cpu-queries", type=int, default=24, help="queries the CPU baseline is timed on (0 = skip)")
    ap.add_argument("--ref-queries", type=int, default=8, help="queries per step of --impl reference")
    ap.add_argument("--cache", type=int, default=1)
    ap.add_argument("--window", type=int, default=4)
    ap.add_argument("--wave", type=int, default=32, help="queries per wave (grouped launches over the wave's members); 0 = one stream per query")
    ap.add_argument("--concurrency", type=int, default=None, help="waves in flight (default 4), or with --wave 0 queries in flight (default 16)")
    ap.add_argument("--quick", action="store_true", help="default line without the sweep / depthwise / MobileNetV3 / plan-miss measurements")
    ap.add_argument("--sweep-groups", type=int, default=1250, help="16-image groups per resolution of the sweep measured inside the default line")
    ap.add_argument("--batch", type=int, default=1, help="images per query (sgs-probe)")
    ap.add_argument("--evict-first", type=int, default=0, help="with --cache 0: mark weight loads evict-first (sgs-probe)")
    ap.add_argument("--option", action="append", default=[], help="library tuning aid as name=value (sgs_set_option), may repeat")
    ap.add_argument("--res", type=int, default=0, help="sweep suite: only this resolution (profiling a single launch shape)")
    ap.add_argument("--mechanism", type=int, default=0, help="sgs-probe: 0 per-tile L2 hints, 1 access-policy window per launch, 2 both")
    ap.add_argument("--budget-mb", type=int, default=0, help="sgs-probe: cache budget in MiB (0 = device maximum)")
    ap.add_argument("--persistent", action="store_true", help="mbv3 suite: only the persistent SubNet kernel (one launch per pass over the queries)")
    ap.add_argument("--family", default="resnet", choices=["resnet", "mbv3"], help="SuperNet of the sched suite")
    ap.add_argument("--suite", default="stream", choices=["stream", "sweep", "sgs", "sgs-probe", "mbv3", "sched", "table", "dw"],
                    help="stream = the default benchmark line; the others measure one more configuration each")
    args = ap.parse_args()
    if args.concurrency is None:
        args.concurrency = 4 if args.wave > 0 else 16
    EXTRA_OPTIONS.extend((o.split("=")[0], int(o.split("=")[1])) for o in args.option)
    if args.impl == "reference":
        run_reference(args)
        return
    if args.suite != "stream":
        run_suite(args)
        return

    import torch
    import paper_2306_17266_b200 as sgs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    peaks = measured_peaks()
    nq = args.queries
    warmup = max(3, args.warmup)
    # replicas: every rank holds the SuperNet and serves its own query stream (no data-path collective)
    blob = wl.make_blob(wl.RESNET, seed=0, bf16_weights=True)
    net = apply_options(sgs.SuperNet(wl.RESNET, blob, sgs.SGS_BF16, device=local))
    from paper_2306_17266_b200 import replicas
    # N replicas serve a stream of N * nq queries (weak scaling); queries whose SubNets are close in the vector
    # encoding go to the same replica, so that each replica's SubGraph cache sees a larger common SubGraph.  Every
    # rank computes the same partition by itself.  With one replica the shard is the stream as it is.
    base = wl.uniform_stream(wl.RESNET, nq * world, seed=2)
    if world > 1:
        enc = np.stack([np.asarray(net.subnet_encode(c)).reshape(-1, 3)[:, :2].reshape(-1) for c in base])
        cfgs = [base[q] for q in replicas.affinity_shards(enc, world)[rank]]
    else:
        cfgs = base
    arr = wl.cfg_array(cfgs)
    x_host = torch.from_numpy(wl.make_inputs(nq, BATCH, RES, seed=1 + rank, bf16=True).reshape(nq * BATCH, RES, RES, 3))
    x_host = x_host.to(torch.bfloat16).contiguous().pin_memory()
    x_dev = x_host.cuda()
    logits = torch.zeros((nq * BATCH, 1000), dtype=torch.float32, device="cuda")
    logits_host = torch.zeros((nq * BATCH, 1000), dtype=torch.float32).pin_memory()
    stream = torch.cuda.Stream()

    def mk_opts(graphs=1, latency=0, conc=None, wave=None):
        return sgs.StreamOpts(cache_enabled=args.cache, window_q=args.window, cache_budget_bytes=0, use_graphs=graphs,
                              record_latency=latency, weights_evict_first=0, concurrency=args.concurrency if conc is None else conc,
                              wave=args.wave if wave is None else wave)

    def step(host=False, o=None):
        o = o or mk_opts()
        if host:
            return net.stream_run(arr, x_host.data_ptr(), BATCH, RES, logits_host.data_ptr(), o, stream.cuda_stream, host=True)
        return net.stream_run(arr, x_dev.data_ptr(), BATCH, RES, logits.data_ptr(), o, stream.cuda_stream)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = 0
        e0.record(stream)
        for _ in range(steps):
            launches += fn().kernel_launches
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, launches

    for _ in range(warmup):
        step()
    sampler = ClockSampler(local)
    sampler.start()
    ms, launches = timed(step, args.steps)
    clocks = sampler.stop()
    value = world * nq * args.steps / (ms * 1e-3)

    # latency distribution (one extra pass with per-query events)
    st_lat = step(o=mk_opts(latency=1))

    # end to end: host buffers in, host logits out, copies inside the timed region
    step(host=True)
    ms_e2e, _ = timed(lambda: step(host=True), args.steps)
    e2e_value = world * nq * args.steps / (ms_e2e * 1e-3)
    in_bytes = nq * BATCH * RES * RES * 3 * 2
    out_bytes = nq * BATCH * 1000 * 4

    out = None
    if rank == 0:
        # Dominant kernel: the tensor-core convolution.  Kernels of several waves overlap in the timed
        # region, so its launches are timed in one more pass of the same stream with one wave at a time: an
        # event pair on the launching stream around every launch, the stream held by a sleeping kernel while
        # the host queues the wave (the intervals then hold device time, not launch latency).
        step(o=mk_opts(conc=1, wave=0))  # (first pass: plans and graphs of this execution mode)
        seq_lat = step(o=mk_opts(conc=1, latency=1, wave=0))
        net.set_option("profile", 2)
        step(o=mk_opts(graphs=0))
        prof = [net.profile_read(c) for c in range(4)]
        net.set_option("profile", 0)
        tc = prof[0]
        total_ms = sum(p["total_ms"] for p in prof)
        share = tc["total_ms"] / total_ms if total_ms > 0 else 0.0
        sec = tc["total_ms"] * 1e-3
        n_launch = max(1, tc["launches"])
        us_launch = sec * 1e6 / n_launch
        achieved_gbs = tc["alg_bytes"] / sec / 1e9 if sec > 0 else 0.0
        achieved_tf = tc["flops"] / sec / 1e12 if sec > 0 else 0.0
        grouped = args.wave > 0
        rec = ncu_record("conv_group_wave32_resnet_b1.counters.txt") if grouped else None
        traffic = float(rec["dram_bytes_per_launch"]) if rec else None
        ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
        flop_per_launch = tc["flops"] / n_launch
        # what bounds a launch: FLOP per byte that actually crosses the DRAM interface (members of a wave share the
        # weights they have in common) against the ridge of the measured peaks; per ALGORITHMIC byte when there is no
        # counter for the kernel as it stands
        # (the counters are cold-cache, an upper bound of the traffic in the timed region, so a launch within a
        # quarter of the ridge counts as tensor bound: the tensor fraction is then also the lower, stricter figure)
        intensity = flop_per_launch / traffic if traffic else tc["flops"] / max(1.0, tc["alg_bytes"])
        bound = "tensor" if intensity >= 0.75 * ridge else "hbm"
        in_flight_gbs = sum(p["alg_bytes"] for p in prof) / (ms / args.steps * 1e-3) / 1e9
        in_flight_tf = st_lat.useful_flops / (ms / args.steps * 1e-3) / 1e12
        hbm_view = {"achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved_gbs / peaks["hbm_gbs"],
                    "what": "algorithmic bytes (sliced weights + input + output + residual of every member) / launch time, launches timed one wave at a time"}
        tensor_view = {"achieved": achieved_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved_tf / peaks["bf16_tflops"],
                       "what": "useful FLOPs (2*M*K'*C'*k*k on the sliced extents) / launch time, launches timed one wave at a time; burst bf16 peak"}
        head = tensor_view if bound == "tensor" else hbm_view
        roofline = {
            "kernel": ("conv_group_kernel (one launch = one stored layer for all members of a wave; sliced implicit GEMM, tcgen05 + TMA)" if grouped
                       else "conv_tc_kernel (sliced implicit-GEMM convolution, tcgen05 + TMA)"),
            "bound": bound, "achieved": head["achieved"], "peak": head["peak"], "unit": head["unit"], "frac": head["frac"],
            "traffic": traffic,
            "traffic_note": (rec or {}).get("note", "no counter record for the kernel source as it stands"),
            "peak_source": peaks["source"],
            "intensity_flop_per_dram_byte": intensity, "ridge_flop_per_byte": ridge,
            "launches": tc["launches"], "avg_launch_us": us_launch,
            "method": "CUDA events around every launch on the launching stream, one wave at a time, host launch latency hidden behind a sleeping kernel",
            "alg_bytes_per_launch": tc["alg_bytes"] / n_launch, "flop_per_launch": flop_per_launch,
            "share_of_kernel_time": share,
            "isolated_launch": {"tensor": tensor_view, "hbm_algorithmic": hbm_view,
                                "dram_measured": ({"achieved": traffic / (us_launch * 1e-6) / 1e9, "unit": "GB/s", "frac": traffic / (us_launch * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                                   "what": "DRAM read + write bytes per launch from the profiler's counters / launch time"} if traffic else None)},
            "in_flight": {"what": "the timed region itself (waves overlap; all kernels together): algorithmic bytes and useful FLOPs of a step / ms_per_step",
                          "alg_gbs": in_flight_gbs, "frac_of_hbm_peak": in_flight_gbs / peaks["hbm_gbs"],
                          "useful_tflops": in_flight_tf, "frac_of_bf16_burst_peak": in_flight_tf / peaks["bf16_tflops"],
                          "frac_of_bf16_sustained_peak": in_flight_tf / peaks["bf16_tflops_sustained"]},
            "kernel_time_ms_by_class": {"conv_tc": prof[0]["total_ms"], "conv_cuda_core": prof[1]["total_ms"],
                                        "depthwise": prof[2]["total_ms"], "other": prof[3]["total_ms"]},
        }
        extras = {}
        if world == 1 and not args.quick:
            extras["plan_miss"] = measure_plan_miss(net, sgs, torch, stream, x_dev, logits, mk_opts())
            sweep_rows = measure_sweep(net, sgs, torch, stream, peaks, n_groups=args.sweep_groups, concurrency=args.concurrency)
            extras["sweep"] = {"workload": SWEEP_WORKLOAD + f", {args.sweep_groups * 16} images per resolution", "rows": sweep_rows}
            fma = sgs.measure_fma_peak(stream.cuda_stream)
            extras["depthwise"] = {"workload": "depthwise k x k (centre window of the stored 7x7), 64 x 56 x 56 x 480 bf16, h-swish: working set beyond L2",
                                   "fp32_fma_tflops_measured": fma, "rows": measure_depthwise(sgs, peaks, fma)}
            extras["mbv3"] = {"workload": "MobileNetV3-shaped SuperNet, 1000-query stream at batch 1, 224x224, configs uniform (seed 3)",
                              **measure_mbv3(sgs, torch, stream, 1000, args.wave, args.concurrency, args.cache, args.window)}
            sgs_rec = ncu_record("sgs_cache_wave_dram_bytes.counters.txt")
            extras["sgs_measured"] = sgs_rec
        cpu = None
        if args.cpu_queries > 0 and world == 1:
            qps, dt, cores = cpu_oracle_qps(args.cpu_queries)
            cpu = {"value": qps, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"first {args.cpu_queries} queries of the same stream, {dt:.1f} s"}
        cs = net.cache_stats()
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "queries_per_step": nq, "batch": BATCH, "res": RES,
                       "l2": "inputs (301 MB per step) and the SuperNet (96 MB) exceed L2; no flush",
                       "cache": bool(args.cache), "window_q": args.window,
                       "execution": (f"waves of {args.wave} queries, one grouped launch per layer, {args.concurrency} waves in flight" if args.wave > 0
                                     else f"one stream per query, {args.concurrency} queries in flight"),
                       "parallelism": f"replicas x{world}" + (", stream sharded by config affinity" if world > 1 else "")},
            "p50_ms": st_lat.p50_ms, "p99_ms": st_lat.p99_ms, "mean_ms": st_lat.mean_ms,
            "one_query_at_a_time": {"queries_per_s": seq_lat.queries_per_s, "p50_ms": seq_lat.p50_ms, "p99_ms": seq_lat.p99_ms},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": out_bytes},
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu,
            "useful_tflops": st_lat.useful_flops / (st_lat.total_ms * 1e-3) / 1e12,
            **extras,
            "sgs": {"weight_bytes_per_query": st_lat.weight_bytes / nq, "hbm_weight_bytes_per_query": st_lat.hbm_weight_bytes / nq,
                    "hit_ratio": st_lat.hit_ratio, "byte_hit_ratio": st_lat.byte_hit_ratio, "cache_updates": st_lat.cache_updates,
                    "budget_bytes": cs.budget_bytes, "l2_bytes": cs.l2_bytes},
        }
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
