#!/usr/bin/env python
"""Benchmark of the MLA shared-prefix decode attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg1] [--mode auto|hybrid|absorb]
    python bench.py --impl reference ...      # the float64 CPU checker on the host cores
    python bench.py --sweep                   # config 4 fan-out sweep (one JSON line per batch size)

One step = one pass of the whole path (Algorithm 1 lines 4-8: naive shared attention, query
absorption, absorb suffix attention, split merge, W_UV projection, LSE combine) over one batch of
synthetic requests.  Metric: decode-attention queries/s (one query = one request's token across
all heads).  Prints one JSON line.  With N > 1 (torchrun) every rank runs an independent replica
on its own requests (the path shards by request with no exchange): weak scaling.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mla_decode_attention_queries_per_s"
UNIT = "queries/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu capture
# of that kernel at that configuration (key: (config, kernel)); None where no capture exists.
NCU_TRAFFIC_BYTES = {
    ("cfg1", "naive_attn"): 275_997_696,
    ("cfg3", "absorb_attn"): 652_403_968,
    ("cfg4_B512", "naive_attn"): 1_163_312_528,
}
MIN_REGION_MS = 50.0      # every timed region is repeated until this much GPU time has been measured
MAX_REPEATS = 400


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------ work accounting
def algorithmic_work(cfg, suffix_lens, mode_name, fp8=False):
    """Algorithmic flops and bytes of one step (Table 1 terms plus the once-only reads of q and the
    weights and the write of out); with the 8-bit expanded cache K_nope and V cost one byte per element."""
    H, B, Ls = cfg.H, cfg.B, cfg.Ls
    sum_ln = sum(suffix_lens)
    W = 4 * H * 65536
    if mode_name == "absorb":
        flops = H * (2176 * (B * Ls + sum_ln) + 4 * 65536 * B)
        bytes_ = 1152 * Ls + W + 1152 * sum_ln + 640 * H * B
    else:
        flops = H * (640 * B * Ls + 2176 * sum_ln + 4 * 65536 * B)
        bytes_ = ((256 if fp8 else 512) * H + 128) * Ls + W + 1152 * sum_ln + 640 * H * B
    return flops, bytes_


def dominant_kernel(cfg, suffix_lens, mode_name, fp8=False):
    """(kernel id, name, bound, algorithmic bytes per launch, flops per launch) of the kernel that
    carries most of the step's roofline time."""
    H, B, Ls = cfg.H, cfg.B, cfg.Ls
    sum_ln = sum(suffix_lens)
    naive_bytes = ((256 if fp8 else 512) * H + 128) * Ls + 384 * B * H   # expanded K/V + rope keys once, q once
    naive_flops = 640 * B * H * Ls
    if mode_name == "absorb":
        absorb_bytes = 1152 * (B * Ls + sum_ln) + 1152 * B * H   # latent tokens per request + Q_A|q_pe
        absorb_flops = 2176 * H * (B * Ls + sum_ln)
        return 2, "absorb_attn", absorb_bytes, absorb_flops
    absorb_bytes = 1152 * sum_ln + 1152 * B * H
    absorb_flops = 2176 * H * sum_ln
    pk = _peaks()
    t_naive = max(naive_bytes / (pk["hbm_gbs"] * 1e9), naive_flops / (pk["bf16_tflops"] * 1e12))
    t_abs = max(absorb_bytes / (pk["hbm_gbs"] * 1e9), absorb_flops / (pk["bf16_tflops"] * 1e12))
    if t_naive >= t_abs:
        return 0, "naive_attn", naive_bytes, naive_flops
    return 2, "absorb_attn", absorb_bytes, absorb_flops


# ------------------------------------------------------------------ multi-rank helpers (no data-path collective)
def rank_config(cfg, rank):
    """Each rank serves its own requests: same prefix and weights (same seed for the shared draws would need
    the same generator, so the whole problem is re-drawn with a rank-shifted seed); rank 0 keeps the config."""
    return cfg if rank == 0 else dataclasses.replace(cfg, seed=cfg.seed + 1000 * rank)


def max_over_ranks(ms, world, device):
    """Timing of a multi-rank run is the slowest rank's (MAX all-reduce); the only collective in the bench."""
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(per_rank_batch, world, ms_per_step):
    """queries/s of the whole job: every rank processes `per_rank_batch` queries per step (weak scaling)."""
    return world * per_rank_batch / (ms_per_step * 1e-3)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {}
        for k in dir(nv):
            if k.startswith("nvmlClocksEventReason") or k.startswith("nvmlClocksThrottleReason"):
                v = getattr(nv, k)
                if isinstance(v, int) and v:
                    names.setdefault(v, k.replace("nvmlClocksEventReason", "").replace("nvmlClocksThrottleReason", ""))
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                if get_reasons:
                    r = int(get_reasons(self.h))
                    for bit, name in names.items():
                        if bit and (r & bit) == bit and bin(bit).count("1") == 1:
                            self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.001)

    def __enter__(self):
        if self.nv:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        if self._thr:
            self._stop.set()
            self._thr.join()

    def summary(self):
        idle = {"GpuIdle", "None", "ApplicationsClocksSetting"}
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_min_mhz": (min(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
                "reasons": sorted(r for r in self.reasons if r not in idle)}


# ------------------------------------------------------------------ CPU checker timing
def time_oracle_sample(inp, heads, target_requests=None):
    """Times the float64 CPU checker, as it stands, on all requests x the first `heads` heads and
    scales to all heads.  Returns (queries/s, seconds, cores, sample description)."""
    import numpy as np  # noqa: F401
    from oracle import mla_oracle as O
    from paper_2509_21081_b200 import inputs as I
    cfg = inp.cfg
    f = I.to_f64
    nb = cfg.B if target_requests is None else min(cfg.B, target_requests)
    args = (f(inp.q_nope), f(inp.q_pe), f(inp.ckv_shared), f(inp.kpe_shared),
            [f(x) for x in inp.ckv_suffix], [f(x) for x in inp.kpe_suffix], f(inp.w_uk), f(inp.w_uv), inp.scale)
    pairs = [(b, h) for h in range(heads) for b in range(nb)]
    t0 = time.perf_counter()
    O.mla_decode(*args, pairs=pairs)
    dt = time.perf_counter() - t0
    scaled = dt * (cfg.H / heads)
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count()])
    except Exception:
        cores = os.cpu_count()
    return nb / scaled, dt, int(cores), f"{nb} requests x {heads} of {cfg.H} heads, time scaled by {cfg.H / heads:g}"


# ------------------------------------------------------------------ main arms
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2509_21081_b200 import inputs as I
    cfg = I.CONFIGS[args.config]
    inp = I.make_inputs(cfg)
    # Size the per-step sample (heads) so that the K timed steps take about two minutes in total.
    _, t1, _, _ = time_oracle_sample(inp, 1)
    for _ in range(max(args.warmup - 1, 0)):
        time_oracle_sample(inp, 1)
    K = max(args.steps, 1)
    heads = max(1, min(cfg.H, args.ref_heads, int(120.0 / (K * max(t1, 1e-3)))))
    vals = []
    for _ in range(K):
        qps, dt, cores, sample = time_oracle_sample(inp, heads)
        vals.append((qps, dt))
    qps = statistics.median(v[0] for v in vals)
    ms = cfg.B / qps * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": qps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": _workload_name(cfg)},
            "cpu_baseline": {"value": qps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": qps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def _workload_name(cfg):
    return (f"{cfg.name}: B={cfg.B} H={cfg.H} Ls={cfg.Ls} Ln=[{cfg.suffix_lo},{cfg.suffix_hi}] "
            f"page={cfg.page_size} d=(128,64,128,512) bf16")


def bench_config(cfg, args, mode, rank, world, device_index, with_cpu=True, with_e2e=True, max_steps=None, fp8=False):
    """One configuration: K steps per timed region, the region repeated until MIN_REGION_MS of GPU time
    has been measured (median of the repeats reported; the clock sampler runs over all of them), then
    the dominant kernel's duration inside the step and alone, optionally per-stage times, the end-to-end
    figures and the CPU checker."""
    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder

    dev = "cuda"
    # Each rank draws its own requests (seed shifted by rank); the prefix and weights are replicated.
    rcfg = rank_config(cfg, rank)
    inp = I.make_inputs(rcfg)
    pc = I.build_pages(inp, poison=False)
    max_pages = pc.block_table.shape[1]
    # Two full copies of everything a step touches, used alternately, so that no step finds the
    # previous step's data in the 126 MB L2 (each copy alone is larger than L2 for configs 1-4).
    n_sets = 2
    sets = []
    prepare_ms = None
    for k in range(n_sets):
        dev_in = (inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), inp.w_uk.to(dev), inp.w_uv.to(dev))
        # the one-off expansion of the prefix (not part of a step): timed on the second set, after the first
        # has paid for context and module loading
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        pe0.record()
        dec = TyphoonMLADecoder(cfg.H, *dev_in, inp.scale, cfg.B, max_pages, pc.page_size, fp8_shared=fp8)
        pe1.record()
        if k == 1:
            torch.cuda.synchronize()
            prepare_ms = pe0.elapsed_time(pe1)
        sets.append(dict(dec=dec, q_nope=inp.q_nope.to(dev), q_pe=inp.q_pe.to(dev), ckv=pc.ckv_pages.to(dev),
                         kpe=pc.kpe_pages.to(dev), bt=pc.block_table.to(dev), sl=pc.seq_lens.to(dev),
                         out=torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16, device=dev)))
    resolved = mode if mode != b.MODE_AUTO else sets[0]["dec"].choose_mode(cfg.B, sum(inp.suffix_lens))
    mode_name = b.MODE_NAMES[resolved]

    def step(i):
        s = sets[i % n_sets]
        s["dec"].decode(s["q_nope"], s["q_pe"], s["ckv"], s["kpe"], s["bt"], s["sl"], mode=mode, out=s["out"])

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    W, K = max(args.warmup, 3), max(args.steps, 1)
    if max_steps:
        K = min(K, max_steps)
    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    launches_per_step = b.typhoon_mla_last_launch_count()
    assert b.typhoon_mla_check_status(sets[0]["dec"].shared) == 0 and b.typhoon_mla_check_status(sets[1]["dec"].shared) == 0
    kid, kname, k_bytes, k_flops = dominant_kernel(cfg, inp.suffix_lens, mode_name, fp8)

    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def region(fn, n):
        """n calls of fn bracketed by a barrier + synchronize on both sides; device time in ms (max over ranks)."""
        barrier()
        ev0.record()
        for i in range(n):
            fn(i)
        ev1.record()
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), world, dev)

    def repeated(fn, n):
        """Repeats the n-call region until MIN_REGION_MS of device time has been measured (at least 3
        times); returns the per-call times of the repeats."""
        runs, total = [], 0.0
        while (total < MIN_REGION_MS or len(runs) < (3 if MIN_REGION_MS > 0 else 1)) and len(runs) < MAX_REPEATS:
            ms = region(fn, n)
            runs.append(ms / n)
            total += ms
        return runs

    # ---- device-resident timing: regions of exactly K steps, nothing else on the stream
    with ClockSampler(device_index) as clocks:
        step_runs = repeated(step, K)
    ms_per_step = statistics.median(step_runs)
    value = whole_job_value(cfg.B, world, ms_per_step)

    # ---- the same steps again with a pair of CUDA events around every launch of the dominant kernel
    # (on the stream it is launched on).  Event records cost several microseconds per step and, with
    # programmatic launches, change the order in which the two streams' kernels get their SMs (an event in
    # front of a kernel delays it behind the side stream's kernels), so this second timed region runs with
    # ordinary stream-ordered launches and is only used for the kernel's duration inside a step; its own
    # step time is reported next to it.
    n_prof = int(min(2000, max(K, MIN_REGION_MS / max(ms_per_step, 1e-3))))
    b.typhoon_mla_set_programmatic_launch(False)
    for i in range(3):
        step(i)
    b.typhoon_mla_profile_begin(kid, n_prof)
    instrumented_ms_per_step = region(step, n_prof) / n_prof
    k_ms, k_n = b.typhoon_mla_profile_end()
    b.typhoon_mla_set_programmatic_launch(True)

    # ---- roofline of the dominant kernel
    pk = _peaks()
    k_avg_s = (k_ms / max(k_n, 1)) * 1e-3
    t_mem = k_bytes / (pk["hbm_gbs"] * 1e9)
    t_cmp = k_flops / (pk["bf16_tflops_sustained"] * 1e12)
    if t_mem >= t_cmp:
        achieved = k_bytes / k_avg_s / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / pk["hbm_gbs"]}
    else:
        # timed inside a long loop under the power cap: the sustained figure is the denominator; the
        # fraction of the burst figure is printed next to it
        achieved = k_flops / k_avg_s / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                "frac": achieved / pk["bf16_tflops_sustained"], "frac_of_burst_peak": achieved / pk["bf16_tflops"],
                "burst_peak": pk["bf16_tflops"]}
    roof.update({"traffic": None if fp8 else NCU_TRAFFIC_BYTES.get((cfg.name, kname)), "kernel": kname,
                 "kernel_ms": k_avg_s * 1e3, "launches_timed": k_n,
                 "ms_per_step_with_kernel_events": instrumented_ms_per_step, "peak_source": pk["source"],
                 "algorithmic_bytes": k_bytes, "algorithmic_flops": k_flops})
    flops, bytes_ = algorithmic_work(cfg, inp.suffix_lens, mode_name, fp8)
    t_lb = max(flops / (pk["bf16_tflops"] * 1e12), bytes_ / (pk["hbm_gbs"] * 1e9))
    roof["step_frac_of_combined_roofline"] = t_lb / (ms_per_step * 1e-3)
    # The same kernel with the side stream switched off (every kernel alone on the GPU), outside the
    # timed region: what the kernel reaches when it does not share the machine.
    b.typhoon_mla_set_overlap(False)
    n_alone = int(min(2000, max(5, min(K, 50), 0.5 * MIN_REGION_MS / max(ms_per_step, 1e-3))))
    for i in range(3):
        step(i)
    b.typhoon_mla_profile_begin(kid, n_alone)
    for i in range(n_alone):
        step(i)
    a_ms, a_n = b.typhoon_mla_profile_end()
    b.typhoon_mla_set_overlap(True)
    a_s = (a_ms / max(a_n, 1)) * 1e-3
    alone = (k_bytes / a_s / 1e9) if roof["bound"] == "hbm" else (k_flops / a_s / 1e12)
    roof.update({"kernel_ms_alone": a_s * 1e3, "achieved_alone": alone, "frac_alone": alone / roof["peak"]})
    if roof["bound"] == "tensor":
        roof["frac_alone_of_burst_peak"] = alone / pk["bf16_tflops"]
    # second column: the same fractions against the data-sheet peaks (8 TB/s HBM3e, 2.25 PFLOP/s dense bf16)
    nominal = 8000.0 if roof["bound"] == "hbm" else 2250.0
    roof.update({"nominal_peak": nominal, "frac_of_nominal": roof["achieved"] / nominal,
                 "frac_alone_of_nominal": alone / nominal})

    # ---- per-stage times (the layout of the paper's Fig. 4 / Fig. 8: stage 1 = naive shared attention, stage 2
    # = absorb attention, plus the projections and the merge), every kernel alone on the GPU: side stream
    # off, ordinary launches, a CUDA-event pair around each launch
    stages = None
    if getattr(args, "stages", False):
        b.typhoon_mla_set_overlap(False)
        b.typhoon_mla_set_programmatic_launch(False)
        stages = {}
        n_st = max(5, min(K, 20))
        for k_id, k_name in enumerate(b.KERNEL_NAMES):
            for i in range(2):
                step(i)
            b.typhoon_mla_profile_begin(k_id, n_st)
            for i in range(n_st):
                step(i)
            s_ms, s_n = b.typhoon_mla_profile_end()
            if s_n:
                stages[k_name + "_ms"] = s_ms / s_n
        b.typhoon_mla_set_overlap(True)
        b.typhoon_mla_set_programmatic_launch(True)

    # ---- end to end: per-step tensors from pinned host memory, result read back, every step
    e2e = None
    if with_e2e:
        # Twelve steps are kept in flight ("lanes"), each on its own stream with its own decoder (prepared
        # prefix, workspace, staging) and pinned buffers, so that the copies of one step overlap the kernels
        # of the others, as a serving loop with several micro-batches would do.  Every step still copies
        # its inputs in and its result out.  Lane k reads the device-resident caches of input set k % 2.
        # (A lane's copy out waits for its kernels, and the copy queues run in submission order, so with only
        # a few lanes the next lanes' copies in sit behind it: measured 237-250 / 180 / 105-147 / 95 / 95 us per
        # step with 2 / 4 / 6 / 8 / 12 lanes on one GPU.)
        n_lanes = int(os.environ.get("TYPHOON_MLA_BENCH_LANES", "12"))
        lanes = []
        for k in range(n_lanes):
            s = sets[k % n_sets]
            dec = s["dec"] if k < n_sets else TyphoonMLADecoder(
                cfg.H, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), s["dec"].w_uk, s["dec"].w_uv, inp.scale,
                cfg.B, max_pages, pc.page_size, fp8_shared=fp8)
            lanes.append(dict(dec=dec, ckv=s["ckv"], kpe=s["kpe"], stream=torch.cuda.Stream(),
                              h=(inp.q_nope.pin_memory(), inp.q_pe.pin_memory(), pc.block_table.pin_memory(),
                                 pc.seq_lens.pin_memory(),
                                 torch.empty(cfg.B, cfg.H, 128, dtype=torch.bfloat16).pin_memory())))
        streams = [ln["stream"] for ln in lanes]

        def step_host(i):
            ln = lanes[i % n_lanes]
            h = ln["h"]
            with torch.cuda.stream(ln["stream"]):
                ln["dec"].decode_host(h[0], h[1], ln["ckv"], ln["kpe"], h[2], h[3], h[4], mode=mode)

        def fork():
            for st in streams:
                st.wait_stream(torch.cuda.current_stream())

        def join():
            for st in streams:
                torch.cuda.current_stream().wait_stream(st)

        fork()
        for i in range(W):
            step_host(i)
        join()
        # regions of K steps (fork, K host-fed steps round robin over the lanes, join), repeated like the
        # device-resident regions; the median is reported
        e_runs, total = [], 0.0
        while (total < MIN_REGION_MS or len(e_runs) < (3 if MIN_REGION_MS > 0 else 1)) and len(e_runs) < MAX_REPEATS:
            barrier()
            ev0.record()
            fork()
            for i in range(K):
                step_host(i)
            join()
            ev1.record()
            barrier()
            ms = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
            e_runs.append(ms / K)
            total += ms
        e_ms = statistics.median(e_runs)
        # One step in flight, as a decode loop sees it: copy in, step, copy out, wait for the result, then the
        # next step (lane 0 and lane 1 alternately so that L2 does not hold the previous step's cache lines).
        # Host clock around the loop: the launch path and the wake-up after the synchronise are part of it.
        n_lat = int(min(2000, max(K, MIN_REGION_MS / max(e_ms, 1e-3))))
        for i in range(3):
            step_host(i % 2)
            lanes[i % 2]["stream"].synchronize()
        barrier()
        t0 = time.perf_counter()
        for i in range(n_lat):
            step_host(i % 2)
            lanes[i % 2]["stream"].synchronize()
        lat_ms = (time.perf_counter() - t0) * 1e3 / n_lat
        lat_ms = max_over_ranks(lat_ms, world, dev)
        h2d = inp.q_nope.numel() * 2 + inp.q_pe.numel() * 2 + pc.block_table.numel() * 4 + pc.seq_lens.numel() * 4
        d2h = cfg.B * cfg.H * 128 * 2
        e2e = {"value": whole_job_value(cfg.B, world, e_ms), "unit": UNIT, "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "repeats": len(e_runs), "min_ms_per_step": min(e_runs), "max_ms_per_step": max(e_runs),
               "pipelining": f"{n_lanes} steps in flight on {n_lanes} streams (own decoder, workspace, staging and pinned buffers each)",
               "e2e_latency_ms": lat_ms, "e2e_latency_steps": n_lat,
               "e2e_latency_value": whole_job_value(cfg.B, world, lat_ms),
               "e2e_latency_note": "one step in flight: pinned host inputs copied in, step, result copied out, stream synchronised, host clock"}
        for ln in lanes[n_sets:]:
            ln["dec"].close()

    cpu = None
    if with_cpu and rank == 0 and world == 1:
        heads = max(1, min(cfg.H, args.ref_heads))
        qps, dt, cores, sample = time_oracle_sample(inp, heads)
        cpu = {"value": qps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": dt}

    for s in sets:
        s["dec"].close()
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if not fp8 else "bf16 (expanded shared K/V stored as e4m3 codes, widened exactly to f16 operands)",
            "data": "synthetic",
            # `config` names the workload and how L2 is kept cold; how this arm ran it is in `run`
            "config": {"workload": _workload_name(cfg),
                       "l2": f"{n_sets} full input sets used alternately, each larger than the 126 MB L2"},
            "run": {"mode": mode_name, "requested_mode": b.MODE_NAMES[mode],
                    "parallelism": f"replicas x{world} (shard by request, no exchange)",
                    "timing": f"regions of {K} steps repeated until {MIN_REGION_MS:g} ms of device time; median of the repeats"},
            "timed_regions": {"repeats": len(step_runs), "min_ms_per_step": min(step_runs), "max_ms_per_step": max(step_runs)},
            "clocks": clocks.summary(), "e2e": e2e, "stages": stages, "gpu_launches": launches_per_step * K,
            "prepare_shared_ms": prepare_ms,
            "roofline": roof, "cpu_baseline": cpu}
    return line


# Configurations reported next to the headline one in the default run: the other benchmark configurations,
# the fan-out sweep at the batch sizes on either side of the crossover and in the compute-bound regime.
EXTRA_CONFIGS = (("cfg2", 0), ("cfg3", 0), ("cfg4", 8), ("cfg4", 128), ("cfg4", 512), ("cfg4", 1024))


def bench_extra_configs(args, rank, world, device_index):
    """Short lines for the other benchmark configurations (mode AUTO, same timing method, at most 20 steps per
    region): step time, resolved mode, the dominant kernel and its roofline fractions inside the step and
    alone, the sampled clocks."""
    import gc
    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    out = []
    for name, batch in EXTRA_CONFIGS:
        cfg = I.CONFIGS[name]
        if batch:
            cfg = cfg.with_batch(batch)
        ln = bench_config(cfg, args, b.MODE_AUTO, rank, world, device_index, with_cpu=False, with_e2e=False, max_steps=20)
        r = ln["roofline"]
        out.append({"workload": ln["config"]["workload"], "mode": ln["run"]["mode"], "value": ln["value"],
                    "ms_per_step": ln["ms_per_step"], "steps": ln["steps"], "timed_regions": ln["timed_regions"],
                    "gpu_launches": ln["gpu_launches"], "dominant_kernel": r["kernel"], "bound": r["bound"],
                    "peak": r["peak"], "unit": r["unit"], "achieved": r["achieved"], "frac": r["frac"],
                    "achieved_alone": r["achieved_alone"], "frac_alone": r["frac_alone"],
                    "frac_of_burst_peak": r.get("frac_of_burst_peak"), "frac_alone_of_burst_peak": r.get("frac_alone_of_burst_peak"),
                    "frac_of_nominal": r["frac_of_nominal"], "kernel_ms": r["kernel_ms"], "kernel_ms_alone": r["kernel_ms_alone"],
                    "step_frac_of_combined_roofline": r["step_frac_of_combined_roofline"], "clocks": ln["clocks"]})
        gc.collect()
        torch.cuda.empty_cache()
    return out


def bench_extension(cfg, args, device_index):
    """Measurement of the two extensions of the path (one GPU, device-resident inputs, two input sets
    alternated, CUDA events): --sq S = S query tokens per request (rows = (request, token) pairs, causal
    among the new tokens); --tree G:L = the config's prefix as the root of all requests plus G groups of
    B/G requests with a further shared prefix of L tokens each.  One JSON line, queries = rows."""
    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    dev = "cuda"
    W, K = max(args.warmup, 3), max(args.steps, 1)
    H, B, Ls = cfg.H, cfg.B, cfg.Ls
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=False)
    dims = b.make_dims(H)
    S_q = max(args.sq, 1)
    rows = B * S_q
    if args.tree:
        G_, L_ = (int(x) for x in args.tree.split(":"))
        assert B % G_ == 0 and S_q == 1
    sets = []
    for _ in range(2):
        w_uk, w_uv = inp.w_uk.to(dev), inp.w_uv.to(dev)
        root = b.typhoon_mla_prepare_shared(dims, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), w_uk, w_uv)
        levels = [([root], [0, rows])]
        if args.tree:
            g = torch.Generator(device="cpu")
            g.manual_seed(cfg.seed + 99)
            br = [b.typhoon_mla_prepare_shared(dims, torch.randn(L_, 512, generator=g).to(torch.bfloat16).to(dev),
                                               torch.randn(L_, 64, generator=g).to(torch.bfloat16).to(dev), w_uk, w_uv)
                  for _ in range(G_)]
            levels.append((br, [i * (B // G_) for i in range(G_ + 1)]))
        bt, sl = pc.block_table.to(dev), pc.seq_lens.to(dev)
        if S_q > 1:
            bt, sl = b.typhoon_mla_expand_query_rows(bt, sl, S_q)
        q_nope = inp.q_nope.to(dev).repeat_interleave(S_q, dim=0).contiguous()
        q_pe = inp.q_pe.to(dev).repeat_interleave(S_q, dim=0).contiguous()
        ws = torch.empty(b.typhoon_mla_tree_workspace_bytes(levels, rows, bt.shape[1], pc.page_size), dtype=torch.uint8,
                         device=dev)
        sets.append(dict(levels=levels, q_nope=q_nope, q_pe=q_pe, ckv=pc.ckv_pages.to(dev), kpe=pc.kpe_pages.to(dev),
                         bt=bt, sl=sl, ws=ws, out=torch.empty(rows, H, 128, dtype=torch.bfloat16, device=dev)))

    def step(i):
        s = sets[i % 2]
        b.typhoon_mla_decode_tree(s["levels"], s["q_nope"], s["q_pe"], s["ckv"], s["kpe"], pc.page_size, s["bt"], s["sl"],
                                  inp.scale, s["out"], s["ws"])

    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    launches = b.typhoon_mla_last_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(device_index) as clocks:
        ev0.record()
        for i in range(K):
            step(i)
        ev1.record()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / K
    # algorithmic work: Table 1's hybrid terms with rows = B * S_q queries (the suffix is stored once per
    # request), every shared prefix read once, plus the once-only reads of q and the weights and the write of out
    sum_ln_rows = int(sets[0]["sl"].clamp(min=0).sum().item())
    prefix_tokens_rows = rows * Ls + (rows * L_ if args.tree else 0)          # (query row, prefix token) pairs
    prefix_tokens = Ls + (G_ * L_ if args.tree else 0)
    flops = H * (640 * prefix_tokens_rows + 2176 * sum_ln_rows + 4 * 65536 * rows)
    bytes_ = (512 * H + 128) * prefix_tokens + 4 * H * 65536 + 1152 * sum(inp.suffix_lens) + 640 * H * rows
    pk = _peaks()
    t_lb = max(flops / (pk["bf16_tflops"] * 1e12), bytes_ / (pk["hbm_gbs"] * 1e9))
    what = (f"S_q={S_q} query tokens per request" if S_q > 1 else "") + \
        (f"root prefix + {G_} groups with {L_} more shared tokens each" if args.tree else "")
    return {"metric": METRIC, "value": rows / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"{cfg.name}: B={B} H={H} Ls={Ls} Ln=[{cfg.suffix_lo},{cfg.suffix_hi}], {what}",
                       "rows": rows, "entry_point": "typhoon_mla_decode_tree",
                       "l2": "2 full input sets used alternately"},
            "clocks": clocks.summary(), "gpu_launches": launches * K,
            "work": {"algorithmic_flops": flops, "algorithmic_bytes": bytes_, "t_lower_bound_ms": t_lb * 1e3,
                     "step_frac_of_combined_roofline": t_lb / (ms * 1e-3), "peak_source": pk["source"]}}


def bench_naive_everywhere(cfg, args, device_index):
    """--naive-suffix: the naive formulation on the shared AND the non-shared part (the paper's naive-only
    curves in Fig. 8): every request's suffix is expanded once into per-head K/V (as a naive KV cache would hold
    it; not part of the step) and attended with the shared-prefix kernel, one launch per request, next to the
    shared prefix's launch; no absorb branch.  Built from typhoon_mla_decode_tree (level 0: the prefix for all
    requests; level 1: one group per request whose "prefix" is that request's suffix).  B <= 255."""
    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    from paper_2509_21081_b200.decoder import TyphoonMLADecoder
    dev = "cuda"
    W, K = max(args.warmup, 3), max(args.steps, 1)
    H, B = cfg.H, cfg.B
    assert B <= 255, "one shared-prefix launch per request: at most 255 requests"
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=False)
    dims = b.make_dims(H)
    w_uk, w_uv = inp.w_uk.to(dev), inp.w_uv.to(dev)
    q_nope, q_pe = inp.q_nope.to(dev), inp.q_pe.to(dev)
    sets = []
    for _ in range(2):
        root = b.typhoon_mla_prepare_shared(dims, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), w_uk, w_uv)
        own = [b.typhoon_mla_prepare_shared(dims, inp.ckv_suffix[r].to(dev), inp.kpe_suffix[r].to(dev), w_uk, w_uv)
               if inp.ckv_suffix[r].shape[0] > 0 else None for r in range(B)]
        levels = [([root], [0, B]), (own, list(range(B + 1)))]
        ws = torch.empty(b.typhoon_mla_tree_workspace_bytes(levels, B, 0, pc.page_size), dtype=torch.uint8, device=dev)
        sets.append(dict(levels=levels, ws=ws, out=torch.empty(B, H, 128, dtype=torch.bfloat16, device=dev)))

    def step(i):
        s = sets[i % 2]
        b.typhoon_mla_decode_tree(s["levels"], q_nope, q_pe, None, None, pc.page_size, None, None, inp.scale, s["out"], s["ws"])

    for i in range(W):
        step(i)
    torch.cuda.synchronize()
    launches = b.typhoon_mla_last_launch_count()
    # same result as the hybrid step (both are the same attention)
    dec = TyphoonMLADecoder(H, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), w_uk, w_uv, inp.scale, B, pc.block_table.shape[1])
    ref = dec.decode(q_nope, q_pe, pc.ckv_pages.to(dev), pc.kpe_pages.to(dev), pc.block_table.to(dev), pc.seq_lens.to(dev),
                     mode=b.MODE_HYBRID).float()
    max_diff = float((sets[0]["out"].float() - ref).abs().max())
    dec.close()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(device_index) as clocks:
        ev0.record()
        for i in range(K):
            step(i)
        ev1.record()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / K
    sum_ln = sum(inp.suffix_lens)
    bytes_naive = (512 * H + 128) * (cfg.Ls + sum_ln) + 640 * H * B     # every cached token's expanded K/V read once
    return {"metric": METRIC, "value": B / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"{_workload_name(cfg)}, naive formulation on prefix and suffixes (one launch per request)",
                       "entry_point": "typhoon_mla_decode_tree", "l2": "2 full input sets used alternately"},
            "clocks": clocks.summary(), "gpu_launches": launches * K,
            "check": {"max_abs_diff_vs_hybrid_step": max_diff},
            "work": {"expanded_cache_bytes_read": bytes_naive}}


def bench_sharded(cfg, args, device_index, rank, world):
    """--shard seq:G / head:G: one rank's share of a step whose context is sharded over G GPUs, by sequence
    (slice of the prefix + the suffixes of the requests the rank owns -> fp32 partial, all-gather, combine of G
    partials) or by head (H / G heads -> all-gather along heads).  Launched on G GPUs (torchrun, world == G) the
    all-gather is NCCL's and inside the timed region; on one GPU the line is rank 0's compute (its partial step
    plus the combine over G partials, the other ranks' partials being stand-in copies) and the exchange is
    reported as bytes and as a modelled time at the pool's measured 770 GB/s per direction, not timed."""
    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    from paper_2509_21081_b200 import sharded as S
    kind, G_ = args.shard.split(":")
    G_ = int(G_)
    assert kind in ("seq", "head") and G_ >= 1 and world in (1, G_)
    dev = "cuda"
    W, K = max(args.warmup, 3), max(args.steps, 1)
    H, B = cfg.H, cfg.B
    inp = I.make_inputs(cfg)
    pc = I.build_pages(inp, poison=False)
    comm = S.TorchDistComm() if world > 1 else None
    Dec = S.SequenceShardedDecoder if kind == "seq" else S.HeadShardedDecoder
    sets = []
    for _ in range(2):
        dec = Dec(rank, G_, H, inp.ckv_shared.to(dev), inp.kpe_shared.to(dev), inp.w_uk.to(dev), inp.w_uv.to(dev),
                  inp.scale, B, pc.block_table.shape[1], comm=comm)
        a = (inp.q_nope.to(dev), inp.q_pe.to(dev), pc.ckv_pages.to(dev), pc.kpe_pages.to(dev), pc.block_table.to(dev),
             pc.seq_lens.to(dev))
        if kind == "head":   # a rank is handed its own heads' queries
            a = (a[0][:, dec.h0:dec.h1].contiguous(), a[1][:, dec.h0:dec.h1].contiguous()) + a[2:]
        sets.append((dec, a))
    mode = {"auto": b.MODE_AUTO, "absorb": b.MODE_ABSORB, "hybrid": b.MODE_HYBRID, "naive": b.MODE_NAIVE}[args.mode]
    if kind == "seq":
        o_parts = torch.zeros(G_, B, H, 128, dtype=torch.float32, device=dev)
        lse_parts = torch.zeros(G_, B, H, dtype=torch.float32, device=dev)
        out = torch.empty(B, H, 128, dtype=torch.bfloat16, device=dev)
    else:
        Hl = H // G_
        out_l = torch.empty(B, Hl, 128, dtype=torch.bfloat16, device=dev)

    def step(i):
        dec, a = sets[i % 2]
        if kind == "seq":
            lens = lens_of[i % 2]
            b.typhoon_mla_decode_partial(dec.shared, a[0], a[1], a[2], a[3], dec.page_size, a[4], lens, dec.scale,
                                         o_parts[rank], lse_parts[rank], dec.workspace, mode=mode)
            step.launches = b.typhoon_mla_last_launch_count() + 1
            if comm is not None:
                torch.distributed.all_gather_into_tensor(o_parts, o_parts[rank].clone())
                torch.distributed.all_gather_into_tensor(lse_parts, lse_parts[rank].clone())
            b.typhoon_mla_combine_partials(o_parts, lse_parts, out)
        else:
            b.typhoon_mla_decode(dec.shared, a[0], a[1], a[2], a[3], dec.page_size, a[4], a[5], dec.scale, out_l,
                                 dec.workspace, mode=mode)
            step.launches = b.typhoon_mla_last_launch_count()
            if comm is not None:
                comm.all_gather(out_l)
    lens_of = [S.local_seq_lens(a[5], rank, G_) for _, a in sets]

    for i in range(W):
        step(i)
    if kind == "seq" and comm is None:   # stand-ins for the other ranks' partials
        for r in range(1, G_):
            o_parts[r].copy_(o_parts[0]); lse_parts[r].copy_(lse_parts[0])
    torch.cuda.synchronize()
    if comm is not None:
        torch.distributed.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(device_index) as clocks:
        ev0.record()
        for i in range(K):
            step(i)
        ev1.record()
        torch.cuda.synchronize()
    ms = max_over_ranks(ev0.elapsed_time(ev1) / K, world, "cuda") if world > 1 else ev0.elapsed_time(ev1) / K
    xbytes = (G_ - 1) * B * H * 129 * 4 if kind == "seq" else (G_ - 1) * B * (H // G_) * 128 * 2   # received per rank
    return {"metric": METRIC, "value": B / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"{_workload_name(cfg)}, context sharded by {'sequence' if kind == 'seq' else 'head'} over {G_} GPUs",
                       "shard": args.shard, "timed": "all ranks with the NCCL all-gather" if world > 1 else
                       "rank 0's compute on one GPU (partial step + combine); exchange not timed",
                       "l2": "2 full input sets used alternately"},
            "clocks": clocks.summary(), "gpu_launches": step.launches * K,
            "exchange": {"bytes_received_per_rank": xbytes, "modelled_us_at_770_GBps": xbytes / 770e9 * 1e6}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg1", choices=["cfg0", "cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--mode", default="auto", choices=["auto", "absorb", "hybrid", "naive"])
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (config 4 sweep)")
    ap.add_argument("--sweep", action="store_true", help="config 4 fan-out sweep over batch sizes and modes")
    ap.add_argument("--ref-heads", type=int, default=64, help="heads the CPU checker is timed on (scaled up)")
    ap.add_argument("--sq", type=int, default=1, help="extension: query tokens per request (rows = B * S_q)")
    ap.add_argument("--tree", default="", help="extension: G:L = G request groups with L more shared prefix tokens each")
    ap.add_argument("--naive-suffix", action="store_true", help="extension: naive formulation on the suffixes too (Fig. 8's naive-only curves)")
    ap.add_argument("--shard", default="", help="extension: seq:G or head:G = one rank's share of a context sharded over G GPUs")
    ap.add_argument("--stages", action="store_true", help="also time every kernel of the step alone (implied by --sweep)")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--min-region-ms", type=float, default=MIN_REGION_MS,
                    help="device time every timed region is repeated up to (0: each region once, e.g. under a profiler)")
    ap.add_argument("--fp8-shared", action="store_true",
                    help="extension: expanded shared-prefix K/V stored as E4M3 codes (typhoon_mla_prepare_shared_fp8)")
    ap.add_argument("--no-extra", action="store_true", help="headline configuration only (skip the other configurations' short lines)")
    args = ap.parse_args()
    globals()["MIN_REGION_MS"] = max(args.min_region_ms, 0.0)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2509_21081_b200 import binding as b
    from paper_2509_21081_b200 import inputs as I
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local))
    mode = {"auto": b.MODE_AUTO, "absorb": b.MODE_ABSORB, "hybrid": b.MODE_HYBRID, "naive": b.MODE_NAIVE}[args.mode]

    if args.naive_suffix:
        if world > 1:
            raise SystemExit("--naive-suffix is a single-GPU measurement")
        cfg = I.CONFIGS[args.config]
        if args.batch:
            cfg = cfg.with_batch(args.batch)
        print(json.dumps(bench_naive_everywhere(cfg, args, local)), flush=True)
    elif args.shard:
        cfg = I.CONFIGS[args.config]
        if args.batch:
            cfg = cfg.with_batch(args.batch)
        line = bench_sharded(cfg, args, local, rank, world)
        if rank == 0:
            print(json.dumps(line), flush=True)
    elif args.sq > 1 or args.tree:
        if world > 1:
            raise SystemExit("--sq / --tree are single-GPU measurements")
        cfg = I.CONFIGS[args.config]
        if args.batch:
            cfg = cfg.with_batch(args.batch)
        print(json.dumps(bench_extension(cfg, args, local)), flush=True)
    elif args.sweep:
        args.stages = True
        base = I.CONFIGS["cfg4"]
        for B in I.CFG4_BATCHES:
            for m in (b.MODE_ABSORB, b.MODE_HYBRID, b.MODE_AUTO):
                line = bench_config(base.with_batch(B), args, m, rank, world, local, with_cpu=False, with_e2e=False)
                if rank == 0:
                    print(json.dumps(line), flush=True)
    else:
        cfg = I.CONFIGS[args.config]
        if args.batch:
            cfg = cfg.with_batch(args.batch)
        line = bench_config(cfg, args, mode, rank, world, local, with_cpu=not args.no_cpu,
                            with_e2e=not args.no_e2e, fp8=args.fp8_shared)
        if args.config == "cfg1" and not args.batch and args.mode == "auto" and not args.no_extra and not args.fp8_shared:
            line["extra_configs"] = bench_extra_configs(args, rank, world, local)
            # the headline workload once more with the expanded cache in 8 bits (an extension: not the headline's precision)
            ln = bench_config(cfg, args, mode, rank, world, local, with_cpu=False, with_e2e=False, max_steps=20, fp8=True)
            r = ln["roofline"]
            line["fp8_shared_cache"] = {
                "workload": ln["config"]["workload"], "storage": ln["dtype"], "mode": ln["run"]["mode"], "value": ln["value"],
                "ms_per_step": ln["ms_per_step"], "steps": ln["steps"], "timed_regions": ln["timed_regions"],
                "dominant_kernel": r["kernel"], "bound": r["bound"], "frac": r["frac"], "frac_alone": r["frac_alone"],
                "kernel_ms": r["kernel_ms"], "kernel_ms_alone": r["kernel_ms_alone"], "algorithmic_bytes": r["algorithmic_bytes"],
                "step_frac_of_combined_roofline": r["step_frac_of_combined_roofline"]}
        if rank == 0:
            print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
