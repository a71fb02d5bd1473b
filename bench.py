#!/usr/bin/env python
"""Benchmark of the MSD hot path on B200.

Headline workload: the W8A16 MSD GEMM decode sweep - M in {1,2,4,8,16,32,64,128} tokens against INT8 per-channel
weights of shape [14336,4096] (MLP up/gate) and [4096,14336] (MLP down), BF16 output.  One *step* is one pass over the
whole sweep (16 msd_gemm_w8a16 calls = 16 decomposition + 16 GEMM kernels).  Eight distinct weight buffers per shape
are rotated so that every call streams weights that are not in L2 (one step touches 940 MB).

The printed JSON line follows the repository's bench contract: `value` is the whole-job weight-streaming rate
(algorithmic bytes / device time) with inputs resident in HBM, `e2e` the same metric through the host-buffer entry
point, `roofline` the achieved fraction of the measured HBM copy bandwidth, `cpu_baseline` the CPU oracle timed on a
bounded sample.  `configs` carries every workload of the headline metric on its own (smallest W8A16 case, the sweep
per call, the W4A16 prefill GEMM, GQA and MLA decode attention), each with a roofline block; `extras` the comparison
arms and the mixture-of-experts calls.  `--impl reference` times the CPU oracle alone.  `--gpus N` (N > 1) starts N
ranks itself (one per GPU, replicas of the sweep) unless a launcher already did.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

M_SWEEP = [1, 2, 4, 8, 16, 32, 64, 128]
SHAPES = [(14336, 4096), (4096, 14336)]          # (N, K)
NBUF = 8
METRIC = "msd_w8a16_decode_gemm_weight_hbm_gbps"
UNIT = "GB/s"
NOMINAL = {"int8_pops": 4.5, "fp4_pflops": 9.0}    # dense datasheet figures, quoted beside the measured ones


def algorithmic_bytes(M, N, K, out_bytes=2):
    """Bytes MSD itself must move for one call: INT8 weight once, BF16 activations, weight scales, the output."""
    return N * K + 2 * M * K + 4 * N + out_bytes * M * N


def executed_ops(M, N, K):
    """INT8 multiply-accumulates executed by the stacked GEMM, counted as 2 ops each: 2 * (2M) * N * K."""
    return 2 * (2 * M) * N * K


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run (every 200 ms)."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.samples.append((time.time(), parts))

    def summary(self, t0=None, t1=None):
        sm, mx, reasons = [], [], set()
        for (ts, p) in list(self.samples):
            if t0 is not None and not (t0 <= ts <= t1):
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for n, v in zip(self.NAMES, p[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        return self.summary()


# ---- synthetic inputs on the device, with the recipes the parity tests use on the host ------------------------------
def gen_activations(torch, g, M, K, device):
    """N(0,1) with floor(K/100) seeded channels scaled x50, rounded to BF16."""
    x = torch.randn((M, K), generator=g, device=device, dtype=torch.float32)
    perm = torch.randperm(K, generator=g, device=device)[:K // 100]
    x[:, perm] *= 50.0
    return x.to(torch.bfloat16).contiguous()


def gen_w8(torch, g, N, K, device):
    """N(0,0.02) weights -> INT8 per output channel: scale = rowmax/127, round-half-to-even, +-127."""
    w = torch.randn((N, K), generator=g, device=device, dtype=torch.float32) * 0.02
    s = w.abs().amax(dim=1) / 127.0
    q = torch.clamp(torch.round(w / s[:, None]), -127, 127).to(torch.int8)
    return q.contiguous(), s.contiguous()


def gen_w4(torch, g, N, K, device):
    """N(0,0.02) weights -> MXFP4: E2M1 values, one E8M0 scale 2^(floor(log2 blockmax) - 2) per 32 K elements."""
    q = torch.empty((N, K // 2), dtype=torch.uint8, device=device)
    e = torch.empty((N, K // 32), dtype=torch.uint8, device=device)
    mids = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], device=device)
    rows = max(1, (1 << 24) // K)
    for r0 in range(0, N, rows):
        w = torch.randn((min(rows, N - r0), K), generator=g, device=device, dtype=torch.float32) * 0.02
        blk = w.view(w.shape[0], K // 32, 32)
        bmax = blk.abs().amax(dim=2).clamp_min(2.0 ** -120)
        ex = torch.floor(torch.log2(bmax)) - 2.0
        v = blk / torch.exp2(ex)[:, :, None]
        code = torch.bucketize(v.abs().clamp_max(6.0), mids).to(torch.uint8) | ((v < 0).to(torch.uint8) << 3)
        code = code.view(w.shape[0], K // 2, 2)
        q[r0:r0 + w.shape[0]] = code[:, :, 0] | (code[:, :, 1] << 4)
        e[r0:r0 + w.shape[0]] = (ex + 127.0).clamp(0, 254).to(torch.uint8)
    return q, e


def gen_kv(torch, g, T, H, D, device):
    """N(0,1) rounded to BF16, then INT8 with one symmetric scale per token per head."""
    k = torch.empty((T, H, D), dtype=torch.int8, device=device)
    s = torch.empty((T, H), dtype=torch.float32, device=device)
    rows = max(1, (1 << 25) // (H * D))
    for t0 in range(0, T, rows):
        x = torch.randn((min(rows, T - t0), H, D), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16).float()
        sc = x.abs().amax(dim=2) / 127.0
        k[t0:t0 + x.shape[0]] = torch.clamp(torch.round(x / sc.clamp_min(1e-30)[:, :, None]), -127, 127).to(torch.int8)
        s[t0:t0 + x.shape[0]] = sc
    return k, s


def make_inputs(torch, device, seed):
    """The sweep's inputs: NBUF weight buffers per shape, one activation matrix per M."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    data = {}
    for (N, K) in SHAPES:
        ws = [gen_w8(torch, g, N, K, device) for _ in range(NBUF)]
        xs = {M: gen_activations(torch, g, M, K, device) for M in M_SWEEP}
        data[(N, K)] = (ws, xs)
    return data


def roofline_block(bound, achieved, peak, unit, peak_kind, **extra):
    blk = {"bound": bound, "achieved": round(achieved, 2), "peak": peak, "unit": unit, "frac": round(achieved / peak, 4),
           "peak_kind": peak_kind}
    blk.update(extra)
    return blk


def run_gpu(args):
    import torch
    from paper_2605_13915_b200 import binding
    from paper_2605_13915_b200.ranks import Ranks

    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the MSD path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    ranks = Ranks("nccl", device)        # replicas only: barrier, MAX of the times, no data-path collective
    world, rank = ranks.world, ranks.rank
    binding.lib()
    peaks, peak_kind = load_peaks()

    data = make_inputs(torch, device, seed=1234 + rank)
    calls = []          # (M, N, K, x, w, s, y, workspace)
    i = 0
    for (N, K) in SHAPES:
        ws_list, xs = data[(N, K)]
        for M in M_SWEEP:
            w, s = ws_list[i % NBUF]
            i += 1
            y = torch.empty((M, N), dtype=torch.bfloat16, device=device)
            wsp = binding.workspace(binding.gemm_w8a16_workspace_bytes(M, N, K), device)
            calls.append((M, N, K, xs[M], w, s, y, wsp))
    step_bytes = sum(algorithmic_bytes(M, N, K) for (M, N, K, *_r) in calls)
    step_ops = sum(executed_ops(M, N, K) for (M, N, K, *_r) in calls)

    def step():
        for (M, N, K, x, w, s, y, wsp) in calls:
            binding.gemm_w8a16(x, w, s, ws=wsp, out=y)

    stream = torch.cuda.Stream(device=device)

    def capture(fn):
        with torch.cuda.stream(stream):
            fn()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                fn()
        return g

    graph = capture(step)

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    def timed(replay, steps, warmup, all_ranks=False):
        """Device time of `steps` replays in ms.  all_ranks: barrier on both sides and the MAX over ranks (the
        headline and end-to-end regions, which every rank runs); otherwise this rank alone (rank 0's breakdown)."""
        sync = barrier if all_ranks else torch.cuda.synchronize
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                replay()
            stream.synchronize()
            sync()
            e0 = torch.cuda.Event(enable_timing=True)
            e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(steps):
                replay()
            e1.record(stream)
            stream.synchronize()
            sync()
            ms = e0.elapsed_time(e1)
        return ranks.max_over_ranks(ms) if all_ranks else ms

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
    ms = timed(graph.replay, args.steps, args.warmup, all_ranks=True)
    binding.last_device_status()

    # ---- the same step with its 16 independent calls spread over four streams (reported beside the headline, which
    # keeps them in one stream as a single client of the library would issue them) ----
    lanes = [torch.cuda.Stream(device=device) for _ in range(4)]

    def step_overlapped():
        cur = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(cur)
        for st in lanes:
            st.wait_event(fork)
        for i, (M, N, K, x, w, s, y, wsp) in enumerate(calls):
            with torch.cuda.stream(lanes[i % len(lanes)]):
                binding.gemm_w8a16(x, w, s, ws=wsp, out=y)
        for st in lanes:
            join = torch.cuda.Event()
            join.record(st)
            cur.wait_event(join)

    ms_overlapped = timed(capture(step_overlapped).replay, args.steps, args.warmup, all_ranks=True)
    binding.last_device_status()

    # ---- end to end: activations and results in pinned host memory, copies inside the timed region ----
    e2e_calls = []
    for (M, N, K, x, w, s, y, wsp) in calls:
        xh = x.cpu().pin_memory()
        yh = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
        wsh = binding.workspace(binding.gemm_w8a16_host_workspace_bytes(M, N, K), device)
        e2e_calls.append((xh, w, s, yh, wsh))

    # The calls of a step are independent (own buffers, own workspace), so they are dealt round robin to eight streams: the
    # host->device copy of one call and the device->host copy of another overlap the GEMM of a third, as a serving
    # loop that double-buffers its requests would run them.  Fork and join are inside the captured step.
    side = [torch.cuda.Stream(device=device) for _ in range(8)]

    def e2e_step():
        cur = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(cur)
        for st in side:
            st.wait_event(fork)
        # largest activation matrices first: their copies (up to 3.7 MB each way) start at once, the small calls fill in
        order = sorted(range(len(e2e_calls)), key=lambda i: -e2e_calls[i][0].numel())
        for j, i in enumerate(order):
            xh, w, s, yh, wsh = e2e_calls[i]
            with torch.cuda.stream(side[j % len(side)]):
                binding.gemm_w8a16_host(xh, w, s, yh, wsh)
        for st in side:
            join = torch.cuda.Event()
            join.record(st)
            cur.wait_event(join)

    e2e_graph = capture(e2e_step)
    e2e_steps = max(1, args.steps // 2)
    ms_e2e = timed(e2e_graph.replay, e2e_steps, args.warmup, all_ranks=True)
    binding.last_device_status()
    h2d = sum(M * K * 2 for (M, N, K, *_r) in calls)
    d2h = sum(M * N * 2 for (M, N, K, *_r) in calls)
    clocks = sampler.summary() if sampler else None

    def timed_clocked(replay, steps, warmup):
        """timed() plus the SM clock seen by nvidia-smi during that region (None when no sample fell inside it)."""
        t0 = time.time()
        ms_ = timed(replay, steps, warmup)
        t1 = time.time()
        c = {"sm_mhz": None, "reasons": []}
        if sampler:
            c = sampler.summary(t0, t1)
            if c["sm_mhz"] is None:          # a region shorter than the sampling period: the samples just around it
                c = sampler.summary(t0 - 0.3, t1 + 0.3)
        return ms_, c

    detail = rank == 0 and world == 1 and not args.no_breakdown     # single-GPU runs only: the scaling runs stay short
    configs, extras = {}, {}
    if detail:
        # ---- per-call breakdown of the sweep (one graph per call, outside the headline region) ----
        per_call = []
        for (M, N, K, x, w, s, y, wsp) in calls:
            ws_list = data[(N, K)][0]

            def one(M=M, N=N, K=K, x=x, y=y, wsp=wsp, ws_list=ws_list):
                for (wq, sc) in ws_list:
                    binding.gemm_w8a16(x, wq, sc, ws=wsp, out=y)
            t = timed(capture(one).replay, 20, 3) / (20 * NBUF) * 1e3
            gbps = algorithmic_bytes(M, N, K) / t / 1e3
            per_call.append({"M": M, "N": N, "K": K, "us": round(t, 2), "gbps": round(gbps, 1),
                             "frac": round(gbps / peaks["hbm_gbs"], 3), "tops": round(executed_ops(M, N, K) / t / 1e6, 2)})
        configs["c1_w8a16_decode_sweep"] = {
            "workload": "M in {1..128} x {[14336,4096],[4096,14336]}, BF16 out; one call at a time, 8 weight buffers rotated",
            "per_call": per_call,
            "roofline": roofline_block("hbm", step_bytes / (ms / args.steps * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s",
                                       f"of {peak_kind}", note="the headline: all 16 calls back to back in one stream")}
        measure_configs(torch, binding, device, capture, timed_clocked, peaks, peak_kind, configs, extras,
                        cpu=not args.no_cpu_baseline)
    if sampler:
        sampler.stop()

    if rank != 0:
        ranks.close()
        return

    ms_per_step = ms / args.steps
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9
    e2e_value = world * step_bytes / (ms_e2e / e2e_steps * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 5), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "configs[1]: W8A16 MSD GEMM decode sweep, M in {1..128} x {[14336,4096],[4096,14336]}, BF16 out",
                   "calls_per_step": len(calls), "l2": f"{NBUF} weight buffers per shape rotated; one step streams "
                   f"{step_bytes / 1e6:.0f} MB (> 126 MB L2)", "launch": "CUDA graph of one step"},
        "tops": round(world * step_ops / (ms_per_step * 1e-3) / 1e12, 2),
        "overlapped": {"value": round(world * step_bytes / (ms_overlapped / args.steps * 1e-3) / 1e9, 1), "unit": UNIT,
                       "ms_per_step": round(ms_overlapped / args.steps, 5),
                       "note": "the step's 16 independent calls on four streams inside one graph: a call's prologue and the "
                               "decomposition of the next overlap the tail of the previous one"},
        "clocks": clocks,
        "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "api": "msd_gemm_w8a16_host (pinned host activations and outputs, weights resident; the step's 16 independent calls dealt round robin to eight streams)"},
        "gpu_launches": 2 * len(calls) * args.steps,
        "roofline": roofline_block("hbm", value / world, peaks["hbm_gbs"], "GB/s", f"of {peak_kind}",
                                   bytes_per_launch=step_bytes // len(calls),
                                   us_per_launch=round(ms_per_step * 1e3 / len(calls), 3), traffic=None,
                                   kernel="gemm_w8a16_kernel (+ decompose_int8_kernel overlapped by PDL)",
                                   note="achieved = algorithmic bytes of the sweep / device time of the timed region"),
        "configs": configs,
        "extras": extras,
    }
    # DRAM traffic of one launch from the committed ncu capture, as long as the kernel's source is the one it was taken from
    traffic_file = os.path.join(ROOT, "profiles", "gemm_w8a16_traffic.json")
    if os.path.exists(traffic_file):
        with open(traffic_file) as f:
            tr = json.load(f)
        src = os.path.join(ROOT, "paper_2605_13915_b200", "csrc", "gemm_w8a16.cu")
        sha = hashlib.sha1(open(src, "rb").read()).hexdigest() if os.path.exists(src) else None
        if tr.get("source_sha1") == sha:
            out["roofline"]["traffic"] = tr["dram_bytes"]
            out["roofline"]["traffic_of"] = tr["launch"] + f"; algorithmic bytes of that launch {tr['algorithmic_bytes']}"
        else:
            out["roofline"]["traffic_of"] = "not reported: the kernel source changed since the committed ncu capture"
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(check=(binding, data, torch))
    print(json.dumps(out), flush=True)
    ranks.close()


def measure_configs(torch, binding, device, capture, timed_clocked, peaks, peak_kind, configs, extras, cpu=True):
    """Every other workload of the headline metric, each timed on its own (graphs of a few calls, device time, inputs
    drawn on the device with the recipes of the parity tests), and the comparison arms."""
    hbm = peaks["hbm_gbs"]
    bf16 = peaks["bf16_tflops"]

    def per_call_us(fn, reps=4, steps=5):
        def many():
            for _ in range(reps):
                fn()
        ms, clk = timed_clocked(capture(many).replay, steps, 3)
        return ms / (steps * reps) * 1e3, clk

    def gen(seed):
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        return g

    # ---- c0: W8A16, M = 16, K = N = 4096, FP32 output, eight weight buffers rotated ----
    g = gen(0)
    M, N, K = 16, 4096, 4096
    x = gen_activations(torch, g, M, K, device)
    wbuf = [gen_w8(torch, g, N, K, device) for _ in range(NBUF)]
    y = torch.empty((M, N), dtype=torch.float32, device=device)
    wsp = binding.workspace(binding.gemm_w8a16_workspace_bytes(M, N, K), device)
    it = [0]

    def f_c0():
        it[0] += 1
        wq, sc = wbuf[it[0] % NBUF]
        binding.gemm_w8a16(x, wq, sc, ws=wsp, out=y)
    t, clk = per_call_us(f_c0, reps=2 * NBUF, steps=10)
    b0 = algorithmic_bytes(M, N, K, out_bytes=4)
    c0 = {"workload": "W8A16 MSD GEMM M=16 K=N=4096, FP32 out, seed 0, 8 weight buffers rotated", "us": round(t, 2),
          "roofline": roofline_block("hbm", b0 / t / 1e3, hbm, "GB/s", f"of {peak_kind}", algorithmic_bytes=b0), "sm_mhz": clk["sm_mhz"]}
    if cpu:
        import oracle
        from paper_2605_13915_b200 import inputs
        c = inputs.gemm_w8_case(16, 4096, 4096, seed=0)
        n = oracle.max_threads()
        res = {}
        for threads in (n, 1):
            oracle.set_threads(threads)
            t0 = time.perf_counter()
            oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64")
            res[threads] = time.perf_counter() - t0
        oracle.set_threads(n)
        c0["cpu_oracle"] = {"seconds_all_cores": round(res[n], 3), "cores": n, "seconds_one_thread": round(res[1], 3)}
    configs["c0_w8a16_m16_4096"] = c0
    del wbuf, x, y, wsp

    # ---- c2: W4A16 prefill, M = 4096, N = K = 8192; seeds 0, 1, 2, the median reported ----
    M, N, K = 4096, 8192, 8192
    runs = []
    for seed in (0, 1, 2):
        g = gen(seed)
        x = gen_activations(torch, g, M, K, device)
        w4, e4 = gen_w4(torch, g, N, K, device)
        wsp = binding.workspace(binding.gemm_w4a16_workspace_bytes(M, N, K), device)
        y = torch.empty((M, N), dtype=torch.bfloat16, device=device)
        prep = binding.prepare_w4a16_scales(e4)      # once per weight, outside the timed calls
        t, clk = per_call_us(lambda: binding.gemm_w4a16(x, w4, None, ws=wsp, out=y, prepared=prep), reps=4, steps=25)
        runs.append((t, clk["sm_mhz"], clk["reasons"]))
    # the same call with row-major scales (relayout inside every call), once, after the timed seeds: a longer FP4 load
    # between the seeds would lower the clock under the power cap for the seeds that follow
    t_rowmajor, _ = per_call_us(lambda: binding.gemm_w4a16(x, w4, e4, ws=wsp, out=y), reps=2, steps=25)
    t, mhz, reasons = sorted(runs)[1]
    pf = 4.0 * M * N * K / t / 1e9
    configs["c2_w4a16_prefill_m4096_8192"] = {
        "workload": "W4A16 MSD GEMM M=4096 N=K=8192, BF16 out; 100 calls per seed, median of seeds 0,1,2; weight scales "
                    "prepared once (msd_prepare_w4a16_scales), msd_gemm_w4a16_prepared timed",
        "us": round(t, 1), "us_per_seed": [round(r[0], 1) for r in runs], "sm_mhz": mhz, "clock_reasons": reasons,
        "us_with_row_major_scales": round(t_rowmajor, 1),
        "executed_fp4_pflops": round(pf, 3), "effective_pflops": round(pf / 2, 3),
        "roofline": roofline_block("tensor", pf, NOMINAL["fp4_pflops"], "PFLOP/s", "nominal dense FP4",
                                   frac_of_4x_measured_bf16=round(pf * 1e3 / (4 * bf16), 3),
                                   peak_4x_measured_bf16=round(4 * bf16 / 1e3, 3))}
    # comparison: the weights expanded to BF16 (torch ops, several passes) and a library BF16 GEMM
    lut = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6, -0., -.5, -1, -1.5, -2, -3, -4, -6], dtype=torch.bfloat16, device=device)
    wb = torch.empty((N, K), dtype=torch.bfloat16, device=device)

    def w4_dequant():
        sc = torch.exp2(e4.to(torch.float32) - 127.0).to(torch.bfloat16).repeat_interleave(32, dim=1)
        wv = wb.view(N, K // 2, 2)
        wv[:, :, 0] = lut[(w4 & 15).long()]
        wv[:, :, 1] = lut[(w4 >> 4).long()]
        wb.mul_(sc)
    t_dq, _ = per_call_us(w4_dequant, reps=1, steps=3)
    t_mm, _ = per_call_us(lambda: torch.matmul(x, wb.t(), out=y), reps=4, steps=10)
    extras["w4a16_prefill_vs_dequant_bf16"] = {
        "msd_us": round(t, 1), "dequant_us": round(t_dq, 1), "library_bf16_gemm_us": round(t_mm, 1),
        "msd_speedup_vs_gemm_alone": round(t_mm / t, 2), "msd_speedup_vs_dequant_plus_gemm": round((t_dq + t_mm) / t, 2),
        "note": "dequant = torch ops (library, several passes over the weights); GEMM = torch.matmul BF16 (library)"}
    del x, w4, e4, y, wsp, wb, lut

    # ---- c3 GQA and c4 MLA decode attention; seeds 0, 1, 2 ----
    from paper_2605_13915_b200 import inputs as gen_host
    attn_cases = {
        "c3_attn_gqa_b32_h32_kv8_d128": (32, 32, 8, 128, 128, False, "batch 32, 32 query / 8 KV heads, d 128, lengths U[2048,8192]"),
        "c4_attn_mla_b64_h64_d576": (64, 64, 1, 576, 512, True, "batch 64, 64 heads on one latent head of 576 (V = first 512), length 16384")}
    for name, (B, Hq, Hkv, D, Dv, alias, what) in attn_cases.items():
        runs, keep = [], []
        for seed in (0, 1, 2):
            g = gen(seed)
            L = gen_host.seqlens_uniform(B, 2048, 8192, seed=seed) if not alias else np.full(B, 16384, np.int32)
            T = int(np.sum(L))
            cu = torch.zeros(B + 1, dtype=torch.int32)
            cu[1:] = torch.from_numpy(np.cumsum(L).astype(np.int32))
            cu = cu.to(device)
            q = torch.randn((B, Hq, D), generator=g, device=device).to(torch.bfloat16)
            k, ks = gen_kv(torch, g, T, Hkv, D, device)
            v, vs = (None, None) if alias else gen_kv(torch, g, T, Hkv, Dv, device)
            wsp = binding.workspace(binding.attn_decode_int8kv_workspace_bytes(B, Hq, Hkv, D, Dv, int(L.max())), device)
            o = torch.empty((B, Hq, Dv), dtype=torch.bfloat16, device=device)
            t, clk = per_call_us(lambda: binding.attn_decode_int8kv(q, k, v, ks, vs, cu, int(L.max()), D ** -0.5, dv=Dv, ws=wsp, out=o),
                                 reps=4, steps=10)
            byts = T * Hkv * ((D + 4) + (0 if alias else Dv + 4))
            runs.append((byts / t / 1e3, t, B / t * 1e6, clk["sm_mhz"], byts))
            # (the three seeds' caches stay allocated until the config is done: a freed cache's block, handed out again at
            # another offset, moved the MLA timing by 5 % - 309 vs 325 us - with the data unchanged)
            keep.append((k, ks, v, vs, q, o, wsp))
        gbps, t, tps, mhz, med_bytes = sorted(runs)[1]
        configs[name] = {"workload": "INT8-KV decode attention: " + what + "; median of seeds 0,1,2", "us": round(t, 1),
                         "tokens_per_s": round(tps), "kv_bytes": med_bytes, "us_per_seed": [round(r[1], 1) for r in runs], "sm_mhz": mhz,
                         "roofline": roofline_block("hbm", gbps, hbm, "GB/s", f"of {peak_kind}")}
        if not alias:
            # comparison arm (seed 2's data): our cache-expansion kernel (INT8 -> BF16 in memory), then BF16 attention on
            # the expanded cache - our own BF16-KV decode kernel, and a library one (torch SDPA, one call per sequence)
            t_msd = runs[2][1]
            kb = torch.empty((T, Hkv, D), dtype=torch.bfloat16, device=device)
            vb = torch.empty((T, Hkv, Dv), dtype=torch.bfloat16, device=device)
            t_deq, _ = per_call_us(lambda: (binding.kv_dequant_bf16(k, ks, out=kb), binding.kv_dequant_bf16(v, vs, out=vb)), reps=2)
            wsb = binding.workspace(int(binding.lib().msd_attn_decode_bf16kv_workspace_bytes(B, Hq, Hkv, D, Dv, int(L.max()))), device)
            ob = torch.empty((B, Hq, Dv), dtype=torch.bfloat16, device=device)
            t_bf, _ = per_call_us(lambda: binding.attn_decode_bf16kv(q, kb, vb, cu, int(L.max()), D ** -0.5, ws=wsb, out=ob), reps=4)
            cu_h = cu.cpu().tolist()
            sdpa = torch.nn.functional.scaled_dot_product_attention

            def f_lib():
                for b in range(B):
                    t0, t1 = cu_h[b], cu_h[b + 1]
                    sdpa(q[b][None, :, None, :], kb[t0:t1].permute(1, 0, 2)[None], vb[t0:t1].permute(1, 0, 2)[None],
                         scale=D ** -0.5, enable_gqa=True)
            try:
                t_lib, _ = per_call_us(f_lib, reps=1)
            except Exception as e:  # the library arm is context, never the product
                t_lib = None
                lib_err = str(e)[:120]
            bf_gbps = 2 * T * Hkv * (D + Dv) / t_bf / 1e3
            extras["attn_gqa_vs_dequant_bf16"] = {
                "msd_us": round(t_msd, 1), "dequant_us": round(t_deq, 1), "bf16_attention_kernel_us": round(t_bf, 1),
                "total_us": round(t_deq + t_bf, 1), "msd_speedup": round((t_deq + t_bf) / t_msd, 2),
                "msd_speedup_vs_bf16_attention_alone": round(t_bf / t_msd, 2),
                "bf16_attention_kernel_roofline": roofline_block("hbm", bf_gbps, hbm, "GB/s", f"of {peak_kind}"),
                "traffic_floor_us": round(5 * T * Hkv * (D + Dv) / hbm / 1e3, 1),
                "note": "dequant = msd_kv_dequant_bf16, attention = msd_attn_decode_bf16kv (both ours; the second alone is what a "
                        "BF16 cache would cost: twice the bytes); traffic_floor = 5 bytes per cache element at the measured HBM peak"}
            if t_lib is not None:
                extras["attn_gqa_vs_dequant_bf16"]["library_bf16_attention_us"] = round(t_lib, 1)
                extras["attn_gqa_vs_dequant_bf16"]["msd_speedup_vs_dequant_plus_library"] = round((t_deq + t_lib) / t_msd, 2)
            else:
                extras["attn_gqa_vs_dequant_bf16"]["library_error"] = lib_err
            del kb, vb, wsb, ob
        del k, ks, v, vs, q, o, wsp, keep

    # ---- extras: the comparison GEMM the method replaces, at M = 16 of both sweep shapes ----
    g = gen(7)
    base = {}
    for (N, K) in SHAPES:
        x = gen_activations(torch, g, 16, K, device)
        ws = [gen_w8(torch, g, N, K, device) for _ in range(4)]
        wsp_b = binding.workspace(binding.gemm_dequant_bf16_workspace_bytes(16, N, K), device)
        wsp_m = binding.workspace(binding.gemm_w8a16_workspace_bytes(16, N, K), device)
        y = torch.empty((16, N), dtype=torch.bfloat16, device=device)
        it = [0]

        def f_base():
            it[0] += 1
            wq, sc = ws[it[0] % 4]
            wp, wb_ = binding._ws_ptr(wsp_b)
            binding._check(binding.lib().msd_gemm_dequant_bf16(x.data_ptr(), wq.data_ptr(), sc.data_ptr(), 16, N, K,
                                                               y.data_ptr(), 0, wp, wb_, torch.cuda.current_stream().cuda_stream), "dequant")

        def f_msd():
            it[0] += 1
            wq, sc = ws[it[0] % 4]
            binding.gemm_w8a16(x, wq, sc, ws=wsp_m, out=y)
        wsp_f = binding.workspace(max(1024, int(binding.lib().msd_gemm_w8a16_fused_dequant_workspace_bytes(16, N, K))), device)

        def f_fused():
            it[0] += 1
            wq, sc = ws[it[0] % 4]
            binding.gemm_w8a16_fused_dequant(x, wq, sc, ws=wsp_f, out=y)
        (tb, _), (tm, _), (tf, _) = per_call_us(f_base), per_call_us(f_msd), per_call_us(f_fused)
        base[f"M16_N{N}_K{K}"] = {"dequant_bf16_us": round(tb, 2), "fused_dequant_us": round(tf, 2), "msd_us": round(tm, 2),
                                  "speedup": round(tb / tm, 2), "speedup_vs_fused_dequant": round(tf / tm, 2)}
        del ws
    base["note"] = ("dequant_bf16 = msd_gemm_dequant_bf16 (weights written back as BF16, then a BF16 GEMM); fused_dequant = "
                    "msd_gemm_w8a16_fused_dequant (INT8 weights converted to BF16 inside the GEMM, into tensor memory)")
    extras["w8a16_vs_dequant_bf16_kernel"] = base

    # ---- extras: W4A16 at the decode sweep's shapes, M = 16 ----
    w4d = {}
    for (N, K) in SHAPES:
        x = gen_activations(torch, g, 16, K, device)
        wq = [gen_w4(torch, g, N, K, device) for _ in range(4)]
        wprep = [binding.prepare_w4a16_scales(e4) for (_q, e4) in wq]
        wsp = binding.workspace(binding.gemm_w4a16_workspace_bytes(16, N, K), device)
        y = torch.empty((16, N), dtype=torch.bfloat16, device=device)
        it4 = [0]

        def f_w4d():
            it4[0] += 1
            q4, e4 = wq[it4[0] % 4]
            binding.gemm_w4a16(x, q4, e4, ws=wsp, out=y)

        def f_w4d_prep():
            it4[0] += 1
            binding.gemm_w4a16(x, wq[it4[0] % 4][0], None, ws=wsp, out=y, prepared=wprep[it4[0] % 4])
        t_row, _ = per_call_us(f_w4d, reps=8)
        t, _ = per_call_us(f_w4d_prep, reps=8)
        b = N * (K // 2 + K // 32)
        w4d[f"M16_N{N}_K{K}"] = {"us": round(t, 2), "us_with_row_major_scales": round(t_row, 2),
                                 "roofline": roofline_block("hbm", b / t / 1e3, hbm, "GB/s", f"of {peak_kind}")}
        del x, wq, wprep, wsp, y
    extras["w4a16_decode_shapes"] = w4d

    # ---- extras: INT8 tensor-peak point, the W8A16 layer at M = 4096 on both sweep shapes ----
    p8 = {}
    for (N, K) in SHAPES:
        M = 4096
        x = gen_activations(torch, g, M, K, device)
        w8, s8 = gen_w8(torch, g, N, K, device)
        wsp = binding.workspace(binding.gemm_w8a16_workspace_bytes(M, N, K), device)
        y = torch.empty((M, N), dtype=torch.bfloat16, device=device)
        t, clk = per_call_us(lambda: binding.gemm_w8a16(x, w8, s8, ws=wsp, out=y), reps=4, steps=25)
        po = 4.0 * M * N * K / t / 1e9
        entry = {"us": round(t, 1), "sm_mhz": clk["sm_mhz"], "executed_int8_pops": round(po, 3),
                 "roofline": roofline_block("tensor", po, NOMINAL["int8_pops"], "POP/s", "nominal dense INT8",
                                            frac_of_2x_measured_bf16=round(po * 1e3 / (2 * bf16), 3))}
        # the comparison path as this library's own kernels: weights expanded to BF16, then the same pipeline as a BF16 GEMM
        wsb = binding.workspace(binding.gemm_dequant_bf16_workspace_bytes(M, N, K), device)
        tdq, _ = per_call_us(lambda: binding.gemm_dequant_bf16(x, w8, s8, ws=wsb), reps=2)
        entry["comparison_dequant_bf16_kernel"] = {"us": round(tdq, 1), "msd_speedup": round(tdq / t, 2),
                                                   "note": "msd_gemm_dequant_bf16: dequantize kernel + BF16 tcgen05 GEMM (ours)"}
        del wsb
        if (N, K) == SHAPES[0]:
            wb = torch.empty((N, K), dtype=torch.bfloat16, device=device)

            def w8_dequant():
                torch.mul(w8.to(torch.bfloat16), s8.to(torch.bfloat16)[:, None], out=wb)
            t_dq, _ = per_call_us(w8_dequant, reps=1, steps=3)
            t_mm, _ = per_call_us(lambda: torch.matmul(x, wb.t(), out=y))
            entry["comparison_dequant_bf16"] = {
                "dequant_us": round(t_dq, 1), "library_bf16_gemm_us": round(t_mm, 1), "msd_speedup_vs_gemm_alone": round(t_mm / t, 2),
                "msd_speedup_vs_dequant_plus_gemm": round((t_dq + t_mm) / t, 2),
                "note": "dequant = torch ops (library); GEMM = torch.matmul BF16 (library); MSD executes twice the MACs at twice the rate"}
            del wb
        p8[f"M4096_N{N}_K{K}"] = entry
        del x, w8, s8, y, wsp
    extras["w8a16_many_rows"] = p8

    # ---- extras: grouped GEMMs (mixture of experts): 32 experts of [2048, 7168], 16 routed tokens each ----
    E, Ng, Kg, per = 32, 2048, 7168, 16
    xg = gen_activations(torch, g, E * per, Kg, device)
    wg = [torch.stack([gen_w8(torch, g, Ng, Kg, device)[0] for _ in range(E)]) for _ in range(2)]
    sg = torch.rand((E, Ng), generator=g, device=device) * 0.001 + 0.0005
    yg = torch.empty((E * per, Ng), dtype=torch.bfloat16, device=device)
    wsg = binding.workspace(int(binding.lib().msd_grouped_gemm_w8a16_workspace_bytes(E * per, per, E, Ng, Kg)), device)
    ws1 = binding.workspace(binding.gemm_w8a16_workspace_bytes(per, Ng, Kg), device)
    itg = [0]

    def f_grouped():
        itg[0] += 1
        binding.grouped_gemm_w8a16(xg, wg[itg[0] % 2], sg, [per] * E, ws=wsg, out=yg)

    def f_loop():
        itg[0] += 1
        wcur = wg[itg[0] % 2]
        for e in range(E):
            binding.gemm_w8a16(xg[e * per:(e + 1) * per], wcur[e], sg[e], ws=ws1, out=yg[e * per:(e + 1) * per])
    (tg, _), (tl, _) = per_call_us(f_grouped, reps=2), per_call_us(f_loop, reps=1)
    extras["moe_grouped_w8a16_e32_n2048_k7168_16_tokens_per_expert"] = {
        "us": round(tg, 1), "roofline": roofline_block("hbm", E * Ng * Kg / tg / 1e3, hbm, "GB/s", f"of {peak_kind}"),
        "one_call_per_expert_us": round(tl, 1), "speedup": round(tl / tg, 2)}
    del wg, sg, wsg
    w4g = []
    for _ in range(2):
        qs, es = zip(*[gen_w4(torch, g, Ng, Kg, device) for _ in range(E)])
        w4g.append((torch.stack(qs), torch.stack(es)))
    ws4 = binding.workspace(int(binding.lib().msd_grouped_gemm_w4a16_workspace_bytes(E, Ng, Kg)), device)

    def f_grouped4():
        itg[0] += 1
        q4, e4 = w4g[itg[0] % 2]
        binding.grouped_gemm_w4a16(xg, q4, e4, [per] * E, ws=ws4, out=yg)
    w4prep = [binding.prepare_w4a16_scales(e4) for (_q, e4) in w4g]

    def f_grouped4_prep():
        itg[0] += 1
        binding.grouped_gemm_w4a16(xg, w4g[itg[0] % 2][0], None, [per] * E, ws=ws4, out=yg, prepared=w4prep[itg[0] % 2])
    t4_row, _ = per_call_us(f_grouped4)
    t4, _ = per_call_us(f_grouped4_prep)
    b4 = E * Ng * (Kg // 2 + Kg // 32)
    extras["moe_grouped_w4a16_e32_n2048_k7168_16_tokens_per_expert"] = {
        "us": round(t4, 1), "roofline": roofline_block("hbm", b4 / t4 / 1e3, hbm, "GB/s", f"of {peak_kind}"),
        "us_with_row_major_scales": round(t4_row, 1),
        "note": "weight scales prepared once (msd_prepare_w4a16_scales); with row-major scales every call first brings "
                "all experts' scales into the blocked layout"}


def cpu_baseline(check=None):
    """Times the CPU oracle, as it stands, on the whole sweep once (every M, both weight shapes, all N and K) and
    compares the GPU result with it element by element."""
    import oracle
    cores = oracle.max_threads()
    binding, data, torch = check
    tot_bytes, tot_s, parity, worst = 0.0, 0.0, True, 0.0
    for (N, K) in SHAPES:
        wq, sc = data[(N, K)][0][0]
        w_np, s_np = wq.cpu().numpy(), sc.cpu().numpy()
        for M in M_SWEEP:
            x = data[(N, K)][1][M]
            x_np = x.cpu().view(torch.int16).numpy().view(np.uint16)
            t0 = time.perf_counter()
            ref = oracle.gemm_w8a16(x_np, w_np, s_np, "f64")
            tot_s += time.perf_counter() - t0
            tot_bytes += algorithmic_bytes(M, N, K)
            y = binding.gemm_w8a16(x, wq, sc)
            torch.cuda.synchronize()
            got = y.float().cpu().numpy().astype(np.float64)
            err = np.abs(got - ref) - np.abs(ref) * 2.0 ** -8
            rel = float((err / np.linalg.norm(ref, axis=1, keepdims=True)).max())
            worst = max(worst, rel)
            parity = parity and rel <= 1e-3
    return {"value": round(tot_bytes / tot_s / 1e9, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"the whole sweep once (8 values of M x 2 weight shapes, full N and K); {tot_s:.1f} s of CPU time",
            "seconds": round(tot_s, 2), "gpu_matches_oracle": parity, "max_rel_row_err_beyond_bf16_ulp": round(worst, 6)}


def run_reference(args):
    """The CPU oracle as the comparison arm: every step is a bounded sample of the sweep.  Under a multi-rank launch
    rank 0 alone runs and prints; the other ranks exit without work."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle
    from paper_2605_13915_b200 import inputs
    ncols = 512
    cases = [(inputs.gemm_w8_case(16, ncols, K, seed=0), K) for (_N, K) in SHAPES]
    step_bytes = sum(algorithmic_bytes(16, ncols, K) for (_c, K) in cases)

    def step():
        for (c, _K) in cases:
            oracle.gemm_w8a16(c.x, c.w, c.w_scale, "f64")

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = step_bytes * args.steps / dt / 1e9
    sample = f"per step: M=16 on both weight shapes, {ncols} output channels each (full K)"
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": world,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 3),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
           "config": {"workload": "configs[1] sample: " + sample},
           "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "kind": "oracle", "cores": oracle.max_threads(),
                            "sample": sample},
           "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n, argv):
    """--gpus N without a launcher: start N ranks of this script under torch.distributed.run on this node and hand
    their exit code back.  (A launcher that already set WORLD_SIZE is left alone.)"""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.abspath(__file__)] + argv
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="msd", choices=["msd", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    args.warmup = max(args.warmup, 3) if args.impl == "msd" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
