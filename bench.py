#!/usr/bin/env python
"""Benchmark of the libtlin hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload fwd128k|fwd32k|fwd8k|decode]
    python bench.py --impl reference ...        # the CPU oracle, as it stands, on the host cores

One JSON line on stdout (rank 0).  A "step" is one pass of the hot path over one batch of synthetic
input: for a forward workload the plan, the W x N exact-softmax attention with the causal window and
the split merge; for the decode workload one cached single-token step (append + attend + merge).
The headline workload is the N=131072 forward; the N=32768 forward and the cached decode are timed
in the same run and reported under "also" (skip with --only).

`value` is measured with the inputs resident in HBM; `e2e` goes through the host-buffer entry
points, host<->device copies inside the timed region.  With --gpus N > 1 (under torchrun) every rank
runs an independent replica of the same workload on its own GPU: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2508_20407_b200 import synth  # noqa: E402

WORKLOADS = {"fwd128k": "cfg4_vlong", "fwd32k": "cfg3_long", "fwd8k": "cfg2_mid", "decode": "cfg5_decode",
             "restore": "restore_vlong", "inner_self": "inner_self", "inner_gen": "inner_gen",
             "bwd_chunk": "train_chunk", "bwd32k": "cfg3_long", "decode_fp8": "cfg5_decode",
             "nsweep": "cfg3_long", "fwd_seq": "train_seq", "bwd_seq": "train_seq", "inner_batched": "inner_self"}
BACKWARD = ("bwd_chunk", "bwd32k", "bwd_seq")      # legs that time tlin_attn_backward on the named shape
NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 7700.0      # datasheet figures, reported beside the measured peaks
REFERENCE_BUDGET_S = 100.0     # --impl reference: target duration of all its steps together
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None
        self.t0 = self.t1 = None

    def launch(self):
        """Starts nvidia-smi (it needs a moment to come up, so this is called before the warm-up)."""
        if self.proc is not None:
            return
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def start(self):
        """Marks the beginning of the timed region."""
        self.launch()
        self.t0 = time.time()

    def stop(self):
        """Marks the end of the timed region and summarises the samples taken inside it."""
        self.t1 = time.time()
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region"}
        if self.proc is None:
            return out
        time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        import datetime
        rows = []
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 8:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(parts[1]), float(parts[2]), parts[4:8]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if self.t0 - 0.01 <= r[0] <= self.t1 + 0.01]
        if not inside and rows:      # region shorter than the sampling period: fall back to samples since launch (warm-up load)
            inside = rows[-3:]
            out["window"] = "last samples before the end of the timed region"
        if inside:
            reasons = set()
            for r in inside:
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       reasons=sorted(reasons), samples=len(inside))
        return out


# ----------------------------------------------------------------------------- timing helpers
def dist_info():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def barrier(world):
    if world > 1:
        torch.distributed.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    t = torch.tensor([x], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def time_steps(step_fn, steps, warmup, world, device, sampler=None, flush_buf=None):
    """Device time of `steps` calls (CUDA events on the current stream), max over ranks, in ms.

    Without `flush_buf` the calls run back to back between one pair of events (the inputs are larger than
    L2, so nothing survives from one call to the next).  With it, every call is timed by its own pair of
    events and the buffer (larger than L2) is overwritten before each call, outside the timed intervals.
    """
    if sampler:
        sampler.launch()
    for i in range(warmup):
        step_fn(i)
    torch.cuda.synchronize()
    barrier(world)
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    if flush_buf is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            step_fn(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
    else:
        pairs = []
        for i in range(steps):
            flush_buf.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step_fn(warmup + i)
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        ms = sum(a.elapsed_time(b) for a, b in pairs)
    clocks = sampler.stop() if sampler else None
    barrier(world)
    torch.cuda.synchronize()
    return max_over_ranks(ms, world, device), clocks


def sustained_leg(step_fn, ms_step, world, device, rank, seconds=1.2):
    """The same call repeated back to back for about `seconds` inside one pair of events (its own loop, beside the
    timed steps), with the SM clock sampled meanwhile: the figure a long-running job sees once the power cap acts."""
    n = max(3, int(seconds * 1e3 / max(ms_step, 1e-3)) + 1)
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    ms, clocks = time_steps(step_fn, n, 3, world, device, sampler)
    return ms / n, n, clocks


L2_BYTES = 126e6

# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, per launch, from one-pass ncu captures of these
# very workloads.  To be set to None whenever the kernel changes.
FWD_TRAFFIC = {"cfg4_vlong": (2191.82e6 + 20.53e6, "ncu, full workload, fwd_tc_kernel<128, 0>"),
               "cfg3_long": (544.79e6 + 10.41e6, "ncu, full workload, fwd_tc_kernel<128, 0>")}
# decode: captured on a smaller cache (B8 H32, 4096 rows: 537.35 MB read + 3.9 MB written for 537.3 MB of cache) and
# scaled by the cached rows of the timed steps; the kernel streams every cached byte once at any size
DECODE_TRAFFIC_RATIO = (537.35 + 3.9) / 537.3
# 8-bit cache: 268.9 MB read + 4.0 MB written for 268.4 MB of codes (B8 H32, 4096 rows), scaled the same way
DECODE_FP8_TRAFFIC_RATIO = (268.9 + 4.0) / 268.4


# ----------------------------------------------------------------------------- the oracle as a timed baseline
def oracle_forward_sample(wl, k_head, v_head, q_head, rows):
    """Last `rows` query rows of one head through the CPU oracle (exactly those rows of the workload)."""
    import oracle
    q = q_head[wl.W - rows:].contiguous().view(1, 1, rows, wl.d)
    t0 = time.perf_counter()
    out, lse = oracle.attn_forward(q, k_head.view(1, 1, wl.N, wl.d), v_head.view(1, 1, wl.N, wl.d), wl.causal_window)
    return time.perf_counter() - t0, out, lse


def cpu_baseline_forward(wl, q_head, k_head, v_head, target_s=12.0):
    import oracle
    cores = oracle.num_threads()
    probe = min(wl.W, max(cores * 4, 8))
    t_probe, _, _ = oracle_forward_sample(wl, k_head, v_head, q_head, probe)
    rows = int(min(wl.W, max(probe, probe * target_s / max(t_probe, 1e-6))))
    rows = max(cores * 4, rows // (cores * 4) * (cores * 4))
    rows = min(rows, wl.W)
    t, out, lse = oracle_forward_sample(wl, k_head, v_head, q_head, rows)
    t_full = t * (wl.B * wl.H * wl.W) / rows
    return dict(value=wl.B * wl.N / t_full, unit="context tokens/s", cores=cores, kind="oracle",
                sample=f"last {rows} of {wl.W} query rows of head (b=0,h=0), all {wl.N} keys: {t:.2f} s, "
                       f"scaled by {wl.B * wl.H * wl.W}/{rows} rows"), (rows, out, lse)


def cpu_baseline_decode(wl, kc_heads, vc_heads, q_new, k_new, v_new, pos, n_heads):
    """One decode step for the first n_heads (b,h) pairs through the CPU oracle."""
    import oracle
    cores = oracle.num_threads()
    kc = kc_heads.clone()
    vc = vc_heads.clone()
    t0 = time.perf_counter()
    out, lse = oracle.decode_step(q_new, k_new, v_new, kc, vc, pos)
    t = time.perf_counter() - t0
    t_full = t * (wl.B * wl.H) / n_heads
    gb = 2.0 * wl.B * wl.H * (pos + 1) * wl.d * 2 / 1e9
    return dict(value=gb / t_full, unit="GB/s", cores=cores, kind="oracle",
                sample=f"one decode step at pos={pos} for {n_heads} of {wl.B * wl.H} (b,h) pairs: {t:.2f} s, "
                       f"scaled by {wl.B * wl.H}/{n_heads}"), (out, lse)


# ----------------------------------------------------------------------------- GPU legs
def allowed_pairs(wl):
    """(query, key) pairs the attention rule lets through, per (b,h): the scores that enter the softmax."""
    if wl.causal_window:
        return wl.W * (wl.N - wl.W) + wl.W * (wl.W + 1) // 2
    return wl.W * wl.N


def fwd_bytes(wl):
    return 2 * (2 * wl.B * wl.H * wl.N * wl.d + 2 * wl.B * wl.H * wl.W * wl.d) + 4 * wl.B * wl.H * wl.W


def run_forward(wl, args, rank, world, device, peaks, with_cpu):
    from paper_2508_20407_b200 import binding as tl
    q, k, v = synth.forward_inputs(wl, device=device)
    out = torch.empty_like(q)
    lse = torch.empty((wl.B, wl.H, wl.W), dtype=torch.float32, device=device)
    tl.ensure_workspace(tl.workspace_bytes_forward(wl.B, wl.H, wl.N, wl.W, wl.d, wl.causal_window), device)
    launches = []

    def step(_):
        tl.tlin_attn_forward(q, k, v, out, lse, wl.causal_window)
        launches.append(tl.tlin_last_launch_count())

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    # small problems would be served from L2 on every call after the first: flush it between timed calls
    flush = torch.empty(int(2.5 * L2_BYTES), dtype=torch.uint8, device=device) if fwd_bytes(wl) < 2 * L2_BYTES else None
    ms, clocks = time_steps(step, args.steps, args.warmup, world, device, sampler, flush)
    ms_step = ms / args.steps
    timed_launches = int(sum(launches[args.warmup:args.warmup + args.steps]))
    flop = 4.0 * wl.B * wl.H * allowed_pairs(wl) * wl.d
    tflops = flop / (ms_step * 1e-3) / 1e12
    t_tensor = flop / (peaks["bf16_tflops"] * 1e12)
    t_hbm = fwd_bytes(wl) / (peaks["hbm_gbs"] * 1e9)
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    if bound == "tensor":
        roof = dict(bound="tensor", achieved=tflops, peak=peaks["bf16_tflops"], unit="TFLOP/s",
                    frac=tflops / peaks["bf16_tflops"])
    else:
        gbs = fwd_bytes(wl) / (ms_step * 1e-3) / 1e9
        roof = dict(bound="hbm", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s", frac=gbs / peaks["hbm_gbs"])
    traffic, traffic_source = FWD_TRAFFIC.get(wl.name, (None, None))
    roof.update(traffic=traffic, traffic_source=traffic_source, algorithmic_bytes=fwd_bytes(wl),
                peak_source=peaks["source"] + " (burst)", kernel="forward (attention kernel + split merge)",
                roofline_ms=max(t_tensor, t_hbm) * 1e3)
    if bound == "tensor" and "bf16_tflops_sustained" in peaks:
        roof["frac_of_sustained_peak"] = tflops / peaks["bf16_tflops_sustained"]
    roof["nominal"] = dict(peak=NOMINAL_BF16_TFLOPS, unit="TFLOP/s", frac=tflops / NOMINAL_BF16_TFLOPS, note="datasheet dense bf16, context only")
    # second ceiling: one exponential per (query, key) pair; the special-function units retire 16 per clock and SM
    exps = float(wl.B) * wl.H * allowed_pairs(wl)
    sfu_rate = 16.0 * 148 * 1.965e9
    roof["secondary"] = dict(bound="special-function unit", exponentials=exps, roofline_ms=exps / sfu_rate * 1e3,
                             note="16 ex2 per clock per SM x 148 SMs x 1965 MHz; the kernel evaluates 5/16 of them on the FMA pipe")

    if getattr(args, "sustained", False) and flush is None:
        ms_s, n_s, clk_s = sustained_leg(step, ms_step, world, device, rank)
        tf_s = flop / (ms_s * 1e-3) / 1e12
        mhz = clk_s["sm_mhz"] if clk_s else None
        roof["sustained"] = dict(calls=n_s, seconds=ms_s * n_s * 1e-3, ms_per_step=ms_s, achieved=tf_s, unit="TFLOP/s",
                                 frac_of_burst_peak=tf_s / peaks["bf16_tflops"],
                                 frac_of_sustained_peak=tf_s / peaks["bf16_tflops_sustained"] if "bf16_tflops_sustained" in peaks else None,
                                 sm_mhz=mhz, reasons=clk_s["reasons"] if clk_s else [],
                                 ms_times_mhz=ms_s * mhz if mhz else None,
                                 ms_times_mhz_of_timed_steps=ms_step * clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None)

    # end to end: pinned host buffers through the host entry point
    e2e = None
    if not args.no_e2e:
        q_h, k_h, v_h = (t.cpu().pin_memory() for t in (q, k, v))
        out_h = torch.empty_like(q_h).pin_memory()
        lse_h = torch.empty((wl.B, wl.H, wl.W), dtype=torch.float32).pin_memory()

        def step_e2e(_):
            tl.tlin_attn_forward_host(q_h, k_h, v_h, out_h, lse_h, q, k, v, out, lse, wl.causal_window)

        n_e2e = max(2, min(args.steps, 5))
        ms_e, _ = time_steps(step_e2e, n_e2e, 1, world, device)
        h2d = sum(t.numel() * t.element_size() for t in (q_h, k_h, v_h))
        d2h = out_h.numel() * out_h.element_size() + lse_h.numel() * 4
        e2e = dict(value=world * wl.B * wl.N / (ms_e / n_e2e * 1e-3), unit="context tokens/s",
                   h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h, ms_per_step=ms_e / n_e2e, steps=n_e2e)
        del q_h, k_h, v_h

    l2_note = ("inputs+outputs %.0f MB > 2 x L2 (126 MB): back-to-back calls, no flush" % (fwd_bytes(wl) / 1e6) if flush is None else
               "inputs+outputs %.0f MB: a %.0f MB buffer is overwritten before every timed call (L2 flush), calls timed one by one"
               % (fwd_bytes(wl) / 1e6, flush.numel() / 1e6))
    del flush
    res = dict(workload=wl.name, shape=dict(B=wl.B, H=wl.H, N=wl.N, W=wl.W, d=wl.d, causal_window=wl.causal_window), l2=l2_note,
               ms_per_step=ms_step, tokens_per_s=world * wl.B * wl.N / (ms_step * 1e-3),
               tflops=tflops, roofline=roof, e2e=e2e, clocks=clocks,
               gpu_launches=timed_launches, launches_per_step=launches[-1] if launches else 0)

    if with_cpu and rank == 0:
        tl.tlin_attn_forward(q, k, v, out, lse, wl.causal_window)
        torch.cuda.synchronize()
        cpu, (rows, ref, ref_lse) = cpu_baseline_forward(wl, q[0, 0].cpu(), k[0, 0].cpu(), v[0, 0].cpu())
        got = out[0, 0, wl.W - rows:].float().cpu().numpy()
        err = abs(got - ref[0, 0]).max()
        lerr = abs(lse[0, 0, wl.W - rows:].cpu().numpy() - ref_lse[0, 0]).max()
        cpu["parity_on_sample"] = dict(max_abs_err=float(err), lse_max_abs_err=float(lerr))
        res["cpu_baseline"] = cpu
    return res


def run_backward(wl, args, rank, world, device, peaks):
    """Backward pass alone (out and lse come from one untimed forward).  FLOPs counted: the five matrix products of the
    chain rule (2.5 x the forward); the two kernels execute seven (both recompute the scores)."""
    from paper_2508_20407_b200 import binding as tl
    q, k, v = synth.forward_inputs(wl, device=device)
    g = torch.Generator(device="cpu").manual_seed(wl.seed + 99)
    dout = torch.randn(q.shape, generator=g, dtype=torch.float32).to(torch.bfloat16).to(device)
    out, lse = tl.tlin_attn_forward(q, k, v, causal_window=wl.causal_window)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    tl.ensure_workspace(tl.workspace_bytes_backward(wl.B, wl.H, wl.N, wl.W, wl.d), device)
    launches = []

    def step(_):
        tl.tlin_attn_backward(q, k, v, out, lse, dout, dq, dk, dv, wl.causal_window)
        launches.append(tl.tlin_last_launch_count())

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    nbytes = 2 * (4 * wl.B * wl.H * wl.N * wl.d + 4 * wl.B * wl.H * wl.W * wl.d)      # q,k,v,out,dout in; dq,dk,dv out
    flush = torch.empty(int(2.5 * L2_BYTES), dtype=torch.uint8, device=device) if nbytes < 2 * L2_BYTES else None
    ms, clocks = time_steps(step, args.steps, args.warmup, world, device, sampler, flush)
    ms_step = ms / args.steps
    flop = 10.0 * wl.B * wl.H * allowed_pairs(wl) * wl.d
    tflops = flop / (ms_step * 1e-3) / 1e12
    # the headline is the library's own choice of arrangement (tlin_set_backward_impl(0)); both arrangements beside it,
    # same call, same timing
    chosen = tl.tlin_backward_arrangement(wl.B, wl.H, wl.N, wl.W, wl.d)
    one_kernel = two_kernels = None
    if wl.d == 128:
        n_counted = len(launches)
        for mode in (1, 2):
            prev = tl.tlin_set_backward_impl(mode)
            try:
                ms1, _ = time_steps(step, args.steps, args.warmup, world, device, None, flush)
            finally:
                tl.tlin_set_backward_impl(prev)
            rec = dict(ms_per_step=ms1 / args.steps, tflops=flop / (ms1 / args.steps * 1e-3) / 1e12)
            if mode == 1:
                two_kernels = dict(rec, note="tlin_set_backward_impl(1): dK/dV kernel, then dQ kernel; seven matrix products, bitwise repeatable")
            else:
                one_kernel = dict(rec, note="tlin_set_backward_impl(2): five matrix products instead of seven, dQ summed by fp32 reductions in L2")
        del launches[n_counted:]
    roof = dict(bound="tensor", achieved=tflops, peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=tflops / peaks["bf16_tflops"],
                traffic=None, algorithmic_bytes=nbytes, peak_source=peaks["source"] + " (burst)",
                kernel=("backward (row statistics, dK/dV kernel, dQ kernel, dQ partial sums)" if chosen != 2 else
                        "backward (row statistics, one dK/dV/dQ kernel with fp32 reductions, dQ rounding)"),
                executed_over_counted_flops=1.4 if chosen != 2 else 1.0, roofline_ms=flop / (peaks["bf16_tflops"] * 1e12) * 1e3)
    if "bf16_tflops_sustained" in peaks:
        roof["frac_of_sustained_peak"] = tflops / peaks["bf16_tflops_sustained"]
    roof["nominal"] = dict(peak=NOMINAL_BF16_TFLOPS, unit="TFLOP/s", frac=tflops / NOMINAL_BF16_TFLOPS, note="datasheet dense bf16, context only")
    l2_note = ("inputs+outputs %.0f MB > 2 x L2 (126 MB): back-to-back calls, no flush" % (nbytes / 1e6) if flush is None else
               "inputs+outputs %.0f MB: a %.0f MB buffer is overwritten before every timed call (L2 flush), calls timed one by one"
               % (nbytes / 1e6, flush.numel() / 1e6))
    return dict(workload=wl.name + " backward", shape=dict(B=wl.B, H=wl.H, N=wl.N, W=wl.W, d=wl.d, causal_window=wl.causal_window),
                l2=l2_note, ms_per_step=ms_step, tflops=tflops, roofline=roof, e2e=None, clocks=clocks, arrangement=chosen, two_kernels=two_kernels, one_kernel=one_kernel,
                gpu_launches=int(sum(launches[args.warmup:])), launches_per_step=launches[-1] if launches else 0)


def run_decode(wl, args, rank, world, device, peaks, with_cpu):
    from paper_2508_20407_b200 import binding as tl
    (kc, vc), (qn, kn, vn) = synth.decode_inputs(wl, device=device)
    ncap = kc.shape[2]
    out = torch.empty((wl.B, wl.H, 1, wl.d), dtype=torch.bfloat16, device=device)
    lse = torch.empty((wl.B, wl.H), dtype=torch.float32, device=device)
    tl.ensure_workspace(tl.workspace_bytes_decode(wl.B, wl.H, ncap, wl.d), device)
    launches = []
    steps = args.decode_steps

    def step(i):
        t = i % wl.W
        tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t, out, lse)
        launches.append(tl.tlin_last_launch_count())

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    ms, clocks = time_steps(step, steps, args.warmup, world, device, sampler)
    ms_step = ms / steps
    # algorithmic bytes of the steps actually timed: K and V rows [0,pos] once each, plus q/k/v_new, out, lse
    tot = 0
    for i in range(args.warmup, args.warmup + steps):
        pos = wl.N + (i % wl.W)
        tot += 2 * wl.B * wl.H * (pos + 1) * wl.d * 2 + 4 * wl.B * wl.H * wl.d * 2 + 4 * wl.B * wl.H
    gbs = tot / (ms * 1e-3) / 1e9
    roof = dict(bound="hbm", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s", frac=gbs / peaks["hbm_gbs"],
                traffic=tot / steps * DECODE_TRAFFIC_RATIO, algorithmic_bytes=tot / steps,
                traffic_source="ncu on a 4096-row cache, scaled by the cached rows (traffic is proportional to them)",
                peak_source=peaks["source"], kernel="decode (split-K kernel + merge)",
                roofline_ms=tot / steps / (peaks["hbm_gbs"] * 1e9) * 1e3,
                nominal=dict(peak=NOMINAL_HBM_GBS, unit="GB/s", frac=gbs / NOMINAL_HBM_GBS, note="datasheet HBM3e, context only"))
    timed_launches = int(sum(launches[args.warmup:args.warmup + steps]))
    if getattr(args, "sustained", False):
        # steady state at the last position of the window, back to back for about a second
        fixed = lambda _i: tl.tlin_decode_step(qn[wl.W - 1], kn[wl.W - 1], vn[wl.W - 1], kc, vc, wl.N + wl.W - 1, out, lse)
        ms_s, n_s, clk_s = sustained_leg(fixed, ms_step, world, device, rank)
        b_s = 2 * wl.B * wl.H * (wl.N + wl.W) * wl.d * 2 + 4 * wl.B * wl.H * wl.d * 2 + 4 * wl.B * wl.H
        gb_s = b_s / (ms_s * 1e-3) / 1e9
        roof["sustained"] = dict(calls=n_s, seconds=ms_s * n_s * 1e-3, ms_per_step=ms_s, achieved=gb_s, unit="GB/s",
                                 frac=gb_s / peaks["hbm_gbs"], sm_mhz=clk_s["sm_mhz"] if clk_s else None,
                                 reasons=clk_s["reasons"] if clk_s else [])
    e2e = None
    if not args.no_e2e:
        host = [t.cpu().pin_memory() for t in (qn, kn, vn)]
        out_h = torch.empty((wl.B, wl.H, 1, wl.d), dtype=torch.bfloat16).pin_memory()
        lse_h = torch.empty((wl.B, wl.H), dtype=torch.float32).pin_memory()
        qd, kd, vd = (torch.empty_like(qn[0]) for _ in range(3))

        def step_e2e(i):
            t = i % wl.W
            tl.tlin_decode_step_host(host[0][t], host[1][t], host[2][t], out_h, lse_h, qd, kd, vd, out, lse, kc, vc, wl.N + t)
            torch.cuda.current_stream().synchronize()   # the caller reads the token's result every step

        n_e2e = min(steps, 32)
        ms_e, _ = time_steps(step_e2e, n_e2e, 1, world, device)
        nb = wl.B * wl.H * wl.d * 2
        e2e = dict(value=world * (tot / steps) / (ms_e / n_e2e * 1e-3) / 1e9, unit="GB/s", h2d_bytes_per_step=3 * nb,
                   d2h_bytes_per_step=nb + wl.B * wl.H * 4, ms_per_step=ms_e / n_e2e, steps=n_e2e)
    res = dict(workload=wl.name, ms_per_step=ms_step, gb_per_s=world * gbs, steps=steps,
               decode_tokens_per_s=world * wl.B / (ms_step * 1e-3), roofline=roof, e2e=e2e, clocks=clocks,
               gpu_launches=timed_launches, launches_per_step=launches[-1] if launches else 0)
    if with_cpu and rank == 0:
        n_heads = 8
        t = 0
        # re-run step 0 so that out/lse hold its result, then compare the sampled heads
        tl.tlin_decode_step(qn[t], kn[t], vn[t], kc, vc, wl.N + t, out, lse)
        torch.cuda.synchronize()
        flat = lambda x: x.reshape(1, wl.B * wl.H, *x.shape[2:])[:, :n_heads].contiguous().cpu()
        cpu, (ref, ref_lse) = cpu_baseline_decode(wl, flat(kc), flat(vc), flat(qn[t]), flat(kn[t]), flat(vn[t]), wl.N + t, n_heads)
        got = flat(out).float().numpy()
        cpu["parity_on_sample"] = dict(max_abs_err=float(abs(got - ref).max()),
                                       lse_max_abs_err=float(abs(lse.reshape(1, -1)[:, :n_heads].cpu().numpy() - ref_lse).max()))
        res["cpu_baseline"] = cpu
    return res


def run_decode_fp8(wl, args, rank, world, device, peaks):
    """Decode over an 8-bit (E4M3) cache of the same shape: half the bytes per cached row.  The cache holds seeded random
    codes (every finite code value, no NaN codes); scales 1/64 per (b,h)."""
    from paper_2508_20407_b200 import binding as tl
    ncap = wl.N + wl.W
    g = torch.Generator(device=device).manual_seed(wl.seed + 8)
    def codes():
        c = torch.randint(0, 254, (wl.B, wl.H, ncap, wl.d), generator=g, device=device, dtype=torch.int16)
        return (c + (c >= 127).to(torch.int16)).to(torch.uint8).contiguous()        # skips 0x7f; 0xff is never drawn
    kc, vc = codes(), codes()
    ks = torch.full((wl.B, wl.H), 1.0 / 64.0, device=device)
    vs = torch.full((wl.B, wl.H), 1.0 / 64.0, device=device)
    _, (qn, kn, vn) = synth.decode_inputs(synth.Workload("fp8_new", wl.B, wl.H, wl.d, 0, wl.W, seed=wl.seed, decode=True), device=device)
    out = torch.empty((wl.B, wl.H, 1, wl.d), dtype=torch.bfloat16, device=device)
    lse = torch.empty((wl.B, wl.H), dtype=torch.float32, device=device)
    tl.ensure_workspace(tl.workspace_bytes_decode(wl.B, wl.H, ncap, wl.d), device)
    launches = []
    steps = args.decode_steps

    def step(i):
        t = i % wl.W
        tl.tlin_decode_step_fp8(qn[t], kn[t], vn[t], kc, vc, ks, vs, wl.N + t, out, lse)
        launches.append(tl.tlin_last_launch_count())

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    ms, clocks = time_steps(step, steps, args.warmup, world, device, sampler)
    ms_step = ms / steps
    tot = 0
    for i in range(args.warmup, args.warmup + steps):
        pos = wl.N + (i % wl.W)
        tot += 2 * wl.B * wl.H * (pos + 1) * wl.d + 4 * wl.B * wl.H * wl.d * 2 + 4 * wl.B * wl.H
    gbs = tot / (ms * 1e-3) / 1e9
    roof = dict(bound="hbm", achieved=gbs, peak=peaks["hbm_gbs"], unit="GB/s", frac=gbs / peaks["hbm_gbs"],
                traffic=tot / steps * DECODE_FP8_TRAFFIC_RATIO,
                traffic_source="ncu on a 4096-row cache, scaled by the cached rows (traffic is proportional to them)",
                algorithmic_bytes=tot / steps, peak_source=peaks["source"], kernel="decode over an 8-bit cache (split-K kernel + merge)",
                roofline_ms=tot / steps / (peaks["hbm_gbs"] * 1e9) * 1e3,
                nominal=dict(peak=NOMINAL_HBM_GBS, unit="GB/s", frac=gbs / NOMINAL_HBM_GBS, note="datasheet HBM3e, context only"))
    return dict(workload=wl.name + " 8-bit cache", ms_per_step=ms_step, gb_per_s=world * gbs, steps=steps,
                decode_tokens_per_s=world * wl.B / (ms_step * 1e-3), roofline=roof, e2e=None, clocks=clocks,
                gpu_launches=int(sum(launches[args.warmup:])), launches_per_step=launches[-1] if launches else 0)


def run_batched(args, rank, world, device, peaks):
    """The inner layers of one depth step of a block (Appendix A: self-attention over the W_oh summary tokens; a generation
    layer over [summary tokens; window]) as a table in ONE launch, beside the same two problems as two calls.  Both read
    the same inputs; a buffer larger than L2 is overwritten before every timed step."""
    from paper_2508_20407_b200 import binding as tl
    wls = [synth.WORKLOADS["inner_self"], synth.WORKLOADS["inner_gen"]]
    tensors = []
    for wl in wls:
        q, k, v = synth.forward_inputs(wl, device=device)
        tensors.append((wl, q, k, v, torch.empty_like(q), torch.empty((wl.B, wl.H, wl.W), dtype=torch.float32, device=device)))
        tl.ensure_workspace(tl.workspace_bytes_forward(wl.B, wl.H, wl.N, wl.W, wl.d, wl.causal_window), device)
    table = [(q, k, v, out, lse, None, wl.causal_window) for (wl, q, k, v, out, lse) in tensors]
    launches = {"batched": [], "separate": []}

    def step_batched(_):
        tl.tlin_attn_forward_batched(table)
        launches["batched"].append(tl.tlin_last_launch_count())

    def step_separate(_):
        n = 0
        for (wl, q, k, v, out, lse) in tensors:
            tl.tlin_attn_forward(q, k, v, out, lse, wl.causal_window)
            n += tl.tlin_last_launch_count()
        launches["separate"].append(n)

    flush = torch.empty(int(2.5 * L2_BYTES), dtype=torch.uint8, device=device)
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    ms_b, clocks = time_steps(step_batched, args.steps, args.warmup, world, device, sampler, flush)
    ms_s, _ = time_steps(step_separate, args.steps, args.warmup, world, device, None, flush)
    ms_b /= args.steps
    ms_s /= args.steps
    flop = sum(4.0 * wl.B * wl.H * allowed_pairs(wl) * wl.d for wl in wls)
    tflops = flop / (ms_b * 1e-3) / 1e12
    roof = dict(bound="tensor", achieved=tflops, peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=tflops / peaks["bf16_tflops"],
                traffic=None, algorithmic_bytes=sum(fwd_bytes(wl) for wl in wls), peak_source=peaks["source"] + " (burst)",
                kernel="forward, two problems in one launch", roofline_ms=flop / (peaks["bf16_tflops"] * 1e12) * 1e3)
    # The same two layers for four requests of 8 heads each (eight problems): alone, a problem of 32 units leaves most of
    # the 148 SMs idle, which is where one launch for the table pays.
    few = []
    for r in range(4):
        for wl in wls:
            w8 = synth.Workload(f"{wl.name}_h8_r{r}", 1, 8, wl.d, wl.N, wl.W, seed=wl.seed + 100 + r, causal_window=wl.causal_window)
            q, k, v = synth.forward_inputs(w8, device=device)
            few.append((w8, q, k, v, torch.empty_like(q), torch.empty((1, 8, w8.W), dtype=torch.float32, device=device)))
    table8 = [(q, k, v, out, lse, None, wl.causal_window) for (wl, q, k, v, out, lse) in few]

    def step_batched8(_):
        tl.tlin_attn_forward_batched(table8)

    def step_separate8(_):
        for (wl, q, k, v, out, lse) in few:
            tl.tlin_attn_forward(q, k, v, out, lse, wl.causal_window)

    ms_b8, _ = time_steps(step_batched8, args.steps, args.warmup, world, device, None, flush)
    ms_s8, _ = time_steps(step_separate8, args.steps, args.warmup, world, device, None, flush)
    ms_b8 /= args.steps
    ms_s8 /= args.steps
    # Cache-hit analogue (Appendix A: per generation layer one row against the W_oh cached summary tokens and the window so
    # far): three layers' rows, B8 H32, caches of 1024 + 64 rows with the new token appended, as one table against three
    # tlin_decode_step calls (two kernels each).
    rows = []
    for li in range(3):
        dwl = synth.Workload(f"layer{li}_hit", 8, 32, 128, 1024 + 63, 1, seed=40 + li, decode=True)
        (kc, vc), (qn, kn, vn) = synth.decode_inputs(dwl, device=device)
        rows.append((qn[0], kn[0], vn[0], kc, vc, dwl.N, torch.empty_like(qn[0]), torch.empty((8, 32), dtype=torch.float32, device=device)))
    tl.ensure_workspace(tl.workspace_bytes_decode(8, 32, 1024 + 64, 128), device)
    ms_dt, _ = time_steps(lambda _i: tl.tlin_decode_step_batched(rows), args.steps, args.warmup, world, device, None, flush)
    ms_ds, _ = time_steps(lambda _i: [tl.tlin_decode_step(*r[:6], r[6], r[7]) for r in rows], args.steps, args.warmup, world, device, None, flush)
    decode_table = dict(batched_ms=ms_dt / args.steps, separate_calls_ms=ms_ds / args.steps, batched_over_separate=ms_dt / ms_ds,
                        what="three problems of B8 H32 d128, 1087 cached rows + the appended row: one launch against six")
    return dict(workload="inner_self + inner_gen as one table", ms_per_step=ms_b, tflops=tflops, roofline=roof, e2e=None, clocks=clocks,
                decode_table=decode_table,
                separate_calls_ms_per_step=ms_s, batched_over_separate=ms_b / ms_s,
                eight_problems_of_8_heads=dict(batched_ms=ms_b8, separate_calls_ms=ms_s8, batched_over_separate=ms_b8 / ms_s8),
                l2="a %.0f MB buffer is overwritten before every timed step (L2 flush), steps timed one by one" % (flush.numel() / 1e6),
                gpu_launches=int(sum(launches["batched"][args.warmup:args.warmup + args.steps])),
                launches_per_step=launches["batched"][-1], separate_launches_per_step=launches["separate"][-1])


def run_n_sweep(args, rank, world, device, peaks):
    """Forward time against context length at fixed B, H, W, d (the paper's claim is cost linear in N, Section 4 and
    Appendix A): N = 8k ... 256k, least-squares line t = a + b*N and its largest relative residual; cfg3/cfg4 also with
    causal_window = 0."""
    from paper_2508_20407_b200 import binding as tl
    pts = []
    for n in (8192, 16384, 32768, 65536, 131072, 262144):
        wl = synth.Workload(f"sweep_N{n}", 1, 32, 128, n, 512, seed=11, causal_window=1)
        q, k, v = synth.forward_inputs(wl, device=device)
        out = torch.empty_like(q)
        lse = torch.empty((wl.B, wl.H, wl.W), dtype=torch.float32, device=device)
        tl.ensure_workspace(tl.workspace_bytes_forward(wl.B, wl.H, wl.N, wl.W, wl.d, 1), device)
        flush = torch.empty(int(2.5 * L2_BYTES), dtype=torch.uint8, device=device) if fwd_bytes(wl) < 2 * L2_BYTES else None
        ms, _ = time_steps(lambda _: tl.tlin_attn_forward(q, k, v, out, lse, 1), args.steps, args.warmup, world, device, None, flush)
        ms /= args.steps
        pts.append(dict(N=n, ms=ms, tflops=4.0 * wl.B * wl.H * wl.W * n * wl.d / (ms * 1e-3) / 1e12))
        del q, k, v, out, lse, flush
        torch.cuda.empty_cache()
    import numpy as np
    x = np.array([p["N"] for p in pts], dtype=np.float64)
    y = np.array([p["ms"] for p in pts], dtype=np.float64)
    b, a = np.polyfit(x, y, 1)
    resid = float(np.max(np.abs(a + b * x - y) / y))
    unmasked = []
    for name in ("cfg3_long", "cfg4_vlong"):
        wl = synth.WORKLOADS[name]
        q, k, v = synth.forward_inputs(wl, device=device)
        out = torch.empty_like(q)
        lse = torch.empty((wl.B, wl.H, wl.W), dtype=torch.float32, device=device)
        row = dict(workload=name)
        for causal in (1, 0):
            tl.ensure_workspace(tl.workspace_bytes_forward(wl.B, wl.H, wl.N, wl.W, wl.d, causal), device)
            ms, _ = time_steps(lambda _: tl.tlin_attn_forward(q, k, v, out, lse, causal), args.steps, args.warmup, world, device)
            row[f"ms_causal_window_{causal}"] = ms / args.steps
        unmasked.append(row)
        del q, k, v, out, lse
        torch.cuda.empty_cache()
    return dict(points=pts, fit=dict(intercept_ms=float(a), ms_per_1k_keys=float(b * 1024), max_rel_residual=resid),
                t_cfg4_over_t_cfg3=unmasked[1]["ms_causal_window_1"] / unmasked[0]["ms_causal_window_1"], flop_ratio=8.0,
                causal_vs_unmasked=unmasked, shape="B1 H32 W512 d128, causal window")


# ----------------------------------------------------------------------------- reference arm (the oracle)
def run_reference(args, rank, world):
    if rank != 0:
        return None
    import oracle
    wl = synth.WORKLOADS[WORKLOADS[args.workload]]
    cores = oracle.num_threads()
    if wl.decode:
        n_heads = max(1, min(cores, 8))
        small = synth.Workload(wl.name, 1, n_heads, wl.d, wl.N, 1, wl.seed, decode=True)
        (kc, vc), (qn, kn, vn) = synth.decode_inputs(small, steps=1)
        times = []
        for i in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            oracle.decode_step(qn[0], kn[0], vn[0], kc, vc, wl.N)
            times.append(time.perf_counter() - t0)
        t = sum(times[args.warmup:]) / args.steps
        t_full = t * (wl.B * wl.H) / n_heads
        gb = 2.0 * wl.B * wl.H * (wl.N + 1) * wl.d * 2 / 1e9
        value, unit, metric = gb / t_full, "GB/s", "decode_kv_GB_per_s"
        sample = f"one decode step at pos={wl.N} for {n_heads} of {wl.B * wl.H} (b,h) pairs per step, scaled"
    else:
        # Rows per step: as many of the head's last query rows as keep the whole run near REFERENCE_BUDGET_S.  Two untimed
        # probes (16 and 128 rows) give the oracle's fixed cost per call (the fp64 copies of K and V) and its cost per row;
        # few rows per call would charge the fixed cost to every row and understate the oracle.
        def head_rows(rows):
            q, k, v = synth.forward_inputs_head(wl, 0, 0, q_rows=slice(wl.W - rows, wl.W))
            return q.view(1, 1, rows, wl.d), k.view(1, 1, wl.N, wl.d), v.view(1, 1, wl.N, wl.d)

        def probe(rows):
            q, k, v = head_rows(rows)
            t0 = time.perf_counter()
            oracle.attn_forward(q, k, v, wl.causal_window)
            return time.perf_counter() - t0

        r_lo, r_hi = min(16, wl.W), min(128, wl.W)
        probe(r_lo)                                         # first touch of the library and the thread pool
        t_lo, t_hi = probe(r_lo), probe(r_hi)
        per_row = max((t_hi - t_lo) / max(r_hi - r_lo, 1), 1e-6)
        fixed = max(t_lo - per_row * r_lo, 0.0)
        per_step = REFERENCE_BUDGET_S / max(args.warmup + args.steps, 1)
        rows = int(min(wl.W, max(8, (per_step - fixed) / per_row)))
        rows = max(8, rows // 8 * 8) if rows < wl.W else wl.W
        q, k, v = head_rows(rows)
        times = []
        for i in range(args.warmup + args.steps):
            t0 = time.perf_counter()
            oracle.attn_forward(q, k, v, wl.causal_window)
            times.append(time.perf_counter() - t0)
        t = sum(times[args.warmup:]) / args.steps
        t_full = t * (wl.B * wl.H * wl.W) / rows
        value, unit, metric = wl.B * wl.N / t_full, "context tokens/s", "context_tokens_per_s"
        sample = f"last {rows} of {wl.W} query rows of head (0,0), all {wl.N} keys per step, scaled by rows"
    return {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_full * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl, max(world, 1)),
            "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def config_of(wl, world):
    """The `config` object of the JSON line; both arms (this library and the oracle) print the same one."""
    if wl.decode:
        kv = 4e-6 * wl.B * wl.H * wl.N * wl.d
        l2 = "cached K+V %.0f MB > L2 (126 MB): steps back to back, no flush" % kv
    elif fwd_bytes(wl) < 2 * L2_BYTES:
        l2 = ("inputs+outputs %.0f MB: a %.0f MB buffer is overwritten before every timed call (L2 flush), calls timed one by one"
              % (fwd_bytes(wl) / 1e6, int(2.5 * L2_BYTES) / 1e6))
    else:
        l2 = "inputs+outputs %.0f MB > 2 x L2 (126 MB): back-to-back calls, no flush" % (fwd_bytes(wl) / 1e6)
    return {"workload": wl.name, "B": wl.B, "H": wl.H, "N": wl.N, "W": wl.W, "d": wl.d, "causal_window": wl.causal_window,
            "parallelism": f"replicas x{world}", "l2": l2}


def compact_leg(leg):
    """An 'also' leg without the long descriptive fields (the headline keeps them): what was run, its time, the
    roofline figures and the clocks."""
    r = leg["roofline"]
    roof = {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac", "frac_of_sustained_peak", "traffic", "algorithmic_bytes",
                              "executed_over_counted_flops", "sustained") if k in r}
    c = leg.get("clocks") or {}
    out = {k: leg[k] for k in ("workload", "shape", "ms_per_step", "tflops", "gb_per_s", "tokens_per_s", "decode_tokens_per_s", "steps",
                               "gpu_launches", "launches_per_step", "separate_calls_ms_per_step", "batched_over_separate",
                               "separate_launches_per_step", "eight_problems_of_8_heads", "decode_table", "arrangement", "two_kernels", "one_kernel") if k in leg and leg[k] is not None}
    out["roofline"] = roof
    out["clocks"] = {"sm_mhz": c.get("sm_mhz"), "sm_max_mhz": c.get("sm_max_mhz"), "reasons": c.get("reasons", [])}
    if leg.get("e2e"):
        out["e2e"] = leg["e2e"]
    out["l2_flush"] = "between calls" if "flush" in leg.get("l2", "") and "no flush" not in leg.get("l2", "") else "inputs larger than L2"
    return out


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", choices=sorted(WORKLOADS), default="fwd128k")
    ap.add_argument("--impl", choices=["tlin", "reference"], default="tlin")
    ap.add_argument("--only", action="store_true", help="time only --workload (no 'also' legs)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-sustained", dest="sustained", action="store_false",
                    help="skip the back-to-back loops of about a second on the workloads with a target")
    ap.add_argument("--decode-steps", type=int, default=0, help="timed decode steps (default: max(steps, 64))")
    ap.add_argument("--shape", default="", help="custom shape B,H,N,W,d[,causal] instead of the named workload (profiling); with --workload decode, N is the "
                         "number of cached rows and W the number of decode steps available")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "tlin" else args.warmup
    if args.decode_steps <= 0:
        args.decode_steps = max(args.steps, 64)
    rank, world, local = dist_info()

    if args.impl == "reference":
        line = run_reference(args, rank, world)
        if line is not None:
            print(json.dumps(line), flush=True)
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    peaks = load_peaks()
    if args.workload == "nsweep":          # a measurement of its own (linearity in N), not a bench line
        res = run_n_sweep(args, rank, world, device, peaks)
        if rank == 0:
            print(json.dumps({"metric": "forward_ms_vs_context_length", "n_gpus": world, "steps": args.steps, "warmup": args.warmup, **res}), flush=True)
        if world > 1:
            torch.distributed.destroy_process_group()
        return 0
    wl = synth.WORKLOADS[WORKLOADS[args.workload]]
    if args.shape:
        v = [int(x) for x in args.shape.split(",")]
        wl = synth.Workload("custom_" + args.shape.replace(",", "_"), v[0], v[1], v[4], v[2], v[3], seed=9,
                            causal_window=v[5] if len(v) > 5 else 1, decode=args.workload in ("decode", "decode_fp8"))
    with_cpu = (not args.no_cpu) and world == 1
    if args.workload in BACKWARD:
        main_res = run_backward(wl, args, rank, world, device, peaks)
    elif args.workload == "inner_batched":
        main_res = run_batched(args, rank, world, device, peaks)
    elif args.workload == "decode_fp8":
        main_res = run_decode_fp8(wl, args, rank, world, device, peaks)
    else:
        runner = run_decode if wl.decode else run_forward
        main_res = runner(wl, args, rank, world, device, peaks, with_cpu)
    also = []
    full_legs = {args.workload: main_res}
    if not args.only and world == 1:
        for name in ("fwd32k", "decode", "restore", "inner_self", "inner_gen", "inner_batched", "fwd_seq", "bwd_chunk", "bwd32k", "bwd_seq", "decode_fp8"):
            if name == args.workload:
                continue
            torch.cuda.empty_cache()
            time.sleep(1.0)     # the legs are independent measurements: let the power state of the previous one settle
            w2 = synth.WORKLOADS[WORKLOADS[name]]
            a2 = argparse.Namespace(**vars(args))
            a2.no_e2e = args.no_e2e or name not in ("fwd32k", "decode")     # host-buffer legs only where they are cheap to set up
            a2.sustained = args.sustained and name in ("fwd32k", "decode")  # the legs with a stated target
            if name in BACKWARD:
                leg = run_backward(w2, a2, rank, world, device, peaks)
            elif name == "inner_batched":
                leg = run_batched(a2, rank, world, device, peaks)
            elif name == "decode_fp8":
                leg = run_decode_fp8(w2, a2, rank, world, device, peaks)
            else:
                leg = (run_decode if w2.decode else run_forward)(w2, a2, rank, world, device, peaks, False)
            full_legs[name] = leg
            also.append(compact_leg(leg))

    if rank == 0:
        if args.workload in BACKWARD:
            metric, unit, value = "attention_backward_TFLOP_per_s", "TFLOP/s", world * main_res["tflops"]
        elif args.workload == "inner_batched":
            metric, unit, value = "attention_forward_TFLOP_per_s", "TFLOP/s", world * main_res["tflops"]
        elif wl.decode:
            metric, unit, value = "decode_kv_GB_per_s", "GB/s", main_res["gb_per_s"]
        else:
            metric, unit, value = "context_tokens_per_s", "context tokens/s", main_res["tokens_per_s"]
        # the three workloads with a stated target (>= 0.60 of the tensor roofline forward, >= 0.70 of the HBM roofline
        # decode), in one compact object at the very end of the line
        targets = {}
        for key, leg_name, bar in (("cfg3", "fwd32k", 0.60), ("cfg4", "fwd128k", 0.60), ("cfg5", "decode", 0.70)):
            leg = full_legs.get(leg_name)
            if leg is None:
                continue
            r, c = leg["roofline"], leg.get("clocks") or {}
            t = dict(ms_per_step=round(leg["ms_per_step"], 5), achieved=round(r["achieved"], 1), unit=r["unit"], peak=r["peak"],
                     frac=round(r["frac"], 4), bar=bar, met=bool(r["frac"] >= bar), sm_mhz=c.get("sm_mhz"), reasons=c.get("reasons", []))
            if "sustained" in r:
                sr = r["sustained"]
                t["sustained"] = dict(seconds=round(sr["seconds"], 2), achieved=round(sr["achieved"], 1), sm_mhz=sr["sm_mhz"], reasons=sr["reasons"],
                                      frac_of_burst_peak=round(sr.get("frac_of_burst_peak", sr.get("frac", 0.0)), 4))
                if sr.get("frac_of_sustained_peak") is not None:
                    t["sustained"]["frac_of_sustained_peak"] = round(sr["frac_of_sustained_peak"], 4)
            targets[key] = t
        line = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world,
            "steps": main_res.get("steps", args.steps), "warmup": args.warmup, "ms_per_step": main_res["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": config_of(wl, world),
            "also": also,
            "tflops": main_res.get("tflops"),
            "gpu_launches": main_res["gpu_launches"], "launches_per_step": main_res["launches_per_step"],
            **{k: main_res[k] for k in ("separate_calls_ms_per_step", "batched_over_separate", "separate_launches_per_step",
                                        "eight_problems_of_8_heads", "decode_table", "arrangement", "two_kernels", "one_kernel") if k in main_res and main_res[k] is not None},
            "cpu_baseline": main_res.get("cpu_baseline"), "e2e": main_res["e2e"], "clocks": main_res["clocks"],
            "roofline": main_res["roofline"], "targets": targets,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
