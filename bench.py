#!/usr/bin/env python
"""Benchmark of the OSC dual-path linear on B200 (one JSON line on stdout).

A step is one pass of the online hot path over one batch: `osc_linear` (fused
extract + MXFP4 quantize kernel, then the dual-path tcgen05 GEMM) on the
Qwen3-8B QKV projection, M=8192 tokens, K=4096, N=6144, two protected channels
per 32-group (K_o=256).  Inputs are seeded and synthetic (outlier-planted
activations, N(0,0.02) weights); the offline weight split is done once before
timing, as in the paper.

  value       TFLOP/s of useful work, 2*M*N*(K+K_o) / step time, inputs resident in HBM
  e2e         the same with X in pinned host memory and Y copied back, copies inside the timed region
  roofline    the dual-path GEMM kernel against the tensor peak of its own FLOP mix
              (FP4 peak = 4 x, measured BF16 peak from MEASURED_PEAKS.json)
  cpu_baseline the CPU oracle timed on a bounded sample of the same workload (rank 0, N=1 only)
  extra       the step against the dual-path roofline of the whole linear (measured-peak and data-sheet
              basis), the quantizer's HBM fraction, the same build's FP8 W8A8 linear on the same shape, and
              extra.configs: one row per shape the benchmark configurations name (median and minimum of 30
              timed iterations, L2 cold and warm, % of the roofline on both bases, speed-up over the own FP8
              linear on the same shape; every row is replayed from a CUDA graph and says so, with the median
              of plain stream launches beside it)

Between timed steps the buffers rotate over 4 independent sets (inputs, workspace,
outputs and prepared weights: ~0.9 GB, 7x the L2), so no step finds its data in L2.

`--impl reference` times the CPU oracle instead (host cores, bounded sample per step).
`--sweep` prints a table over all benchmark shapes to stderr and writes sweep.json into the output folder
(OSC_BENCH_OUT, a scratch folder beside this file by default); it prints no bench line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2604_12782_b200 import roofline, synth  # noqa: E402

WORKLOAD = {"name": "qwen3-8b-qkv", "M": 8192, "K": 4096, "N": 6144, "ch_per_group": 2}
NSETS = 4
METRIC = "OSC linear TFLOP/s"

DATASHEET = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}   # dense peaks and HBM3e bandwidth of the data sheet


def load_traffic():
    """DRAM bytes (read + written) of one launch of the dominant kernel on the bench workload, from the one ncu
    capture whose numbers are kept under profiles/ together with the commit and the command they came from."""
    path = os.path.join(ROOT, "profiles", "dominant_kernel_traffic.txt")
    try:
        with open(path) as f:
            t = json.load(f)
        return float(t["dram_bytes_read"]) + float(t["dram_bytes_write"]), t
    except (OSError, KeyError, ValueError):
        return None, None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p.get("bf16_tflops_sustained"),
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the GPU is busy."""

    def __init__(self, index: int):
        self.samples, self.stamps, self.reasons, self.max_mhz = [], [], set(), None
        self.marks = {}
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown if hasattr(nv, "nvmlClocksEventReasonHwSlowdown") else 0x8,
                 "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4,
                 "hw_power_brake": 0x80}
        n = 0
        while not self._stop.is_set():
            try:
                # an NVML query takes about a millisecond: the clock every round, the reasons every fourth, no sleep in
                # between, so that even a timed region of a few milliseconds gets more than one clock sample
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.stamps.append(time.perf_counter())
                n += 1
                if n % 4 == 1:
                    try:
                        r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                    except Exception:
                        r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                    for k, bit in names.items():
                        if r & bit:
                            self.reasons.add(k)
            except Exception:
                time.sleep(0.001)
            time.sleep(0.00005)   # yields the interpreter lock to the launching thread

    def mark(self, name):
        """Remembers the host time of a boundary of the timed region."""
        self.marks[name] = time.perf_counter()

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
            t_end = time.perf_counter() + 2.0      # the first query can take tens of milliseconds: wait for it, so
            while not self.samples and time.perf_counter() < t_end:   # that the sampler is running when timing starts
                time.sleep(0.001)

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join()
        med = float(np.median(self.samples)) if self.samples else None
        t0, t1 = self.marks.get("t0"), self.marks.get("t1")
        inside = [c for c, t in zip(self.samples, self.stamps) if t0 is not None and t1 is not None and t0 <= t <= t1]
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "samples_in_timed_region": len(inside),
                "sm_mhz_in_timed_region": float(np.median(inside)) if inside else None,
                "span": "sampled from the start of the timed region to the end of all device-timed loops of this run"}


# ------------------------------------------------------------------- multi-process glue
def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time (the job's time): all-reduce MAX over the default process group, if there is one.
    Works with the nccl backend (device = a cuda device) and with gloo (device None -> CPU tensor)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank: float, world: int, ms: float) -> float:
    """Replicas only: every rank processes `units_per_rank` (FLOPs) per step; the job's rate is the sum over
    ranks divided by the slowest rank's time, in TFLOP/s."""
    return world * units_per_rank / (ms * 1e-3) / 1e12


# ---------------------------------------------------------------------- reference arm
def oracle_sample_step(oracle, case, wts, rows):
    """One bounded step of the CPU oracle: Algorithm 2 on `rows` activation rows, then Eq. 5."""
    act = oracle.quantize_extract(case["X"][:rows], case["lut"])
    oracle.gemm_dual(act, wts)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    rows = args.ref_rows
    case = synth.osc_linear_case(0, rows, WORKLOAD["K"], WORKLOAD["N"], WORKLOAD["ch_per_group"])
    wts = oracle.prepare_weights(case["W"], case["lut"])
    ko = wts["K_o"]
    for _ in range(args.warmup):
        oracle_sample_step(oracle, case, wts, min(rows, 8))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_step(oracle, case, wts, rows)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    flops = 2.0 * rows * WORKLOAD["N"] * (WORKLOAD["K"] + ko)
    val = flops / dt / 1e12
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD["name"], **{k: WORKLOAD[k] for k in ("M", "K", "N")}, "K_o": ko},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"{rows} of {WORKLOAD['M']} activation rows x all N per step "
                                       "(weights prepared once, as on the GPU)"},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------ GPU arm
def dev_bf16(torch, bits):
    if isinstance(bits, torch.Tensor):
        return bits
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


class OscProblem:
    """NSETS rotating buffer sets of one OSC linear."""

    def __init__(self, torch, B, case, nsets):
        self.B, self.M, self.K, self.N = B, case["M"], case["K"], case["N"]
        X0, W0 = dev_bf16(torch, case["X"]), dev_bf16(torch, case["W"])
        self.X = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(nsets)]
        self.w = []
        for i in range(nsets):
            Wi = W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous()
            self.w.append(B.osc_prepare_weights(Wi, case["lut"]))
        self.sz = B.osc_act_sizes(self.w[0], self.M)
        self.ws = [torch.empty(self.sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(nsets)]
        self.Y = [torch.empty(self.M, self.N, dtype=torch.bfloat16, device="cuda") for _ in range(nsets)]
        self.K_o, self.K_o_pad = self.w[0].K_o, self.w[0].K_o_pad
        self.n = nsets

    def step(self, i):
        j = i % self.n
        self.B.osc_linear(self.w[j], self.X[j], self.Y[j], self.ws[j])

    def views(self, j):
        sz, ws = self.sz, self.ws[j]
        return ws[sz.xq_offset:], ws[sz.sfa_offset:], ws[sz.xo_offset:]

    def quant(self, i):
        j = i % self.n
        xq, sfa, xo = self.views(j)
        self.B.osc_quantize_extract(self.w[j], self.X[j], xq, sfa, xo)

    def gemm(self, i):
        j = i % self.n
        xq, sfa, xo = self.views(j)
        self.B.osc_gemm_dual(self.w[j], xq, sfa, xo, self.M, self.Y[j])


class Fp8Problem:
    def __init__(self, torch, B, case, nsets):
        self.B, self.M, self.K, self.N = B, case["M"], case["K"], case["N"]
        X0, W0 = dev_bf16(torch, case["X"]), dev_bf16(torch, case["W"])
        self.X = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(nsets)]
        self.w = [B.osc_fp8_prepare_weights(W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous())
                  for i in range(nsets)]
        self.sz = B.osc_fp8_act_sizes(self.w[0], self.M)
        self.ws = [torch.empty(self.sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(nsets)]
        self.Y = [torch.empty(self.M, self.N, dtype=torch.bfloat16, device="cuda") for _ in range(nsets)]
        self.n = nsets

    def step(self, i):
        j = i % self.n
        self.B.osc_fp8_linear(self.w[j], self.X[j], self.Y[j], self.ws[j])

    def quant(self, i):
        j = i % self.n
        self.B.osc_fp8_quantize(self.X[j], self.ws[j][self.sz.x8_offset:], self.ws[j][self.sz.sx_offset:])

    def gemm(self, i):
        j = i % self.n
        self.B.osc_fp8_gemm(self.w[j], self.ws[j][self.sz.x8_offset:], self.ws[j][self.sz.sx_offset:], self.M,
                            self.Y[j])


class Mxfp8Problem:
    """The fallback in its 8-bit micro-scaling form (MXFP8): same interface as Fp8Problem."""

    def __init__(self, torch, B, case, nsets):
        self.B, self.M, self.K, self.N = B, case["M"], case["K"], case["N"]
        X0, W0 = dev_bf16(torch, case["X"]), dev_bf16(torch, case["W"])
        self.X = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(nsets)]
        self.w = [B.osc_mxfp8_prepare_weights(W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous())
                  for i in range(nsets)]
        self.sz = B.osc_mxfp8_act_sizes(self.w[0], self.M)
        self.ws = [torch.empty(self.sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(nsets)]
        self.Y = [torch.empty(self.M, self.N, dtype=torch.bfloat16, device="cuda") for _ in range(nsets)]
        self.n = nsets

    def step(self, i):
        j = i % self.n
        self.B.osc_mxfp8_linear(self.w[j], self.X[j], self.Y[j], self.ws[j])

    def quant(self, i):
        j = i % self.n
        self.B.osc_mxfp8_quantize(self.X[j], self.ws[j][self.sz.x8_offset:], self.ws[j][self.sz.sfa_offset:])

    def gemm(self, i):
        j = i % self.n
        self.B.osc_mxfp8_gemm(self.w[j], self.ws[j][self.sz.x8_offset:], self.ws[j][self.sz.sfa_offset:], self.M,
                              self.Y[j])


def time_loop(torch, fn, steps, warmup):
    """Average milliseconds per call of fn(i) over `steps` calls, CUDA events on the current stream."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / max(steps, 1)


def time_graph(torch, fn, n):
    """Milliseconds of GPU time per call when `n` calls are captured once in a CUDA graph and replayed: what a
    few-row (decode) step costs when the host does not pace the launches."""
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())   # the problem's buffers and weights were prepared there
    with torch.cuda.stream(st):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            for i in range(n):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        g.replay()
        e1.record(st)
        torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def time_split(torch, prob, steps):
    """Per-kernel averages (ms): events between the quantizer and the GEMM of every step."""
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    torch.cuda.synchronize()
    for i in range(steps):
        ev[i][0].record()
        prob.quant(i)
        ev[i][1].record()
        prob.gemm(i)
        ev[i][2].record()
    torch.cuda.synchronize()
    tq = sum(e[0].elapsed_time(e[1]) for e in ev) / steps
    tg = sum(e[1].elapsed_time(e[2]) for e in ev) / steps
    return tq, tg


# ------------------------------------------------------------------ rows per benchmark shape
CALLS_PER_ITERATION = 4   # plain mode: consecutive calls between two events (an event in front of every call would
                          # add its own gap and cut the programmatic overlap between one call's GEMM and the next
                          # call's quantizer, which is how the linears of a layer follow each other)


def per_call_times(torch, fn, iters, warm, graph_calls=0, calls=0):
    """Milliseconds per call of fn(i), one sample per timed iteration.  Plain mode: a timed iteration is
    `calls` (default CALLS_PER_ITERATION) consecutive calls between two events (iters + 1 events on the current
    stream).  Graph mode
    (graph_calls > 0): `graph_calls` calls are captured once in a CUDA graph and every timed iteration is one replay,
    so the host does not pace few-row launches."""
    if graph_calls:
        st = torch.cuda.Stream()
        st.wait_stream(torch.cuda.current_stream())   # the problem's buffers and weights were prepared there
        out = []
        with torch.cuda.stream(st):
            for i in range(3):
                fn(i)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                for i in range(graph_calls):
                    fn(i)
            for _ in range(max(1, warm // 2)):
                g.replay()
            torch.cuda.synchronize()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
            ev[0].record(st)
            for i in range(iters):
                g.replay()
                ev[i + 1].record(st)
            torch.cuda.synchronize()
            out = [ev[i].elapsed_time(ev[i + 1]) / graph_calls for i in range(iters)]
        return out
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    c = calls or CALLS_PER_ITERATION
    ev[0].record()
    for i in range(iters):
        for j in range(c):
            fn(i * c + j)
        ev[i + 1].record()
    torch.cuda.synchronize()
    return [ev[i].elapsed_time(ev[i + 1]) / c for i in range(iters)]


def sets_for_cold_l2(torch, bytes_per_set):
    """Buffer sets to rotate over so that the data touched between two uses of a set exceeds twice the L2."""
    l2 = torch.cuda.get_device_properties(torch.cuda.current_device()).L2_cache_size
    return int(min(24, max(2, math.ceil(2.0 * l2 / max(bytes_per_set, 1)) + 1)))


def config_rows(torch, B, pk, iters=30, warm=5):
    """One row per (M, K, N) the benchmark configurations name: the Qwen3-8B QKV projection at four M, gate_up and
    the FP8 down projection at three M, the four linears of a decoder layer at M = 4096, the two grouped MoE calls.
    Every row: median and minimum of `iters` timed iterations with L2 cold (rotating buffer sets) and warm (one
    set), % of its roofline on the measured-peak and on the data-sheet basis (from the cold median), and the
    speed-up over this build's FP8 W8A8 linear on the same shape.  Inputs are drawn on the device."""
    meas = roofline.peaks(pk["bf16_tflops"], pk["hbm_gbs"])
    sheet = roofline.peaks(DATASHEET["bf16_tflops"], DATASHEET["hbm_gbs"])
    rows = []

    def stats(ms_list):
        a = np.asarray(ms_list) * 1e3
        return float(np.median(a)), float(a.min())

    def settle():
        """A short idle gap in front of every measurement: rows that follow a long tensor-bound row otherwise inherit
        its power-capped clock, and the same row read 60 us in one run and 80 us in the next."""
        torch.cuda.synchronize()
        time.sleep(0.2)

    def measure(prob):
        """Every row the same way: the calls captured once in a CUDA graph (2 x sets calls, rotating over the sets for
        the cold regime, one set for the warm one) and one replay per timed iteration - device time without the
        host's launch path, which paces few-row calls and adds 1-2 us per kernel boundary to the others.  The
        median of the same calls launched one by one on the stream is reported beside it."""
        gc = max(4, 2 * prob.n)
        settle()
        cold = stats(per_call_times(torch, prob.step, iters, warm, gc))
        settle()
        warm_ = stats(per_call_times(torch, lambda i: prob.step(0), iters, warm, gc))
        settle()
        # few-row calls last ~10 us: sixteen of them between two events, so that the events' own gap stays a few per cent
        plain = stats(per_call_times(torch, prob.step, iters, warm, calls=16 if prob.M <= 128 else 0))
        return cold, warm_, plain, "cuda graph replay of %d calls per timed iteration" % gc

    def osc_row(name, M, K, N, cpg, seed):
        case = synth.osc_linear_case_torch(torch, seed, M, K, N, cpg)
        kop = (K // 32 * cpg + 63) // 64 * 64
        per_set = N * K / 2 + N * K / 32 + 2.0 * N * kop + 2.0 * M * K + roofline.osc_intermediate_bytes(M, K, kop) + 2.0 * M * N
        n = sets_for_cold_l2(torch, per_set)
        p = OscProblem(torch, B, case, n)
        cold, warm_, plain, how = measure(p)
        f8 = Fp8Problem(torch, B, case, sets_for_cold_l2(torch, N * K + 3.0 * M * K + 2.0 * M * N))
        settle()
        f8cold = stats(per_call_times(torch, f8.step, iters, warm, max(4, 2 * f8.n)))
        B.osc_sync_check()
        f4, f16 = roofline.osc_flops(M, N, K, p.K_o)
        r_m, r_s = (roofline.osc_roofline_seconds(M, N, K, p.K_o, pkx) * 1e6 for pkx in (meas, sheet))
        rows.append({"name": name, "path": "osc", "M": M, "K": K, "N": N, "K_o": p.K_o, "timing": how, "sets": n,
                     "cold_us_median": cold[0], "cold_us_min": cold[1], "warm_us_median": warm_[0], "warm_us_min": warm_[1],
                     "plain_launches_cold_us_median": plain[0], "plain_launches_cold_us_min": plain[1],
                     "tflops": (f4 + f16) / cold[0] / 1e6, "roof_us": r_m, "roof_us_datasheet": r_s,
                     "pct_roofline": 100.0 * r_m / cold[0], "pct_roofline_datasheet": 100.0 * r_s / cold[0],
                     "pct_roofline_plain_launches": 100.0 * r_m / plain[0],
                     "fp8_cold_us_median": f8cold[0], "speedup_vs_fp8": f8cold[0] / cold[0]})
        del p, f8, case
        torch.cuda.empty_cache()

    def fp8_row(name, M, K, N, seed):
        case = synth.fp8_linear_case_torch(torch, seed, M, K, N)
        n = sets_for_cold_l2(torch, N * K + 3.0 * M * K + 2.0 * M * N)
        p = Fp8Problem(torch, B, case, n)
        cold, warm_, plain, how = measure(p)
        B.osc_sync_check()
        r_m, r_s = (roofline.fp8_roofline_seconds(M, N, K, pkx) * 1e6 for pkx in (meas, sheet))
        rows.append({"name": name, "path": "fp8 fallback (is the own FP8 W8A8 linear)", "M": M, "K": K, "N": N, "timing": how,
                     "sets": n, "cold_us_median": cold[0], "cold_us_min": cold[1], "warm_us_median": warm_[0],
                     "warm_us_min": warm_[1], "plain_launches_cold_us_median": plain[0], "plain_launches_cold_us_min": plain[1],
                     "tflops": roofline.fp8_flops(M, N, K) / cold[0] / 1e6, "roof_us": r_m,
                     "roof_us_datasheet": r_s, "pct_roofline": 100.0 * r_m / cold[0],
                     "pct_roofline_datasheet": 100.0 * r_s / cold[0], "pct_roofline_plain_launches": 100.0 * r_m / plain[0],
                     "fp8_cold_us_median": cold[0], "speedup_vs_fp8": 1.0})
        del p, case
        torch.cuda.empty_cache()

    for M in (16, 128, 2048, 8192):
        osc_row("qkv", M, 4096, 6144, 2, 0)
    for M in (128, 2048, 8192):
        osc_row("gate_up", M, 4096, 24576, 1, 0)
    for M in (128, 2048, 8192):
        fp8_row("down", M, 12288, 4096, 0)
    osc_row("layer.qkv", 4096, 4096, 6144, 2, 1)
    osc_row("layer.o_proj", 4096, 4096, 4096, 1, 2)
    osc_row("layer.gate_up", 4096, 4096, 24576, 1, 3)
    fp8_row("layer.down", 4096, 12288, 4096, 4)

    # grouped (MoE): 128 experts, top-8 of 8192 tokens, Zipf(1.1) load; one set of buffers is 0.7 GB, several times
    # the L2, so the cold and the warm regime coincide and are reported as one
    counts = synth.zipf_expert_rows()
    E, Mt = counts.size, int(counts.sum())
    off = torch.from_numpy(synth.offsets_from_counts(counts)).cuda()
    K, N = 2048, 1536
    c = synth.osc_linear_case_torch(torch, 5, Mt, K, N, 1)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(6)
    Wg = (0.02 * torch.randn(E, N, K, generator=gen, device="cuda", dtype=torch.float32)).to(torch.bfloat16)
    w = B.osc_prepare_weights_grouped(Wg, c["lut"])
    ws = torch.empty(B.osc_act_sizes(w, Mt).workspace_bytes, dtype=torch.uint8, device="cuda")
    Y = torch.empty(Mt, N, dtype=torch.bfloat16, device="cuda")
    settle()
    t = stats(per_call_times(torch, lambda i: B.osc_linear_grouped(w, c["X"], off, Y, ws), iters, warm, 4))
    settle()
    tp = stats(per_call_times(torch, lambda i: B.osc_linear_grouped(w, c["X"], off, Y, ws), iters, warm))
    w8 = B.osc_fp8_prepare_weights_grouped(Wg)
    ws8 = torch.empty(B.osc_fp8_act_sizes(w8, Mt).workspace_bytes, dtype=torch.uint8, device="cuda")
    settle()
    t8 = stats(per_call_times(torch, lambda i: B.osc_fp8_linear_grouped(w8, c["X"], off, Y, ws8), iters, warm, 4))
    B.osc_sync_check()
    f4, f16 = roofline.osc_flops(Mt, N, K, w.K_o)
    byts = 2.0 * Mt * K + E * (N * K / 2 + N * K / 32 + 2.0 * N * w.K_o) + 2.0 * Mt * N
    r_m, r_s = (max(f4 / pkx["fp4"] + f16 / pkx["bf16"], byts / pkx["hbm"]) * 1e6 for pkx in (meas, sheet))
    rows.append({"name": "moe.gate_up(grouped)", "path": "osc", "M": Mt, "K": K, "N": N, "K_o": w.K_o, "E": E,
                 "timing": "cuda graph replay of 4 calls per timed iteration; one buffer set larger than the L2 (cold = warm)", "sets": 1,
                 "cold_us_median": t[0], "cold_us_min": t[1], "warm_us_median": t[0], "warm_us_min": t[1],
                 "plain_launches_cold_us_median": tp[0], "plain_launches_cold_us_min": tp[1],
                 "pct_roofline_plain_launches": 100.0 * r_m / tp[0],
                 "tflops": (f4 + f16) / t[0] / 1e6, "roof_us": r_m, "roof_us_datasheet": r_s,
                 "pct_roofline": 100.0 * r_m / t[0], "pct_roofline_datasheet": 100.0 * r_s / t[0],
                 "fp8_cold_us_median": t8[0], "speedup_vs_fp8": t8[0] / t[0]})
    del w, ws, Y, w8, ws8, Wg, c
    torch.cuda.empty_cache()
    K, N = 768, 2048
    Xd = synth.student_t3_torch(torch, gen, (Mt, K))
    Wg = (0.02 * torch.randn(E, N, K, generator=gen, device="cuda", dtype=torch.float32)).to(torch.bfloat16)
    w8 = B.osc_fp8_prepare_weights_grouped(Wg)
    ws8 = torch.empty(B.osc_fp8_act_sizes(w8, Mt).workspace_bytes, dtype=torch.uint8, device="cuda")
    Y = torch.empty(Mt, N, dtype=torch.bfloat16, device="cuda")
    settle()
    t = stats(per_call_times(torch, lambda i: B.osc_fp8_linear_grouped(w8, Xd, off, Y, ws8), iters, warm, 4))
    settle()
    tp = stats(per_call_times(torch, lambda i: B.osc_fp8_linear_grouped(w8, Xd, off, Y, ws8), iters, warm))
    B.osc_sync_check()
    byts = 2.0 * Mt * K + E * (N * K + 4.0 * N) + 2.0 * Mt * N
    r_m, r_s = (max(roofline.fp8_flops(Mt, N, K) / pkx["fp8"], byts / pkx["hbm"]) * 1e6 for pkx in (meas, sheet))
    rows.append({"name": "moe.down(grouped)", "path": "fp8 fallback (is the own FP8 W8A8 linear)", "M": Mt, "K": K, "N": N, "E": E,
                 "timing": "cuda graph replay of 4 calls per timed iteration; one buffer set larger than the L2 (cold = warm)", "sets": 1,
                 "cold_us_median": t[0], "cold_us_min": t[1], "warm_us_median": t[0], "warm_us_min": t[1],
                 "plain_launches_cold_us_median": tp[0], "plain_launches_cold_us_min": tp[1],
                 "pct_roofline_plain_launches": 100.0 * r_m / tp[0],
                 "tflops": roofline.fp8_flops(Mt, N, K) / t[0] / 1e6, "roof_us": r_m, "roof_us_datasheet": r_s,
                 "pct_roofline": 100.0 * r_m / t[0], "pct_roofline_datasheet": 100.0 * r_s / t[0],
                 "fp8_cold_us_median": t[0], "speedup_vs_fp8": 1.0})
    del w8, ws8, Y, Wg, Xd
    torch.cuda.empty_cache()
    return rows



def run_gpu(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2604_12782_b200 import binding as B   # raises if the CUDA library is missing

    pk = load_peaks()
    peaks = roofline.peaks(pk["bf16_tflops"], pk["hbm_gbs"])
    M, K, N = WORKLOAD["M"], WORKLOAD["K"], WORKLOAD["N"]
    case = synth.osc_linear_case(rank, M, K, N, WORKLOAD["ch_per_group"])   # replicas: one seed per rank
    prob = OscProblem(torch, B, case, NSETS)
    Ko, Kop = prob.K_o, prob.K_o_pad
    torch.cuda.synchronize()
    B.osc_sync_check()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()      # already sampling when the timed region begins (the first NVML query takes milliseconds)
    # ---- timed region: K steps of osc_linear, inputs resident in HBM
    for i in range(args.warmup):
        prob.step(i)
    barrier()
    sampler.mark("t0")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        prob.step(i)
    e1.record()
    barrier()
    sampler.mark("t1")
    ms = e0.elapsed_time(e1) / args.steps
    # ---- same steps again with events between the two kernels (roofline of each kernel)
    tq, tg = time_split(torch, prob, args.steps)
    # ---- and the dominant kernel alone, launched back to back over the rotating buffer sets (operands cold in L2):
    # its average launch duration without the launch gap and the lost overlap that an event in front of it costs
    tg_loop = time_loop(torch, prob.gemm, args.steps, 3)
    # the quantizer the same way (its outputs land in the rotating workspaces; nothing reads them here)
    tq_loop = time_loop(torch, prob.quant, args.steps, 3)
    B.osc_sync_check()

    ms = max_over_ranks(ms, torch.device("cuda", local))
    if args.only_osc:
        sampler.stop()
        print(f"osc_linear {ms:.4f} ms/step (quantizer {tq:.4f} / {tq_loop:.4f} back to back, gemm {tg:.4f} / {tg_loop:.4f})",
              file=sys.stderr)
        return

    flops4, flops16 = roofline.osc_flops(M, N, K, Ko)
    flops = flops4 + flops16
    value = whole_job_value(flops, world, ms)

    # ---- end to end through the C ABI with host buffers (copies inside the timed region)
    Xh = torch.from_numpy(case["X"].view(np.int16)).view(torch.bfloat16).pin_memory()
    Yh = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
    # Rows are independent, so the step is cut into row chunks and pipelined over three streams: upload of chunk
    # c+1, osc_linear on chunk c and download of chunk c-1 overlap (PCIe is full duplex; the link, not the GPU,
    # bounds this number).  Every chunk goes through the same public call with its own slice of the workspace.
    # Two sets of device buffers alternate between steps, so that the uploads of step i+1 run while the last
    # downloads of step i are still on the link; a step's compute starts only when the previous step's results are
    # all back in host memory, and the timed region ends after the last download.
    CH = 8
    rows_c = (M + CH - 1) // CH
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    sz_c = B.osc_act_sizes(prob.w[0], rows_c)
    Xd2, Yd2 = [prob.X[0], prob.X[1]], [prob.Y[0], prob.Y[1]]
    ws_c = [[torch.empty(sz_c.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(CH)] for _ in range(2)]
    ev_in = [[torch.cuda.Event() for _ in range(CH)] for _ in range(2)]
    ev_done = [[torch.cuda.Event() for _ in range(CH)] for _ in range(2)]
    ev_free = [torch.cuda.Event() for _ in range(2)]   # the compute that last read Xd2[p] has finished

    def e2e_step(i):
        p = i % 2
        Xd, Yd = Xd2[p], Yd2[p]
        cur = torch.cuda.current_stream()
        s_in.wait_event(ev_free[p])
        for c in range(CH):
            r0, r1 = c * rows_c, min(M, (c + 1) * rows_c)
            with torch.cuda.stream(s_in):
                Xd[r0:r1].copy_(Xh[r0:r1], non_blocking=True)
                ev_in[p][c].record(s_in)
            cur.wait_event(ev_in[p][c])
            B.osc_linear(prob.w[0], Xd[r0:r1], Yd[r0:r1], ws_c[p][c])
            ev_done[p][c].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[p][c])
                Yh[r0:r1].copy_(Yd[r0:r1], non_blocking=True)
        ev_free[p].record(cur)
        cur.wait_stream(s_out)         # the step ends when its last rows are back in host memory

    torch.cuda.synchronize()
    e2e_steps = max(3, min(args.steps, 20))
    ms_e2e = time_loop(torch, e2e_step, e2e_steps, 3)
    ms_e2e = max_over_ranks(ms_e2e, torch.device("cuda", local))
    e2e_value = whole_job_value(flops, world, ms_e2e)

    # ---- the same build's FP8 W8A8 linear on the same shape (the paper's comparison point)
    f8case = {"X": case["X"], "W": case["W"], "M": M, "K": K, "N": N}
    f8 = Fp8Problem(torch, B, f8case, NSETS)
    ms_f8 = time_loop(torch, f8.step, args.steps, args.warmup)
    f8q, f8g = time_split(torch, f8, args.steps)
    B.osc_sync_check()
    del f8
    torch.cuda.empty_cache()
    configs = None
    if world == 1 and not args.no_configs:
        configs = config_rows(torch, B, pk)
    clocks = sampler.stop()
    if clocks.get("sm_mhz_in_timed_region"):
        clocks["ms_per_step_x_sm_mhz"] = ms * clocks["sm_mhz_in_timed_region"]

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # roofline of the dominant kernel (dual-path GEMM): tensor peak of its own FLOP mix
    p_mix = flops / (flops4 / peaks["fp4"] + flops16 / peaks["bf16"]) / 1e12
    gemm_tflops = flops / (tg_loop * 1e-3) / 1e12
    sheet = roofline.peaks(DATASHEET["bf16_tflops"], DATASHEET["hbm_gbs"])
    p_mix_sheet = flops / (flops4 / sheet["fp4"] + flops16 / sheet["bf16"]) / 1e12
    traffic, traffic_src = load_traffic()
    roof = {"bound": "tensor", "kernel": "gemm_pair_kernel<MODE_OSC> (dual-path GEMM, Eq. 5)", "achieved": gemm_tflops, "peak": p_mix,
            "unit": "TFLOP/s", "frac": gemm_tflops / p_mix, "traffic": traffic,
            "traffic_source": ({k: traffic_src.get(k) for k in ("commit", "captured", "command")} if traffic_src else None),
            "peak_basis": f"{pk['source']} bf16 {pk['bf16_tflops']} TFLOP/s x4 for FP4 (burst), FLOP-mix weighted",
            "frac_of_datasheet_peak": gemm_tflops / p_mix_sheet, "datasheet_peak": p_mix_sheet,
            "ms": tg_loop, "timing": "average over back-to-back launches between two events, rotating buffer sets",
            "frac_of_sustained_peak": (gemm_tflops / (p_mix * pk["bf16_tflops_sustained"] / pk["bf16_tflops"])
                                       if pk.get("bf16_tflops_sustained") else None),
            "ms_between_events_inside_the_step": tg}
    qbytes = roofline.quantize_extract_bytes(M, K, Kop)
    t_roof = roofline.osc_roofline_seconds(M, N, K, Ko, peaks)
    t_roof_sheet = roofline.osc_roofline_seconds(M, N, K, Ko, sheet)
    extra = {
        "pct_dual_path_roofline": 100.0 * t_roof / (ms * 1e-3),
        "roofline_us": t_roof * 1e6,
        "pct_dual_path_roofline_datasheet": 100.0 * t_roof_sheet / (ms * 1e-3),
        "roofline_us_datasheet": t_roof_sheet * 1e6,
        "peaks": {"measured": {"bf16_tflops": pk["bf16_tflops"], "fp8_tflops": 2 * pk["bf16_tflops"],
                               "fp4_tflops": 4 * pk["bf16_tflops"], "hbm_gbs": pk["hbm_gbs"], "source": pk["source"]},
                  "datasheet": {"bf16_tflops": 2250.0, "fp8_tflops": 4500.0, "fp4_tflops": 9000.0, "hbm_gbs": 8000.0}},
        "quant_extract": {"ms": tq_loop, "bytes": qbytes, "gbs": qbytes / (tq_loop * 1e-3) / 1e9,
                          "frac_hbm": qbytes / (tq_loop * 1e-3) / peaks["hbm"],
                          "frac_hbm_datasheet": qbytes / (tq_loop * 1e-3) / sheet["hbm"],
                          "timing": "average over back-to-back launches between two events, rotating buffer sets",
                          "ms_between_events_inside_the_step": tq},
        "fp8_linear": {"ms": ms_f8, "quant_ms": f8q, "gemm_ms": f8g,
                       "tflops": roofline.fp8_flops(M, N, K) / (ms_f8 * 1e-3) / 1e12,
                       "gemm_frac_fp8_peak": roofline.fp8_flops(M, N, K) / (f8g * 1e-3) / peaks["fp8"]},
        "speedup_vs_own_fp8_linear": ms_f8 / ms,
        "speedup_vs_own_fp8_gemm_only": f8g / tg,
        "paper_analytic_speedup_vs_w8a8": roofline.analytic_speedup_vs_w8a8(32, WORKLOAD["ch_per_group"]),
        "configs": configs,
    }

    cpu = None
    if world == 1 and not args.no_cpu:
        import oracle
        oracle.build()
        rows = args.cpu_rows
        wts = oracle.prepare_weights(case["W"], case["lut"])
        t0 = time.perf_counter()
        oracle_sample_step(oracle, case, wts, rows)
        dt = time.perf_counter() - t0
        cpu = {"value": 2.0 * rows * N * (K + Ko) / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(),
               "kind": "oracle", "seconds": dt,
               "sample": f"first {rows} of {M} activation rows x all N={N} (Algorithm 2 + Eq. 5; weights prepared once)"}

    line = {"metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp4(e2m1)+e8m0 x bf16 branch, fp32 accumulate", "data": "synthetic",
            "config": {"workload": WORKLOAD["name"], "M": M, "K": K, "N": N, "K_o": Ko,
                       "l2": f"rotating {NSETS} buffer sets (inputs, weights, workspace, outputs)",
                       "parallelism": "replicas only" if world > 1 else "1 gpu"},
            "roofline": roof, "cpu_baseline": cpu,
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "ms_per_step": ms_e2e, "row_chunks": CH,
                    "h2d_bytes_per_step": int(Xh.numel() * 2), "d2h_bytes_per_step": int(Yh.numel() * 2)},
            "gpu_launches": 2 * args.steps, "clocks": clocks, "extra": extra}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# -------------------------------------------------------------------------------- sweep
def run_sweep(args):
    """All benchmark shapes: OSC linears vs own FP8 on the same shape, FP8 down projection, MoE."""
    import torch
    from paper_2604_12782_b200 import binding as B
    torch.cuda.set_device(0)
    pk = load_peaks()
    peaks = roofline.peaks(pk["bf16_tflops"], pk["hbm_gbs"])
    rows = []
    steps, warm = args.steps, args.warmup

    def want(name):
        return not args.sweep_only or args.sweep_only in name

    def osc_row(name, M, K, N, cpg, seed=0):
        if not want(name):
            return
        case = synth.osc_linear_case(seed, M, K, N, cpg)
        nsets = NSETS if M >= 1024 else 8
        p = OscProblem(torch, B, case, nsets)
        ms = time_loop(torch, p.step, steps, warm)
        tq, tg = time_split(torch, p, steps)
        f8 = Fp8Problem(torch, B, case, nsets)
        ms8 = time_loop(torch, f8.step, steps, warm)
        q8, g8 = time_split(torch, f8, steps)
        B.osc_sync_check()
        f4, f16 = roofline.osc_flops(M, N, K, p.K_o)
        troof = roofline.osc_roofline_seconds(M, N, K, p.K_o, peaks)
        extra = {}
        if M <= 128:   # few rows: the plain loop above is paced by the host; also replay from a CUDA graph
            gms, gms8 = time_graph(torch, p.step, 48), time_graph(torch, f8.step, 48)
            extra = {"graph_ms": gms, "fp8_graph_ms": gms8, "pct_roofline_graph": 100 * troof / (gms * 1e-3),
                     "speedup_vs_fp8_graph": gms8 / gms}
        rows.append({**extra, "name": name, "M": M, "K": K, "N": N, "K_o": p.K_o, "ms": ms, "quant_ms": tq, "gemm_ms": tg,
                     "tflops": (f4 + f16) / ms / 1e9, "pct_roofline": 100 * troof / (ms * 1e-3),
                     "roof_us": troof * 1e6, "fp8_ms": ms8, "fp8_quant_ms": q8, "fp8_gemm_ms": g8,
                     "speedup_vs_fp8": ms8 / ms, "speedup_gemm_only": g8 / tg,
                     "quant_gbs": roofline.quantize_extract_bytes(M, K, p.K_o_pad) / tq / 1e6})
        del p, f8
        torch.cuda.empty_cache()

    def rms_row(name, M, K, N, cpg, seed=0):
        """RMSNorm in front of the OSC linear: fused into the quantizer against the two-step path (own RMSNorm kernel
        writing bf16, then the stand-alone quantizer); the residual stream stands in for X."""
        if not want(name):
            return
        case = synth.osc_linear_case(seed, M, K, N, cpg)
        p = OscProblem(torch, B, case, NSETS)
        gam = dev_bf16(torch, synth.f32_to_bf16_bits(np.random.default_rng(seed).uniform(0.5, 1.5, K).astype(np.float32)))
        Xn = [torch.empty(M, K, dtype=torch.bfloat16, device="cuda") for _ in range(p.n)]
        eps = 1e-6

        def fused_q(i):
            j = i % p.n
            B.osc_rmsnorm_quantize_extract(p.w[j], p.X[j], gam, eps, *p.views(j))

        def norm_only(i):
            j = i % p.n
            B.osc_rmsnorm(p.X[j], gam, eps, Xn[j])

        def two_step_q(i):
            j = i % p.n
            B.osc_rmsnorm(p.X[j], gam, eps, Xn[j])
            B.osc_quantize_extract(p.w[j], Xn[j], *p.views(j))

        def fused_lin(i):
            j = i % p.n
            B.osc_rmsnorm_linear(p.w[j], p.X[j], gam, eps, p.Y[j], p.ws[j])

        def two_step_lin(i):
            j = i % p.n
            B.osc_rmsnorm(p.X[j], gam, eps, Xn[j])
            B.osc_linear(p.w[j], Xn[j], p.Y[j], p.ws[j])

        # with the residual update in front of the norm (h' = h + r written to a scratch stream, so nothing drifts)
        Rr = [torch.roll(p.X[j], 7, 0).contiguous() for j in range(p.n)]
        Hn = torch.empty(M, K, dtype=torch.bfloat16, device="cuda")

        def fused_add_q(i):
            j = i % p.n
            B.osc_add_rmsnorm_quantize_extract(p.w[j], p.X[j], Rr[j], gam, eps, Hn, *p.views(j))

        def fused_add_lin(i):
            j = i % p.n
            B.osc_add_rmsnorm_linear(p.w[j], p.X[j], Rr[j], gam, eps, Hn, p.Y[j], p.ws[j])

        def two_step_add_lin(i):
            j = i % p.n
            B.osc_add_rmsnorm(p.X[j], Rr[j], gam, eps, Hn, Xn[j])
            B.osc_linear(p.w[j], Xn[j], p.Y[j], p.ws[j])

        t = {k: time_loop(torch, f, steps, warm) for k, f in
             (("fused_quant_ms", fused_q), ("norm_ms", norm_only), ("two_step_quant_ms", two_step_q),
              ("fused_linear_ms", fused_lin), ("two_step_linear_ms", two_step_lin),
              ("add_fused_quant_ms", fused_add_q), ("add_fused_linear_ms", fused_add_lin),
              ("add_two_step_linear_ms", two_step_add_lin))}
        B.osc_sync_check()
        byts = roofline.quantize_extract_bytes(M, K, p.K_o_pad)   # one read of the rows + the quantizer's outputs
        t["add_fused_quant_frac_hbm"] = (byts + 4.0 * M * K) / (t["add_fused_quant_ms"] * 1e-3) / peaks["hbm"]
        rows.append({"name": name, "M": M, "K": K, "N": N, "K_o": p.K_o, **t, "ms": t["fused_linear_ms"],
                     "fused_quant_gbs": byts / t["fused_quant_ms"] / 1e6,
                     "fused_quant_frac_hbm": byts / (t["fused_quant_ms"] * 1e-3) / peaks["hbm"],
                     "speedup_linear": t["two_step_linear_ms"] / t["fused_linear_ms"]})
        del p, Xn, Rr, Hn
        torch.cuda.empty_cache()

    def profile_row(name, S, K, seed=0):
        """Algorithm 1 (offline): threshold of Eq. 1 over the slice, per-token per-group vote, table and Eq. 2-4 counters.
        Two passes over the activations (the threshold needs the whole slice first): 2 x 2 bytes per element."""
        if not want(name):
            return
        Xb, _ = synth.osc_activations_only(seed, S, K, 1)
        X0 = dev_bf16(torch, Xb)
        n = NSETS
        Xs = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(n)]
        scratch = torch.empty(B.osc_profile_scratch_bytes(K), dtype=torch.uint8, device="cuda")
        lut = torch.empty(K // 32, dtype=torch.int8, device="cuda")
        nh, nt = (torch.empty(K // 32, dtype=torch.int32, device="cuda") for _ in range(2))
        tb = torch.empty(1, dtype=torch.int32, device="cuda")
        ms = time_loop(torch, lambda i: B.osc_profile_lut(Xs[i % n], 5.0, scratch, lut, nh, nt, tb), steps, warm)
        B.osc_sync_check()
        byts = 2 * 2.0 * S * K
        rows.append({"name": name, "M": S, "K": K, "ms": ms, "gbs": byts / ms / 1e6,
                     "frac_hbm": byts / (ms * 1e-3) / peaks["hbm"], "roof_us": byts / peaks["hbm"] * 1e6,
                     "pct_roofline": 100 * byts / peaks["hbm"] / (ms * 1e-3)})
        del Xs
        torch.cuda.empty_cache()

    def swiglu_row(name, M, I, N, seed=0):
        """SwiGLU in front of the FP8 down projection: fused into the per-token quantizer against the two-step path (own
        SwiGLU kernel writing bf16, then the stand-alone FP8 quantizer)."""
        if not want(name):
            return
        rng = np.random.default_rng(seed)
        case = synth.fp8_linear_case(seed, 1, I, N)
        n = NSETS
        GU0 = dev_bf16(torch, synth.f32_to_bf16_bits(np.concatenate(
            [rng.standard_normal((M, I), dtype=np.float32) * 3.0, rng.standard_normal((M, I), dtype=np.float32)], axis=1)))
        GUs = [GU0 if i == 0 else torch.roll(GU0, 97 * i, 0).contiguous() for i in range(n)]
        W0 = dev_bf16(torch, case["W"])
        ws_ = [B.osc_fp8_prepare_weights(W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous()) for i in range(n)]
        sz = B.osc_fp8_act_sizes(ws_[0], M)
        wk = [torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
        Hs = [torch.empty(M, I, dtype=torch.bfloat16, device="cuda") for _ in range(n)]
        Ys = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(n)]

        def fused_q(i):
            j = i % n
            B.osc_swiglu_fp8_quantize(GUs[j], I, wk[j][sz.x8_offset:], wk[j][sz.sx_offset:])

        def act_only(i):
            j = i % n
            B.osc_swiglu(GUs[j], I, Hs[j])

        def two_step_q(i):
            j = i % n
            B.osc_swiglu(GUs[j], I, Hs[j])
            B.osc_fp8_quantize(Hs[j], wk[j][sz.x8_offset:], wk[j][sz.sx_offset:])

        def fused_lin(i):
            j = i % n
            B.osc_swiglu_fp8_linear(ws_[j], GUs[j], Ys[j], wk[j])

        def two_step_lin(i):
            j = i % n
            B.osc_swiglu(GUs[j], I, Hs[j])
            B.osc_fp8_linear(ws_[j], Hs[j], Ys[j], wk[j])

        t = {k: time_loop(torch, f, steps, warm) for k, f in
             (("fused_quant_ms", fused_q), ("swiglu_ms", act_only), ("two_step_quant_ms", two_step_q),
              ("fused_linear_ms", fused_lin), ("two_step_linear_ms", two_step_lin))}
        B.osc_sync_check()
        byts = 2.0 * M * 2 * I + 1.0 * M * I + 4.0 * M     # gate and up read once, codes and scales written
        rows.append({"name": name, "M": M, "K": I, "N": N, **t, "ms": t["fused_linear_ms"],
                     "fused_quant_gbs": byts / t["fused_quant_ms"] / 1e6,
                     "fused_quant_frac_hbm": byts / (t["fused_quant_ms"] * 1e-3) / peaks["hbm"],
                     "speedup_linear": t["two_step_linear_ms"] / t["fused_linear_ms"]})
        del GUs, ws_, wk, Hs, Ys
        torch.cuda.empty_cache()

    def fp8_row(name, M, K, N, seed=0):
        if not want(name):
            return
        case = synth.fp8_linear_case(seed, M, K, N)
        nsets = NSETS if M >= 1024 else 8
        f8 = Fp8Problem(torch, B, case, nsets)
        ms8 = time_loop(torch, f8.step, steps, warm)
        q8, g8 = time_split(torch, f8, steps)
        B.osc_sync_check()
        troof = roofline.fp8_roofline_seconds(M, N, K, peaks)
        extra = {}
        if M <= 128:
            gms8 = time_graph(torch, f8.step, 48)
            extra = {"graph_ms": gms8, "pct_roofline_graph": 100 * troof / (gms8 * 1e-3)}
        rows.append({**extra, "name": name, "M": M, "K": K, "N": N, "ms": ms8, "quant_ms": q8, "gemm_ms": g8,
                     "tflops": roofline.fp8_flops(M, N, K) / ms8 / 1e9, "pct_roofline": 100 * troof / (ms8 * 1e-3),
                     "roof_us": troof * 1e6, "quant_gbs": roofline.fp8_quantize_bytes(M, K) / q8 / 1e6})
        del f8
        torch.cuda.empty_cache()

    def mxfp8_row(name, M, K, N, seed=0):
        if not want(name):
            return
        case = synth.fp8_linear_case(seed, M, K, N)
        nsets = NSETS if M >= 1024 else 8
        p8 = Mxfp8Problem(torch, B, case, nsets)
        ms8 = time_loop(torch, p8.step, steps, warm)
        q8, g8 = time_split(torch, p8, steps)
        B.osc_sync_check()
        # same FLOPs and FP8 peak as the per-token form; bytes: X, W8 + its scales, Y (+ the two-kernel intermediates
        # are implementation traffic, not counted)
        byts = 2.0 * M * K + N * K * (1 + 1 / 32) + 2.0 * M * N
        troof = max(roofline.fp8_flops(M, N, K) / peaks["fp8"], byts / peaks["hbm"])
        rows.append({"name": name, "M": M, "K": K, "N": N, "ms": ms8, "quant_ms": q8, "gemm_ms": g8,
                     "tflops": roofline.fp8_flops(M, N, K) / ms8 / 1e9, "pct_roofline": 100 * troof / (ms8 * 1e-3),
                     "roof_us": troof * 1e6, "quant_gbs": (2.0 * M * K + M * K * (1 + 1 / 32)) / q8 / 1e6})
        del p8
        torch.cuda.empty_cache()

    def dyn_row(name, M, K, N, cpg, seed=0):
        """The dynamic-protection control group (run-time per-group maximum) on the shape of an OSC row."""
        if not want(name):
            return
        case = synth.osc_linear_case(seed, M, K, N, cpg)
        X0, W0 = dev_bf16(torch, case["X"]), dev_bf16(torch, case["W"])
        n = NSETS
        Xs = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(n)]
        ws_ = [B.osc_dyn_prepare_weights(W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous()) for i in range(n)]
        sz = B.osc_dyn_act_sizes(ws_[0], M)
        wk = [torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
        Ys = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(n)]
        ms = time_loop(torch, lambda i: B.osc_dyn_linear(ws_[i % n], Xs[i % n], Ys[i % n], wk[i % n]), steps, warm)
        tq = time_loop(torch, lambda i: B.osc_dyn_quantize_extract(
            ws_[i % n], Xs[i % n], wk[i % n][sz.xq_offset:], wk[i % n][sz.sfa_offset:], wk[i % n][sz.xo_offset:],
            wk[i % n][sz.idx_offset:], wk[i % n][sz.val_offset:]), steps, warm)
        B.osc_sync_check()
        rows.append({"name": name, "M": M, "K": K, "N": N, "ms": ms, "quant_ms": tq,
                     "note": "high-precision branch over all K channels (one non-zero per 32), weights unzeroed"})
        del ws_, wk, Ys, Xs
        torch.cuda.empty_cache()

    def nvfp4_row(name, M, K, N, seed=0):
        """OSC on NVFP4 (blocks of 16, one flagged channel per block: K_o = K/16, as large as two per 32)."""
        if not want(name):
            return
        case = synth.osc16_linear_case(seed, M, K, N)
        ex, ew = synth.nvfp4_tensor_exponent(case["X"]), synth.nvfp4_tensor_exponent(case["W"])
        X0, W0 = dev_bf16(torch, case["X"]), dev_bf16(torch, case["W"])
        n = NSETS
        Xs = [X0 if i == 0 else torch.roll(X0, 97 * i, 0).contiguous() for i in range(n)]
        ws_ = [B.osc_nvfp4_prepare_weights(W0 if i == 0 else torch.roll(W0, 61 * i, 0).contiguous(), case["lut16"], ew)
               for i in range(n)]
        sz = B.osc_nvfp4_act_sizes(ws_[0], M)
        wk = [torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda") for _ in range(n)]
        Ys = [torch.empty(M, N, dtype=torch.bfloat16, device="cuda") for _ in range(n)]
        ms = time_loop(torch, lambda i: B.osc_nvfp4_linear(ws_[i % n], Xs[i % n], ex, Ys[i % n], wk[i % n]), steps, warm)
        tq = time_loop(torch, lambda i: B.osc_nvfp4_quantize_extract(
            ws_[i % n], Xs[i % n], ex, wk[i % n][sz.xq_offset:], wk[i % n][sz.sfa_offset:], wk[i % n][sz.xo_offset:]),
            steps, warm)
        tg = time_loop(torch, lambda i: B.osc_nvfp4_gemm(
            ws_[i % n], wk[i % n][sz.xq_offset:], wk[i % n][sz.sfa_offset:], wk[i % n][sz.xo_offset:], M, ex, Ys[i % n]),
            steps, warm)
        B.osc_sync_check()
        Ko = ws_[0].K_o
        f4, f16 = roofline.osc_flops(M, N, K, Ko)
        troof = roofline.osc_roofline_seconds(M, N, K, Ko, peaks)
        rows.append({"name": name, "M": M, "K": K, "N": N, "K_o": Ko, "ms": ms, "quant_ms": tq, "gemm_ms": tg,
                     "tflops": (f4 + f16) / ms / 1e9, "pct_roofline": 100 * troof / (ms * 1e-3), "roof_us": troof * 1e6})
        del ws_, wk, Ys, Xs
        torch.cuda.empty_cache()

    for M in (16, 64, 128, 2048, 8192):
        osc_row("qkv", M, 4096, 6144, 2)
    for M in (16, 64, 128, 2048, 8192):
        osc_row("gate_up", M, 4096, 24576, 1)
        fp8_row("down_fp8", M, 12288, 4096)
        mxfp8_row("down_mxfp8", M, 12288, 4096)
    rms_row("qkv.rmsnorm_fused", 8192, 4096, 6144, 2)
    rms_row("qkv.rmsnorm_fused", 2048, 4096, 6144, 2)
    swiglu_row("down.swiglu_fused", 8192, 12288, 4096)
    swiglu_row("down.swiglu_fused", 2048, 12288, 4096)
    profile_row("profile.algorithm1", 8192, 4096)
    nvfp4_row("qkv.nvfp4_g16", 8192, 4096, 6144)
    nvfp4_row("qkv.nvfp4_g16", 2048, 4096, 6144)
    dyn_row("qkv.dynamic_protection", 8192, 4096, 6144, 2)
    dyn_row("qkv.dynamic_protection", 2048, 4096, 6144, 2)
    osc_row("layer.qkv", 4096, 4096, 6144, 2)
    osc_row("layer.o_proj", 4096, 4096, 4096, 1)
    osc_row("layer.gate_up", 4096, 4096, 24576, 1)
    fp8_row("layer.down_fp8", 4096, 12288, 4096)

    # the four linears of one Qwen3-8B layer at M = 4096 back to back on one stream (independent tensors per linear):
    # what the programmatic dependent launches between consecutive kernels are worth
    if want("layer.chain"):
        M = 4096
        qkv = OscProblem(torch, B, synth.osc_linear_case(0, M, 4096, 6144, 2), 2)
        opj = OscProblem(torch, B, synth.osc_linear_case(1, M, 4096, 4096, 1), 2)
        gup = OscProblem(torch, B, synth.osc_linear_case(2, M, 4096, 24576, 1), 2)
        dwn = Fp8Problem(torch, B, synth.fp8_linear_case(3, M, 12288, 4096), 2)
        parts = [qkv, opj, gup, dwn]
        each = [time_loop(torch, p.step, steps, warm) for p in parts]

        def chain(i):
            for p in parts:
                p.step(i)
        ms = time_loop(torch, chain, steps, warm)
        gms = time_graph(torch, chain, 8)
        B.osc_sync_check()
        troof = (roofline.osc_roofline_seconds(M, 6144, 4096, qkv.K_o, peaks) + roofline.osc_roofline_seconds(M, 4096, 4096, opj.K_o, peaks)
                 + roofline.osc_roofline_seconds(M, 24576, 4096, gup.K_o, peaks) + roofline.fp8_roofline_seconds(M, 4096, 12288, peaks))
        rows.append({"name": "layer.chain(qkv,o_proj,gate_up,down_fp8)", "M": M, "ms": ms, "graph_ms": gms,
                     "sum_of_separate_ms": sum(each), "pct_roofline": 100 * troof / (ms * 1e-3), "roof_us": troof * 1e6})
        del parts, qkv, opj, gup, dwn
        torch.cuda.empty_cache()

    # the same layer with its producers: RMSNorm in front of QKV and gate/up, SwiGLU between gate/up and down (the down
    # projection really consumes the gate/up output); fused into the quantizers against separate kernels
    if want("layer.fused"):
        M, eps = 4096, 1e-6
        qkv = OscProblem(torch, B, synth.osc_linear_case(0, M, 4096, 6144, 2), 2)
        opj = OscProblem(torch, B, synth.osc_linear_case(1, M, 4096, 4096, 1), 2)
        gup = OscProblem(torch, B, synth.osc_linear_case(2, M, 4096, 24576, 1), 2)
        dwn = Fp8Problem(torch, B, synth.fp8_linear_case(3, M, 12288, 4096), 2)
        gam = dev_bf16(torch, synth.f32_to_bf16_bits(np.random.default_rng(0).uniform(0.5, 1.5, 4096).astype(np.float32)))
        Xn = torch.empty(M, 4096, dtype=torch.bfloat16, device="cuda")
        Hh = torch.empty(M, 12288, dtype=torch.bfloat16, device="cuda")

        def fused(i):
            j = i % 2
            B.osc_rmsnorm_linear(qkv.w[j], qkv.X[j], gam, eps, qkv.Y[j], qkv.ws[j])
            B.osc_linear(opj.w[j], opj.X[j], opj.Y[j], opj.ws[j])
            B.osc_rmsnorm_linear(gup.w[j], gup.X[j], gam, eps, gup.Y[j], gup.ws[j])
            B.osc_swiglu_fp8_linear(dwn.w[j], gup.Y[j], dwn.Y[j], dwn.ws[j])

        def separate(i):
            j = i % 2
            B.osc_rmsnorm(qkv.X[j], gam, eps, Xn)
            B.osc_linear(qkv.w[j], Xn, qkv.Y[j], qkv.ws[j])
            B.osc_linear(opj.w[j], opj.X[j], opj.Y[j], opj.ws[j])
            B.osc_rmsnorm(gup.X[j], gam, eps, Xn)
            B.osc_linear(gup.w[j], Xn, gup.Y[j], gup.ws[j])
            B.osc_swiglu(gup.Y[j], 12288, Hh)
            B.osc_fp8_linear(dwn.w[j], Hh, dwn.Y[j], dwn.ws[j])

        ms_f, ms_s = time_loop(torch, fused, steps, warm), time_loop(torch, separate, steps, warm)
        B.osc_sync_check()
        rows.append({"name": "layer.fused(rmsnorm+qkv,o_proj,rmsnorm+gate_up,swiglu+down_fp8)", "M": M, "ms": ms_f,
                     "separate_kernels_ms": ms_s, "speedup": ms_s / ms_f})
        # the same with the activation in the epilogue of the gate|up projection: the [M, 2I] matrix is never written,
        # the down projection's quantizer reads H [M, I]
        gu_w = [B.osc_prepare_weights_gate_up(torch.roll(dev_bf16(torch, synth.osc_linear_case(2, 1, 4096, 24576, 1)["W"]), 61 * j, 0).contiguous(),
                                              synth.osc_linear_case(2, 1, 4096, 24576, 1)["lut"]) for j in range(1)]
        gu_ws = torch.empty(B.osc_linear_swiglu_workspace_bytes(gu_w[0], M), dtype=torch.uint8, device="cuda")
        Hd = torch.empty(M, 12288, dtype=torch.bfloat16, device="cuda")

        def fused_epilogue(i):
            j = i % 2
            B.osc_rmsnorm_linear(qkv.w[j], qkv.X[j], gam, eps, qkv.Y[j], qkv.ws[j])
            B.osc_linear(opj.w[j], opj.X[j], opj.Y[j], opj.ws[j])
            B.osc_rmsnorm_linear_swiglu(gu_w[0], gup.X[j], gam, eps, Hd, gu_ws)
            B.osc_fp8_linear(dwn.w[j], Hd, dwn.Y[j], dwn.ws[j])

        ms_e = time_loop(torch, fused_epilogue, steps, warm)
        B.osc_sync_check()
        rows.append({"name": "layer.fused_epilogue(rmsnorm+qkv,o_proj,rmsnorm+gate_up+swiglu,down_fp8)", "M": M, "ms": ms_e,
                     "fused_quantizers_ms": ms_f, "separate_kernels_ms": ms_s, "speedup_vs_separate": ms_s / ms_e})
        del gu_w, gu_ws, Hd
        # the same with the two residual updates of the layer in the picture: h' = h + branch output in front of each
        # norm, written to a scratch stream so that the values do not drift over the timed iterations
        Hn = [torch.empty(M, 4096, dtype=torch.bfloat16, device="cuda") for _ in range(2)]

        def fused_res(i):
            j = i % 2
            B.osc_add_rmsnorm_linear(qkv.w[j], qkv.X[j], dwn.Y[j], gam, eps, Hn[0], qkv.Y[j], qkv.ws[j])
            B.osc_linear(opj.w[j], opj.X[j], opj.Y[j], opj.ws[j])
            B.osc_add_rmsnorm_linear(gup.w[j], gup.X[j], opj.Y[j], gam, eps, Hn[1], gup.Y[j], gup.ws[j])
            B.osc_swiglu_fp8_linear(dwn.w[j], gup.Y[j], dwn.Y[j], dwn.ws[j])

        def separate_res(i):
            j = i % 2
            B.osc_add_rmsnorm(qkv.X[j], dwn.Y[j], gam, eps, Hn[0], Xn)
            B.osc_linear(qkv.w[j], Xn, qkv.Y[j], qkv.ws[j])
            B.osc_linear(opj.w[j], opj.X[j], opj.Y[j], opj.ws[j])
            B.osc_add_rmsnorm(gup.X[j], opj.Y[j], gam, eps, Hn[1], Xn)
            B.osc_linear(gup.w[j], Xn, gup.Y[j], gup.ws[j])
            B.osc_swiglu(gup.Y[j], 12288, Hh)
            B.osc_fp8_linear(dwn.w[j], Hh, dwn.Y[j], dwn.ws[j])

        ms_f, ms_s = time_loop(torch, fused_res, steps, warm), time_loop(torch, separate_res, steps, warm)
        B.osc_sync_check()
        rows.append({"name": "layer.fused_with_residual(add+rmsnorm+qkv,o_proj,add+rmsnorm+gate_up,swiglu+down_fp8)", "M": M,
                     "ms": ms_f, "separate_kernels_ms": ms_s, "speedup": ms_s / ms_f})
        del qkv, opj, gup, dwn, Xn, Hh, Hn
        torch.cuda.empty_cache()

    # MoE: 128 experts, top-8 of 8192 tokens, Zipf(1.1) load
    counts = synth.zipf_expert_rows()
    E = counts.size
    off = torch.from_numpy(synth.offsets_from_counts(counts)).cuda()
    c = synth.moe_gate_up_case(E, counts, weight_pool=8)
    Xd = dev_bf16(torch, c["X"])
    Wd = dev_bf16(torch, c["W"].reshape(E * c["N"], c["K"])).view(E, c["N"], c["K"])
    w = B.osc_prepare_weights_grouped(Wd, c["lut"])
    sz = B.osc_act_sizes(w, c["M"])
    ws = torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda")
    Y = torch.empty(c["M"], c["N"], dtype=torch.bfloat16, device="cuda")
    ms = time_loop(torch, lambda i: B.osc_linear_grouped(w, Xd, off, Y, ws), steps, warm)
    B.osc_sync_check()
    Mt, K, N = c["M"], c["K"], c["N"]
    f4, f16 = roofline.osc_flops(Mt, N, K, w.K_o)
    byts = 2.0 * Mt * K + E * (N * K / 2 + N * K / 32 + 2.0 * N * w.K_o) + 2.0 * Mt * N
    troof = max(f4 / peaks["fp4"] + f16 / peaks["bf16"], byts / peaks["hbm"])
    rows.append({"name": "moe.gate_up(grouped)", "M": Mt, "K": K, "N": N, "K_o": w.K_o, "ms": ms,
                 "tflops": (f4 + f16) / ms / 1e9, "pct_roofline": 100 * troof / (ms * 1e-3), "roof_us": troof * 1e6})
    # the same layer with the dispatch fused behind the quantizer: 8192 tokens quantized once, their quantized rows
    # gathered to the 65536 (token, expert) rows; the caller never builds the permuted bf16 matrix
    T_tok = Mt // 8
    Xtok = Xd[:T_tok].contiguous()
    row_token = torch.from_numpy(np.random.default_rng(0).integers(0, T_tok, size=Mt).astype(np.int32)).cuda()
    wsg = torch.empty(B.osc_gather_workspace_bytes(w, T_tok, Mt), dtype=torch.uint8, device="cuda")
    msg = time_loop(torch, lambda i: B.osc_linear_grouped_gather(w, Xtok, row_token, off, Y, wsg), steps, warm)
    B.osc_sync_check()
    bytsg = 2.0 * T_tok * K + E * (N * K / 2 + N * K / 32 + 2.0 * N * w.K_o) + 2.0 * Mt * N
    troofg = max(f4 / peaks["fp4"] + f16 / peaks["bf16"], bytsg / peaks["hbm"])
    rows.append({"name": "moe.gate_up(grouped, gathered from 8192 tokens)", "M": Mt, "K": K, "N": N, "K_o": w.K_o, "ms": msg,
                 "tflops": (f4 + f16) / msg / 1e9, "pct_roofline": 100 * troofg / (msg * 1e-3), "roof_us": troofg * 1e6,
                 "speedup_vs_permuted_input": ms / msg})
    # the same grouped problem on NVFP4 / G = 16 (the same protected channels, written as a table per 16-group)
    lut32 = np.asarray(c["lut"]).reshape(K // 32, -1)
    lut16 = np.full((K // 16, lut32.shape[1]), -1, np.int8)
    for g in range(K // 32):
        for j, ch in enumerate(lut32[g]):
            if ch >= 0:
                lut16[2 * g + (ch >= 16), j] = ch % 16
    ex4, ew4 = synth.nvfp4_tensor_exponent(c["X"]), synth.nvfp4_tensor_exponent(c["W"])
    w4 = B.osc_nvfp4_prepare_weights_grouped(Wd, lut16, ew4)
    ws4 = torch.empty(B.osc_nvfp4_act_sizes(w4, Mt).workspace_bytes, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    ms4 = time_loop(torch, lambda i: B.osc_nvfp4_linear_grouped(w4, Xd, off, ex4, Y, ws4), steps, warm)
    B.osc_sync_check()
    rows.append({"name": "moe.gate_up_nvfp4_g16(grouped)", "M": Mt, "K": K, "N": N, "K_o": w4.K_o, "ms": ms4,
                 "tflops": (f4 + f16) / ms4 / 1e9, "vs_mxfp4": ms4 / ms})
    del w4, ws4
    wg, Yg = w, Y
    wgu = B.osc_prepare_weights_gate_up_grouped(Wd, c["lut"])     # the same experts with the SwiGLU in the epilogue
    wsgu = torch.empty(B.osc_swiglu_gather_workspace_bytes(wgu, T_tok, Mt), dtype=torch.uint8, device="cuda")
    del Xd, Wd, ws
    c = synth.moe_down_case(E, counts, weight_pool=8)
    Xd = dev_bf16(torch, c["X"])
    Wd = dev_bf16(torch, c["W"].reshape(E * c["N"], c["K"])).view(E, c["N"], c["K"])
    w = B.osc_fp8_prepare_weights_grouped(Wd)
    sz = B.osc_fp8_act_sizes(w, c["M"])
    ws = torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda")
    Y = torch.empty(c["M"], c["N"], dtype=torch.bfloat16, device="cuda")
    ms = time_loop(torch, lambda i: B.osc_fp8_linear_grouped(w, Xd, off, Y, ws), steps, warm)
    B.osc_sync_check()
    Mt, K, N = c["M"], c["K"], c["N"]
    byts = 2.0 * Mt * K + E * (N * K + 4.0 * N) + 2.0 * Mt * N
    troof = max(roofline.fp8_flops(Mt, N, K) / peaks["fp8"], byts / peaks["hbm"])
    rows.append({"name": "moe.down_fp8(grouped)", "M": Mt, "K": K, "N": N, "ms": ms,
                 "tflops": roofline.fp8_flops(Mt, N, K) / ms / 1e9, "pct_roofline": 100 * troof / (ms * 1e-3),
                 "roof_us": troof * 1e6})
    # the expert layer with its producers: RMSNorm of the 8192 tokens fused into the quantizer in front of the gather,
    # SwiGLU of the experts' gate|up rows fused into the FP8 quantizer in front of the down projection (I = 768)
    gamma = torch.ones(wg.K, dtype=torch.bfloat16, device="cuda")
    Xn = torch.empty_like(Xtok)
    Hh = torch.empty(Mt, K, dtype=torch.bfloat16, device="cuda")

    def moe_fused(i):
        B.osc_rmsnorm_linear_grouped_gather(wg, Xtok, gamma, 1e-6, row_token, off, Yg, wsg)
        B.osc_swiglu_fp8_linear_grouped(w, Yg, off, Y, ws)

    def moe_separate(i):
        B.osc_rmsnorm(Xtok, gamma, 1e-6, Xn)
        B.osc_linear_grouped_gather(wg, Xn, row_token, off, Yg, wsg)
        B.osc_swiglu(Yg, K, Hh)
        B.osc_fp8_linear_grouped(w, Hh, off, Y, ws)

    def moe_fused_epilogue(i):
        B.osc_rmsnorm_linear_swiglu_grouped_gather(wgu, Xtok, gamma, 1e-6, row_token, off, Hh, wsgu)
        B.osc_fp8_linear_grouped(w, Hh, off, Y, ws)

    ms_f, ms_s = time_loop(torch, moe_fused, steps, warm), time_loop(torch, moe_separate, steps, warm)
    ms_e = time_loop(torch, moe_fused_epilogue, steps, warm)
    B.osc_sync_check()
    rows.append({"name": "moe.layer.fused(rmsnorm+gather+gate_up, swiglu+down_fp8)", "M": Mt, "ms": ms_f,
                 "separate_kernels_ms": ms_s, "speedup": ms_s / ms_f})
    rows.append({"name": "moe.layer.fused_epilogue(rmsnorm+gather+gate_up+swiglu, down_fp8)", "M": Mt, "ms": ms_e,
                 "separate_kernels_ms": ms_s, "speedup": ms_s / ms_e})
    del w, ws, wg, wgu, wsgu, Yg, wsg, Xtok, Xn, Hh
    w = B.osc_mxfp8_prepare_weights_grouped(Wd)
    sz = B.osc_mxfp8_act_sizes(w, c["M"])
    ws = torch.empty(sz.workspace_bytes, dtype=torch.uint8, device="cuda")
    ms = time_loop(torch, lambda i: B.osc_mxfp8_linear_grouped(w, Xd, off, Y, ws), steps, warm)
    B.osc_sync_check()
    byts = 2.0 * Mt * K + E * N * K * (1 + 1 / 32) + 2.0 * Mt * N
    troof = max(roofline.fp8_flops(Mt, N, K) / peaks["fp8"], byts / peaks["hbm"])
    rows.append({"name": "moe.down_mxfp8(grouped)", "M": Mt, "K": K, "N": N, "ms": ms,
                 "tflops": roofline.fp8_flops(Mt, N, K) / ms / 1e9, "pct_roofline": 100 * troof / (ms * 1e-3),
                 "roof_us": troof * 1e6})

    out_dir = os.environ.get("OSC_BENCH_OUT", os.path.join(ROOT, "bench_out"))
    os.makedirs(out_dir, exist_ok=True)
    with open(os.path.join(out_dir, "sweep.json"), "w") as f:
        json.dump({"peaks": pk, "rows": rows}, f, indent=1)
    for r in rows:
        print(json.dumps(r), file=sys.stderr)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="osc", choices=["osc", "reference"])
    ap.add_argument("--no-cpu", action="store_true", help="skip the cpu_baseline leg")
    ap.add_argument("--no-configs", action="store_true", help="skip extra.configs (the rows per benchmark shape)")
    ap.add_argument("--cpu-rows", type=int, default=8192, help="activation rows of the cpu_baseline sample")
    ap.add_argument("--ref-rows", type=int, default=128, help="activation rows per step of --impl reference")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--sweep-only", default="", help="with --sweep: only the rows whose name contains this text")
    ap.add_argument("--only-osc", action="store_true",
                    help="skip the e2e, FP8 and cpu legs (short runs under a profiler; prints no bench line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "osc" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.sweep:
        run_sweep(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
