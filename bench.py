#!/usr/bin/env python
"""Benchmark of the attention forward pass (one step = one attn_fwd call over the whole workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--also c3,c4] [--impl reference]

Prints ONE JSON line.  The workload is c5 (B=2 H=16 N=65536 d=128 bf16 causal), the largest of the five
configurations; c3, c4, c2, a d = 64 shape that fills the GPU (d64-n8k) and the shape of the paper's own sweep (B = 8,
N = 131072, d = 64, with and without the causal mask) are measured the same way and reported, each with its own roofline
block, under `also`.

How a workload is timed.  The two scan orders are launched in alternation, cyclic, sawtooth, cyclic, ..., every
launch between its own pair of CUDA events on the launch stream, after a warm-up of the same alternating launches
that lasts at least a quarter of a second, so that both orders see the same (warm, power-capped) GPU.  A step is one
launch of the headline order (sawtooth unless --scan-order says otherwise); `ms_per_step` is the mean over the K
headline launches, `value` the attention-forward TFLOP/s that is (4*B*H*N^2*d, halved under the causal mask), the
other order's figure sits beside it.  After the timed region one more launch of each order is timed together with
the SM cycles its first CTA counted: that gives the clock the kernel really ran at and two figures that do not depend
on the clock, cycles per K/V step and the fraction of the tensor peak at that clock.

`e2e` goes through attn_fwd_host with pinned host buffers, copies included.  `roofline` compares the kernel with
the measured bf16 tensor peak of this GPU pool, `cpu_baseline` times the fp64 oracle on a bounded sample of the same
workload.  With --gpus N > 1 (under torchrun) every rank runs the same workload on its own GPU: the path has no
exchange step, so the ranks are independent replicas and `value` is the sum of their throughputs over the slowest
rank's time.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import workloads as wl

METRIC = "attention_fwd_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_BF16_TFLOPS = 1590.0
# Dense 16-bit tensor throughput of one SM per clock: a tcgen05.mma of shape 128 x 128 x 16 (2 * 128 * 128 * 16 =
# 524288 FLOP) occupies the SM's tensor pipe for 64 cycles, i.e. 8192 FLOP per clock per SM; 148 SMs at the 1965 MHz
# maximum clock give 2383 TFLOP/s, at the clock a launch really ran at correspondingly less.
FLOP_PER_CLK_PER_SM = 8192.0
WARMUP_LOAD_SECONDS = 0.25

# DRAM bytes one launch moves: (dram__bytes_read.sum, dram__bytes_write.sum) of a one-launch ncu capture of the present
# kernel on the full-size workload with the default launch plan (three metrics, one pass).
# Keyed by (workload, scan order, pairing in force); anything else reports null.
NCU_DRAM_BYTES_PER_LAUNCH = {
    ("c3", "cyclic", "none"): (404312832, 113961984),
    ("c3", "sawtooth", "none"): (406504192, 114424576),
    ("c4", "cyclic", "mirrored"): (968785152, 250669568),
    ("c4", "sawtooth", "mirrored"): (974485504, 251215616),
    ("c4", "cyclic", "none"): (1200302336, 258832896),
    ("c4", "sawtooth", "none"): (1640605184, 259677952),
    ("c5", "cyclic", "mirrored"): (2634280960, 521590528),
    ("c5", "sawtooth", "mirrored"): (2511834112, 526502400),
    ("c5", "cyclic", "none"): (5354950144, 535655936),
    ("c5", "sawtooth", "none"): (7901230592, 532906240),
}


# What the paper reports for the two shapes of its sweep that bench.py also times (its Section 4.3, CuTile results, sawtooth
# order): another machine and another kernel, context for the reader, not a target.
PAPER_CONTEXT = {
    "sweep-d64-b8": {"tflops": 69.0, "what": "paper, GB10, CuTile kernel with 64x64 tiles, sawtooth order, B=8 S=131072 D=64 non-causal"},
    "sweep-d64-b8-causal": {"tflops": 66.0, "what": "paper, GB10, CuTile kernel with 64x64 tiles, sawtooth order, B=8 S=131072 D=64 causal"},
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"burst": float(p["bf16_tflops"]), "sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    except Exception:
        return {"burst": FALLBACK_BF16_TFLOPS, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML, about once a millisecond, while a timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.index, self.period = index, period_s
        self.samples, self.power, self.reasons, self.max_mhz = [], [], {}, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons[name] = self.reasons.get(name, 0) + 1
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_mhz_min": min(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "reason_samples": self.reasons, "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None, "sampling": "NVML, about 1 ms apart, timed region only"}


L2_BYTES = 126 * 1000 * 1000          # B200
L2_FLUSH_BYTES = 256 << 20


def needs_l2_flush(w: wl.Workload) -> bool:
    """Workloads whose tensors would stay in L2 from one launch to the next are timed with a write of a buffer
    larger than L2 before every launch."""
    return w.compulsory_bytes <= 2 * L2_BYTES


def max_over_ranks(ms: float, dist=None, device=None) -> float:
    """The slowest rank's time: what the whole job took.  `dist` is torch.distributed once a process
    group exists (any backend), else None for a single process."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tflops(flops_per_rank: float, ms: float, world: int) -> float:
    """Independent replicas: every rank does the same work, the job lasts as long as its slowest rank."""
    return flops_per_rank * world / ms / 1e9


def time_oracle_rows(w: wl.Workload, b: int, h: int, rows: np.ndarray, threads: int = 0):
    """Seconds the oracle takes for the given query rows of head (b, h), and the FLOPs that is (4 * keys seen * d per row)."""
    from oracle import attention as ora
    q = wl.bits_to_f64(wl.head_bits(w, "q", b, h), w.dtype)
    k = wl.bits_to_f64(wl.head_bits(w, "k", b, h), w.dtype)
    v = wl.bits_to_f64(wl.head_bits(w, "v", b, h), w.dtype)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    t0 = time.perf_counter()
    ora.attention_rows(q[rows], rows, k, v, w.scale, w.causal, threads)
    secs = time.perf_counter() - t0
    keys = (rows + 1).sum() if w.causal else len(rows) * w.N
    return secs, 4.0 * float(keys) * w.d


def oracle_sample_rows(w: wl.Workload, b: int, h: int, seconds: float, flops_per_second: float) -> np.ndarray:
    """Seeded, sorted query rows of one head whose oracle run should take about `seconds`: every row if that fits."""
    per_row = 4.0 * w.d * (w.N / 2.0 if w.causal else w.N)
    n = int(max(64, min(w.N, seconds * flops_per_second / per_row)))
    if n >= w.N:
        return np.arange(w.N, dtype=np.int64)
    return np.sort(np.random.default_rng([w.seed + 7, b, h]).choice(w.N, size=n, replace=False)).astype(np.int64)


def config_of(w: wl.Workload, extra=None):
    c = {"workload": f"{w.name}: B={w.B} H={w.H} N={w.N} d={w.d} {w.dtype} {'causal' if w.causal else 'non-causal'}",
         "seed": w.seed, "scale": "1/sqrt(d)", "k_scale": w.k_scale,
         "l2": ("inputs larger than L2 (Q+K+V+O = %d MiB)" % (w.compulsory_bytes >> 20)) if not needs_l2_flush(w) else
               ("L2 flushed before every timed launch by writing a %d MiB buffer (Q+K+V+O = %d MiB)" % (L2_FLUSH_BYTES >> 20, w.compulsory_bytes >> 20))}
    if extra:
        c.update(extra)
    return c


def run_reference(args, w: wl.Workload):
    """The CPU oracle as the reference arm: each step computes a seeded sample of the query rows of one head."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import attention as ora
    heads = list(wl.all_heads(w))
    cores = ora.threads_available()
    per_step_seconds = 0.5
    rows = {bh: oracle_sample_rows(w, bh[0], bh[1], per_step_seconds, 3.5e9 * cores) for bh in heads[:max(1, min(len(heads), args.steps + args.warmup))]}
    keys = list(rows)
    for i in range(args.warmup):
        bh = keys[i % len(keys)]
        time_oracle_rows(w, bh[0], bh[1], rows[bh])
    secs, flops = 0.0, 0.0
    for i in range(args.steps):
        bh = keys[(args.warmup + i) % len(keys)]
        s, f = time_oracle_rows(w, bh[0], bh[1], rows[bh])
        secs += s
        flops += f
    value = flops / secs / 1e12
    n_rows = len(rows[keys[0]])
    sample = (f"per step: {n_rows} seeded query rows of one head of {w.name} against every key they may see "
              f"(N={w.N}, d={w.d}); FLOPs counted as 4 * keys seen * d per row")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


class Bench:
    """Device-side measurements of one process (one GPU)."""

    def __init__(self, args, local, dist):
        import torch
        import paper_2601_16032_b200 as sa
        self.torch, self.sa, self.args, self.dist = torch, sa, args, dist
        self.dev = torch.device("cuda", local)
        self.local = local
        self.stream = torch.cuda.Stream(device=self.dev)
        self.sh = self.stream.cuda_stream
        self.flush_buf = None
        self.sm_count = torch.cuda.get_device_properties(self.dev).multi_processor_count
        self.orders = {"cyclic": sa.CYCLIC, "sawtooth": sa.SAWTOOTH}

    def opts(self):
        sa, a = self.sa, self.args
        o = sa.Opts()
        o.max_ctas = a.max_ctas
        o.digit_order = sa.HEAD_FASTEST if a.digit_order == "head" else sa.TILE_FASTEST
        o.pairing = {"default": sa.PAIR_DEFAULT, "none": sa.PAIR_NONE, "mirrored": sa.PAIR_MIRRORED, "adjacent": sa.PAIR_ADJACENT}[a.pairing]
        return o

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        self.torch.cuda.synchronize(self.dev)

    def host_tensors(self, w, pinned):
        torch = self.torch
        host = {}
        for name in ("q", "k", "v"):
            t = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.int16)
            if pinned:
                t = t.pin_memory()
            arr = t.numpy()
            for b, h in wl.all_heads(w):
                arr[b, h] = wl.head_bits(w, name, b, h).view(np.int16)
            host[name] = t
        return host

    def timed_launches(self, fns, flush):
        """Runs the callables in order, each between its own pair of events on the launch stream; returns their times in ms
        (max over ranks, launch by launch).  With `flush` a buffer larger than L2 is overwritten before each."""
        torch = self.torch
        if flush and self.flush_buf is None:
            self.flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=self.dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in fns]
        self.barrier()
        with torch.cuda.stream(self.stream):
            for fn, (a, b) in zip(fns, pairs):
                if flush:
                    self.flush_buf.fill_(1)
                a.record(self.stream)
                fn()
                b.record(self.stream)
        self.barrier()
        return [max_over_ranks(a.elapsed_time(b), self.dist, self.dev) for a, b in pairs]

    def measure(self, w, steps, warmup, headline, only_order=None, host=None):
        """One workload: inputs from its seed, the alternating timed region, the clock-free figures, the roofline block."""
        torch, sa = self.torch, self.sa
        adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
        host = host or self.host_tensors(w, pinned=False)
        devb = {n: torch.empty((w.B, w.H, w.N, w.d), dtype=torch.int16, device=self.dev) for n in ("q", "k", "v", "o")}
        for n in ("q", "k", "v"):
            devb[n].copy_(host[n])
        opts = self.opts()
        plan = sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, opts)

        def launch(order):
            sa.attn_fwd_ex(devb["q"].data_ptr(), devb["k"].data_ptr(), devb["v"].data_ptr(), devb["o"].data_ptr(),
                           w.B, w.H, w.N, w.d, w.scale, int(w.causal), self.orders[order], adt, self.sh, opts)

        other = "cyclic" if headline == "sawtooth" else "sawtooth"
        seq = [headline] if only_order else [other, headline]      # one round of the alternation; the headline order last
        flush = needs_l2_flush(w)
        # Warm-up: the same alternation, W rounds and at least WARMUP_LOAD_SECONDS of GPU work.
        rounds, t_round = 0, None
        while rounds < warmup or (t_round is not None and rounds * t_round < WARMUP_LOAD_SECONDS * 1e3 and rounds < 2000):
            ms = self.timed_launches([lambda o=o: launch(o) for o in seq], flush)
            t_round = sum(ms) if t_round is None else min(t_round, sum(ms))
            rounds += 1
        with ClockSampler(self.local) as clocks:
            times = self.timed_launches([lambda o=o: launch(o) for _ in range(steps) for o in seq], flush)
        sa.attn_device_status()
        per_order = {o: times[i::len(seq)] for i, o in enumerate(seq)}
        ms_head = float(np.mean(per_order[headline]))
        # One more launch of each order, timed together with the cycles its first CTA counted.
        trace0 = [e for e in sa.attn_schedule_trace(w.B, w.H, w.N, w.d, int(w.causal), sa.SAWTOOTH, adt, opts) if e.cta == 0]
        kv_steps_cta0 = sum(e.n_kv for e in trace0)
        legs = {}
        for o in seq:
            ms1 = self.timed_launches([lambda o=o: launch(o)], flush)[0]
            cycles = sa.attn_last_kernel_cycles()
            mhz = cycles / (ms1 * 1e3)
            tf1 = w.flops / ms1 / 1e9
            legs[o] = {"ms": ms1, "tflops": tf1, "cta0_cycles": cycles, "kernel_mhz": mhz,
                       "cycles_per_kv_step": cycles / kv_steps_cta0,
                       "frac_of_clock_scaled_peak": tf1 * 1e12 / (FLOP_PER_CLK_PER_SM * self.sm_count * mhz * 1e6)}
        sa.attn_device_status()
        clk = clocks.summary()
        clk["kernel_mhz"] = legs[headline]["kernel_mhz"]
        peaks = measured_peaks()
        tf_head = w.flops / ms_head / 1e9
        pairing_name = {1: "none", 2: "mirrored", 3: "adjacent"}[plan.pairing]
        default_plan = self.args.max_ctas == 0 and self.args.digit_order == "tile"
        dram = NCU_DRAM_BYTES_PER_LAUNCH.get((w.name, headline, pairing_name)) if default_plan else None
        # Which measured peak the run is compared with: the launches ran one after the other for the warm-up load and the
        # timed region, i.e. as a sustained, power-capped load, when the kernel's own clock sat under 80 % of the maximum.
        capped = bool(clk.get("sm_max_mhz")) and legs[headline]["kernel_mhz"] < 0.8 * clk["sm_max_mhz"]
        peak_kind = "sustained" if capped else "burst"
        block = {
            "config": config_of(w, {"scan_order": headline, "grid": plan.grid, "rows_per_item": plan.rows_per_item, "block_n": plan.block_n,
                                    "kv_stages": plan.kv_stages, "pairing": pairing_name,
                                    "timing": f"{len(seq)} scan orders launched in alternation, per-launch CUDA events, {rounds} warm-up rounds"}),
            "ms_per_step": ms_head, "ms_per_step_median": float(np.median(per_order[headline])), "tflops": tf_head,
            "orders": {o: {"ms_mean": float(np.mean(v)), "ms_median": float(np.median(v)), "tflops": w.flops / float(np.mean(v)) / 1e9,
                           "launches": len(v)} for o, v in per_order.items()},
            "single_launch": legs,
            "clocks": clk,
            "launches_in_timed_region": len(times),
            "roofline": {"bound": "tensor", "achieved": tf_head, "peak": peaks[peak_kind], "unit": UNIT, "frac": tf_head / peaks[peak_kind],
                         "peak_kind": f"{peak_kind} bf16 matmul, of {peaks['source']}",
                         "frac_of_burst": tf_head / peaks["burst"], "frac_of_sustained": tf_head / peaks["sustained"],
                         "frac_of_nominal_2250": tf_head / NOMINAL_BF16_TFLOPS,
                         "frac_of_clock_scaled_peak": legs[headline]["frac_of_clock_scaled_peak"],
                         "cycles_per_kv_step": legs[headline]["cycles_per_kv_step"],
                         "flops_per_launch": w.flops, "launch_ms": ms_head,
                         "traffic": (dram[0] + dram[1]) if dram else None, "compulsory_bytes": w.compulsory_bytes,
                         "dram_read_bytes": dram[0] if dram else None, "compulsory_read_bytes": 3 * w.compulsory_bytes // 4,
                         "read_amplification": (dram[0] / (3 * w.compulsory_bytes / 4)) if dram else None},
        }
        if w.d == 64:
            # The tensor work of a step halves at d = 64 and its softmax does not: the step is as long as the softmax of a
            # tile, which is bound by the schedulers' issue slots and the MUFU.  Counters of one launch (ncu, d64-n8k-small):
            # 1466 instructions issued per scheduler and step, 1536 MUFU cycles per scheduler and step.
            cps = legs[headline]["cycles_per_kv_step"]
            block["roofline"]["alu"] = {"bound": "alu", "what": "softmax of two Q tiles per K/V step on each of the SM's four schedulers",
                                        "issue_slots_per_step": 1466, "mufu_cycles_per_step": 1536,
                                        "frac_issue": 1466 / cps, "frac_mufu": 1536 / cps}
        if len(seq) == 2:
            block["sawtooth_over_cyclic"] = float(np.mean(per_order["cyclic"]) / np.mean(per_order["sawtooth"]))
        return block, devb, launch

    def dynamic_leg(self, w, devb, launch_static, headline, rounds):
        """attn_fwd_dynamic beside attn_fwd_ex, single launches alternating."""
        torch, sa = self.torch, self.sa
        adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
        po = self.opts()
        po.pairing = sa.PAIR_NONE        # the dynamic schedule claims single items
        n_scratch = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, po).grid)
        scratch = torch.zeros(n_scratch // 4, dtype=torch.int32, device=self.dev)

        def dyn():
            sa.attn_fwd_dynamic(devb["q"].data_ptr(), devb["k"].data_ptr(), devb["v"].data_ptr(), devb["o"].data_ptr(), w.B, w.H, w.N, w.d,
                                w.scale, int(w.causal), self.orders[headline], adt, self.sh, po, scratch.data_ptr(), n_scratch)

        flush = needs_l2_flush(w)
        self.timed_launches([dyn, dyn], flush)
        ms = self.timed_launches([f for _ in range(rounds) for f in (lambda: launch_static(headline), dyn)], flush)
        sa.attn_device_status()
        sta, dy = float(np.mean(ms[0::2])), float(np.mean(ms[1::2]))
        return {"what": "attn_fwd_dynamic beside attn_fwd_ex, same scan order, single launches alternating",
                "static_ms": sta, "dynamic_ms": dy, "static_tflops": w.flops / sta / 1e9, "dynamic_tflops": w.flops / dy / 1e9}

    def host_call_us(self):
        """Median host time of one attn_fwd call (argument checks, cached tensor maps, launch), measured through the ctypes
        binding on a small workload whose kernel is short, so that the launch queue never fills."""
        torch, sa = self.torch, self.sa
        t = torch.zeros((1, 1, 256, 64), dtype=torch.float16, device=self.dev)
        o = torch.empty_like(t)
        args = (t.data_ptr(), t.data_ptr(), t.data_ptr(), o.data_ptr(), 1, 1, 256, 64, 0.125, 0, sa.SAWTOOTH, sa.F16, self.sh)
        for _ in range(20):
            sa.attn_fwd(*args)
        torch.cuda.synchronize(self.dev)
        times = []
        for _ in range(10):
            t0 = time.perf_counter()
            for _ in range(20):
                sa.attn_fwd(*args)
            times.append((time.perf_counter() - t0) / 20 * 1e6)
            torch.cuda.synchronize(self.dev)
        sa.attn_device_status()
        return float(np.median(times))


def host_call_us_from_c():
    """The same call timed from C (profile_host_call.cu, built beside the library): what the library itself costs per
    call, without the ctypes marshalling.  None when the program is not there and cannot be built."""
    import re
    import subprocess
    try:
        from paper_2601_16032_b200 import build as lib_build
        exe = lib_build.build_host_call_probe()
        out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
        m = re.search(r"median ([0-9.]+) us", out.stdout)
        return float(m.group(1)) if out.returncode == 0 and m else None
    except Exception:
        return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c5", choices=sorted(wl.CONFIGS) + sorted(wl.STUDY_CASES))
    ap.add_argument("--scan-order", default="both", choices=["both", "cyclic", "sawtooth"],
                    help="both: the orders alternate and `value` is the sawtooth order; else only that order is launched")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--digit-order", default="tile", choices=["tile", "head"],
                    help="which digit of the linear work index varies fastest: the Q block (default) or the head")
    ap.add_argument("--pairing", default="default", choices=["default", "none", "mirrored", "adjacent"],
                    help="how the static walk groups work items (default: mirrored pairs under the causal mask)")
    ap.add_argument("--max-ctas", type=int, default=0, help="cap on the persistent grid (the paper's 'active SMs'); 0 = all SMs")
    ap.add_argument("--also", default="c3,c4,d64-n8k,c2,sweep-d64-b8,sweep-d64-b8-causal",
                    help="further workloads measured the same way (single GPU only; '' for none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=0, help="end-to-end steps (default: min(steps, 5))")
    ap.add_argument("--cpu-seconds", type=float, default=15.0, help="about how long the CPU baseline may take")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = wl.CONFIGS.get(args.workload) or wl.STUDY_CASES[args.workload]

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import paper_2601_16032_b200 as sa
    from paper_2601_16032_b200 import build as lib_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        lib_build.build()  # compiles the CUDA library in-tree if it is missing or older than its sources
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    bench = Bench(args, local, dist)
    headline = "cyclic" if args.scan_order == "cyclic" else "sawtooth"
    only = None if args.scan_order == "both" else args.scan_order
    adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
    numel = w.B * w.H * w.N * w.d

    host = bench.host_tensors(w, pinned=not args.skip_e2e)
    block, devb, launch = bench.measure(w, args.steps, args.warmup, headline, only, host)
    dyn = bench.dynamic_leg(w, devb, launch, headline, max(3, min(args.steps, 10))) if only is None else None
    host_us = bench.host_call_us()
    host_us_c = host_call_us_from_c() if rank == 0 else None

    # End to end: host buffers in, host buffer out, copies inside the timed region.
    e2e = None
    if not args.skip_e2e:
        e2e_steps = args.e2e_steps or min(args.steps, 5)
        host["o"] = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.int16).pin_memory()
        e2e_opts = bench.opts()

        def e2e_step():
            sa.attn_fwd_host(host["q"].data_ptr(), host["k"].data_ptr(), host["v"].data_ptr(), host["o"].data_ptr(),
                             devb["q"].data_ptr(), devb["k"].data_ptr(), devb["v"].data_ptr(), devb["o"].data_ptr(),
                             w.B, w.H, w.N, w.d, w.scale, int(w.causal), bench.orders[headline], adt, bench.sh, e2e_opts)

        bench.timed_launches([e2e_step, e2e_step], False)
        e2e_ms = float(np.mean(bench.timed_launches([e2e_step] * e2e_steps, False)))
        sa.attn_device_status()
        e2e = {"value": whole_job_tflops(w.flops, e2e_ms, world), "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_bytes_per_step": 3 * numel * 2, "d2h_bytes_per_step": numel * 2}
    del devb, launch, host
    torch.cuda.empty_cache()

    # The other configurations, measured the same way from their seeds (single GPU only).
    also = {}
    if world == 1 and args.also:
        for name in [n for n in args.also.split(",") if n and n != w.name]:
            wk = wl.CONFIGS.get(name) or wl.STUDY_CASES[name]
            n_steps = max(5, min(args.steps, int(400.0 / (wk.flops / 1e12))))  # about 0.4 s per order
            blk, dv, ln = bench.measure(wk, n_steps, args.warmup, headline, only)
            if only is None:
                blk["dynamic_schedule"] = bench.dynamic_leg(wk, dv, ln, headline, 5)
            blk["steps"] = n_steps
            if name in PAPER_CONTEXT:
                blk["paper_context"] = dict(PAPER_CONTEXT[name], ratio=blk["tflops"] / PAPER_CONTEXT[name]["tflops"])
            also[name] = blk
            del dv, ln
            torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": whole_job_tflops(w.flops, block["ms_per_step"], world), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": block["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == wl.BF16 else "f16", "data": "synthetic",
        "config": dict(block["config"], parallelism="replicas only" if world > 1 else "single GPU"),
        "clocks": block["clocks"],
        "gpu_launches": block["launches_in_timed_region"],
        "roofline": block["roofline"],
        "orders": block["orders"], "single_launch": block["single_launch"], "ms_per_step_median": block["ms_per_step_median"],
        "host_call_us": host_us, "host_call_us_from_c": host_us_c,
    }
    if "sawtooth_over_cyclic" in block:
        line["sawtooth_over_cyclic"] = block["sawtooth_over_cyclic"]
    if e2e is not None:
        line["e2e"] = e2e
    if dyn is not None:
        line["dynamic_schedule"] = dyn
    if also:
        line["also"] = also
    if not args.skip_cpu_baseline:
        from oracle import attention as ora
        cores = ora.threads_available()
        b, h = next(iter(wl.all_heads(w)))
        rows = oracle_sample_rows(w, b, h, args.cpu_seconds, 3.5e9 * cores)
        secs, fl = time_oracle_rows(w, b, h, rows)
        line["cpu_baseline"] = {"value": fl / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "seconds": secs,
                                "sample": f"{len(rows)} seeded query rows of head (0, 0) of {w.name} against every key they may see; "
                                          f"FLOPs counted as 4 * keys seen * d per row"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
