#!/usr/bin/env python
"""Benchmark of the attention forward pass (one step = one attn_fwd call over the whole workload).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl reference]

Prints ONE JSON line.  `value` is attention-forward TFLOP/s (4*B*H*N^2*d, halved under the causal
mask) of the sawtooth scan order with the inputs resident in HBM; the cyclic order is timed the same
way and reported beside it.  `e2e` goes through attn_fwd_host with pinned host buffers, copies
included.  `roofline` compares the kernel with the measured bf16 tensor peak of this GPU pool,
`cpu_baseline` times the fp64 oracle on a bounded sample of the same workload.

With --gpus N > 1 (under torchrun) every rank runs the same workload on its own GPU: the path has no
exchange step, so the ranks are independent replicas and `value` is the sum of their throughputs
over the slowest rank's time.  `--impl reference` times the CPU oracle instead (rank 0 only).
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
# DRAM bytes one launch of the bench workload moves (dram__bytes_read.sum + dram__bytes_write.sum of
# an ncu capture of the same kernel; see the summary under profiles/).  None until captured.
NCU_DRAM_BYTES_PER_LAUNCH = {
    # c3-small (half of c3's heads, same kernel): 202,101,760 B read + 47,526,144 B written, scaled by 2 heads-wise
    "c3": 2 * (202101760 + 47526144),
    "c3-small": 202101760 + 47526144,
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
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
                        self.reasons.add(name)
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
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


L2_BYTES = 126 * 1000 * 1000          # B200
L2_FLUSH_BYTES = 256 << 20


def needs_l2_flush(w: wl.Workload) -> bool:
    """Workloads whose tensors would stay in L2 from one launch to the next are timed launch by launch with a write
    of a buffer larger than L2 in between."""
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


def oracle_sample_heads(w: wl.Workload, n_heads: int):
    return list(wl.all_heads(w))[:n_heads]


def time_oracle(w: wl.Workload, heads, threads: int = 0):
    """Seconds the oracle takes for every row of the given heads, and the FLOPs that is."""
    from oracle import attention as ora
    total, flops = 0.0, 0.0
    for b, h in heads:
        q = wl.bits_to_f64(wl.head_bits(w, "q", b, h), w.dtype)
        k = wl.bits_to_f64(wl.head_bits(w, "k", b, h), w.dtype)
        v = wl.bits_to_f64(wl.head_bits(w, "v", b, h), w.dtype)
        idx = np.arange(w.N, dtype=np.int64)
        t0 = time.perf_counter()
        ora.attention_rows(q, idx, k, v, w.scale, w.causal, threads)
        total += time.perf_counter() - t0
        flops += 4.0 * float(w.N) ** 2 * w.d / (2 if w.causal else 1)
    return total, flops


def config_of(w: wl.Workload, extra=None):
    c = {"workload": f"{w.name}: B={w.B} H={w.H} N={w.N} d={w.d} {w.dtype} {'causal' if w.causal else 'non-causal'}",
         "seed": w.seed, "scale": "1/sqrt(d)", "k_scale": w.k_scale,
         "l2": ("inputs larger than L2 (Q+K+V+O = %d MiB)" % (w.compulsory_bytes >> 20)) if not needs_l2_flush(w) else
               ("L2 flushed before every timed launch by writing a %d MiB buffer (Q+K+V+O = %d MiB)" % (L2_FLUSH_BYTES >> 20, w.compulsory_bytes >> 20))}
    if extra:
        c.update(extra)
    return c


def run_reference(args, w: wl.Workload):
    """The CPU oracle as the reference arm: each step computes every row of one head."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import attention as ora
    heads = list(wl.all_heads(w))
    for i in range(args.warmup):
        time_oracle(w, [heads[i % len(heads)]])
    secs, flops = 0.0, 0.0
    for i in range(args.steps):
        s, f = time_oracle(w, [heads[i % len(heads)]])
        secs += s
        flops += f
    value = flops / secs / 1e12
    sample = f"per step: every query row of one head of {w.name} ({w.N} rows x {w.N} keys, d={w.d})"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config_of(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": ora.threads_available(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c3", choices=sorted(wl.CONFIGS) + sorted(wl.STUDY_CASES))
    ap.add_argument("--scan-order", default="both", choices=["both", "cyclic", "sawtooth"],
                    help="orders to time; `value` is the sawtooth order unless only cyclic is timed")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--digit-order", default="tile", choices=["tile", "head"],
                    help="which digit of the linear work index varies fastest: the Q block (default) or the head")
    ap.add_argument("--max-ctas", type=int, default=0, help="cap on the persistent grid (the paper's 'active SMs'); 0 = all SMs")
    ap.add_argument("--also", default="c2,c4,c5",
                    help="further workloads timed briefly in both orders (single GPU only; '' for none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=0, help="end-to-end steps (default: min(steps, 10))")
    ap.add_argument("--cpu-heads", type=int, default=-1, help="heads the CPU baseline computes (default: sized to ~15 s)")
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

    dev = torch.device("cuda", local)
    adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
    shape = (w.B, w.H, w.N, w.d)
    numel = w.B * w.H * w.N * w.d

    # Inputs: the seeded workload, generated on the host into pinned buffers (they also feed the e2e leg).
    host = {}
    for name in ("q", "k", "v"):
        t = torch.empty(shape, dtype=torch.int16).pin_memory()
        arr = t.numpy()
        for b, h in wl.all_heads(w):
            arr[b, h] = wl.head_bits(w, name, b, h).view(np.int16)
        host[name] = t
    host["o"] = torch.empty(shape, dtype=torch.int16).pin_memory()
    devb = {n: torch.empty(shape, dtype=torch.int16, device=dev) for n in ("q", "k", "v", "o")}
    for n in ("q", "k", "v"):
        devb[n].copy_(host[n])
    stream = torch.cuda.Stream(device=dev)
    sh = stream.cuda_stream

    run_opts = None
    if args.max_ctas > 0 or args.digit_order == "head":
        run_opts = sa.Opts()
        run_opts.max_ctas = args.max_ctas
        run_opts.digit_order = sa.HEAD_FASTEST if args.digit_order == "head" else sa.TILE_FASTEST

    def make_step(bufs, wk, a_dt):
        def step(order):
            sa.attn_fwd_ex(bufs["q"].data_ptr(), bufs["k"].data_ptr(), bufs["v"].data_ptr(), bufs["o"].data_ptr(),
                           wk.B, wk.H, wk.N, wk.d, wk.scale, int(wk.causal), order, a_dt, sh, run_opts)
        return step

    step = make_step(devb, w, adt)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    flush_buf = [None]

    def timed(fn, steps, flush=False):
        """Milliseconds of `steps` calls of fn on the launch stream (CUDA events), max over ranks.  With `flush` every
        call is timed by its own pair of events and a buffer larger than L2 is overwritten before it."""
        if flush:
            if flush_buf[0] is None:
                flush_buf[0] = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
            barrier()
            with torch.cuda.stream(stream):
                for a, b in pairs:
                    flush_buf[0].fill_(1)
                    a.record(stream)
                    fn()
                    b.record(stream)
            barrier()
            return max_over_ranks(sum(a.elapsed_time(b) for a, b in pairs), dist, dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(steps):
                fn()
            e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev)

    orders = {"cyclic": sa.CYCLIC, "sawtooth": sa.SAWTOOTH}
    timed_orders = ["sawtooth", "cyclic"] if args.scan_order == "both" else [args.scan_order]  # the headline order first
    headline = "sawtooth" if "sawtooth" in timed_orders else "cyclic"
    results = {}
    with ClockSampler(local) as clocks:
        for name in timed_orders:
            for _ in range(args.warmup):
                step(orders[name])
            results[name] = timed(lambda: step(orders[name]), args.steps, needs_l2_flush(w)) / args.steps
    sa.attn_device_status()
    clk = clocks.summary()
    # SM clock the last timed kernel really ran at: cycles its first CTA counted over the launch time.
    clk["kernel_mhz"] = sa.attn_last_kernel_cycles() / (results[timed_orders[-1]] * 1e3)

    # The two orders launch by launch in alternation, so that neither sees a hotter or a cooler GPU.
    ab = None
    if len(timed_orders) == 2:
        pairs = max(3, min(args.steps, 20))
        acc = {"cyclic": [], "sawtooth": []}
        for _ in range(pairs):
            for name in timed_orders:
                acc[name].append(timed(lambda: step(orders[name]), 1))
        ab = {n: float(np.median(v)) for n, v in acc.items()}

    # The dynamic tile schedule (work items claimed from a counter) beside the static one, same launches alternating.
    dyn = None
    if len(timed_orders) == 2:
        plan0 = sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt)
        n_scratch = sa.attn_dynamic_scratch_bytes(plan0.grid)
        scratch = torch.zeros(n_scratch // 4, dtype=torch.int32, device=dev)

        def dyn_step(order):
            sa.attn_fwd_dynamic(devb["q"].data_ptr(), devb["k"].data_ptr(), devb["v"].data_ptr(), devb["o"].data_ptr(),
                                w.B, w.H, w.N, w.d, w.scale, int(w.causal), order, adt, sh, None, scratch.data_ptr(), n_scratch)

        pairs = max(3, min(args.steps, 20))
        acc = {"static": [], "dynamic": []}
        for _ in range(3):
            dyn_step(orders["sawtooth"])
        for _ in range(pairs):
            acc["static"].append(timed(lambda: step(orders["sawtooth"]), 1))
            acc["dynamic"].append(timed(lambda: dyn_step(orders["sawtooth"]), 1))
        sa.attn_device_status()
        dyn = {n: float(np.median(v)) for n, v in acc.items()}

    # End to end: host buffers in, host buffer out, copies inside the timed region.
    e2e = None
    if not args.skip_e2e:
        e2e_steps = args.e2e_steps or min(args.steps, 10)

        def e2e_step():
            sa.attn_fwd_host(host["q"].data_ptr(), host["k"].data_ptr(), host["v"].data_ptr(), host["o"].data_ptr(),
                             devb["q"].data_ptr(), devb["k"].data_ptr(), devb["v"].data_ptr(), devb["o"].data_ptr(),
                             w.B, w.H, w.N, w.d, w.scale, int(w.causal), orders[headline], adt, sh)

        for _ in range(2):
            e2e_step()
        e2e_ms = timed(e2e_step, e2e_steps) / e2e_steps
        sa.attn_device_status()
        e2e = {"value": whole_job_tflops(w.flops, e2e_ms, world), "unit": UNIT, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "h2d_bytes_per_step": 3 * numel * 2, "d2h_bytes_per_step": numel * 2}

    # The other configurations, timing only (inputs drawn on the device from a seed), single GPU only.
    also = {}
    if world == 1 and args.also:
        del devb
        torch.cuda.empty_cache()
        for name in [n for n in args.also.split(",") if n]:
            wk = wl.CONFIGS.get(name) or wl.STUDY_CASES[name]
            tdt = torch.bfloat16 if wk.dtype == wl.BF16 else torch.float16
            g = torch.Generator(device=dev).manual_seed(wk.seed)
            bufs = {}
            for n in ("q", "k", "v"):
                bufs[n] = torch.randn((wk.B, wk.H, wk.N, wk.d), device=dev, generator=g, dtype=torch.float32).to(tdt)
            if wk.k_scale != 1.0:
                bufs["k"] *= wk.k_scale
            bufs["o"] = torch.empty_like(bufs["q"])
            a_dt = sa.BF16 if wk.dtype == wl.BF16 else sa.F16
            st = make_step(bufs, wk, a_dt)
            n_steps = max(3, min(args.steps, int(200.0 / (wk.flops / 1e12))))  # about 0.2 s per order
            entry = {"workload": config_of(wk)["workload"], "steps": n_steps}
            for oname in ("cyclic", "sawtooth"):
                for _ in range(3):
                    st(orders[oname])
                ms = timed(lambda: st(orders[oname]), n_steps, needs_l2_flush(wk)) / n_steps
                entry[oname] = {"value": wk.flops / ms / 1e9, "unit": UNIT, "ms_per_step": ms}
            n_scr = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(wk.B, wk.H, wk.N, wk.d, int(wk.causal), a_dt).grid)
            scr = torch.zeros(n_scr // 4, dtype=torch.int32, device=dev)

            def dyn_also(order, bufs=bufs, wk=wk, a_dt=a_dt, scr=scr, n_scr=n_scr):
                sa.attn_fwd_dynamic(bufs["q"].data_ptr(), bufs["k"].data_ptr(), bufs["v"].data_ptr(), bufs["o"].data_ptr(),
                                    wk.B, wk.H, wk.N, wk.d, wk.scale, int(wk.causal), order, a_dt, sh, None, scr.data_ptr(), n_scr)

            for _ in range(3):
                dyn_also(orders["sawtooth"])
            ms = timed(lambda: dyn_also(orders["sawtooth"]), n_steps, needs_l2_flush(wk)) / n_steps
            entry["sawtooth_dynamic_schedule"] = {"value": wk.flops / ms / 1e9, "unit": UNIT, "ms_per_step": ms}
            sa.attn_device_status()
            also[name] = entry
            del bufs
            torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    flops = w.flops
    ms_head = results[headline]
    tf_head = whole_job_tflops(flops, ms_head, 1)  # one GPU's throughput; `value` is the job's
    # Which measured peak the run is compared with: the sustained one when the timed launches ran as one long,
    # power-capped load (half a second or more of it, or the cap seen by NVML with the kernel's own clock under 80 % of
    # the maximum), else the burst one.  Both fractions are in the line either way.
    timed_region_s = ms_head * args.steps / 1e3
    capped = "sw_power_cap" in clk.get("reasons", []) and clk.get("sm_max_mhz") and clk["kernel_mhz"] < 0.8 * clk["sm_max_mhz"]
    peak_kind = "sustained" if (timed_region_s >= 0.5 or capped) else "burst"
    peak = peaks[peak_kind]
    plan = sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, run_opts)
    line = {
        "metric": METRIC, "value": whole_job_tflops(flops, ms_head, world), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_head, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == wl.BF16 else "f16", "data": "synthetic",
        "config": config_of(w, {"scan_order": headline, "parallelism": "replicas only" if world > 1 else "single GPU",
                                "grid": plan.grid, "rows_per_item": plan.rows_per_item, "block_n": plan.block_n,
                                "kv_stages": plan.kv_stages}),
        "clocks": clk,
        "gpu_launches": args.steps,
        "roofline": {"bound": "tensor", "achieved": tf_head, "peak": peak, "unit": UNIT, "frac": tf_head / peak,
                     "peak_kind": f"{peak_kind} bf16 matmul, of {peaks['source']}",
                     "frac_of_burst": tf_head / peaks["burst"], "frac_of_sustained": tf_head / peaks["sustained"],
                     "frac_of_nominal_2250": tf_head / NOMINAL_BF16_TFLOPS,
                     "flops_per_launch": flops, "launch_ms": ms_head,
                     "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(w.name), "compulsory_bytes": w.compulsory_bytes},
    }
    if e2e is not None:
        line["e2e"] = e2e
    for name in timed_orders:
        if name != headline:
            line[name] = {"value": whole_job_tflops(flops, results[name], world), "unit": UNIT, "ms_per_step": results[name]}
    if ab is not None:
        line["alternating_launches"] = {"cyclic_ms": ab["cyclic"], "sawtooth_ms": ab["sawtooth"],
                                        "sawtooth_over_cyclic": ab["cyclic"] / ab["sawtooth"]}
    if dyn is not None:
        line["dynamic_schedule"] = {"what": "attn_fwd_dynamic vs attn_fwd, sawtooth, single launches alternating",
                                    "static_ms": dyn["static"], "dynamic_ms": dyn["dynamic"],
                                    "dynamic_tflops": whole_job_tflops(flops, dyn["dynamic"], world)}
    if also:
        line["also"] = also
    if not args.skip_cpu_baseline:
        from oracle import attention as ora
        per_head_flops = 4.0 * float(w.N) ** 2 * w.d / (2 if w.causal else 1)
        n_heads = args.cpu_heads if args.cpu_heads > 0 else max(1, min(w.B * w.H, int(15.0 * 2.5e9 * ora.threads_available() / per_head_flops)))
        heads = oracle_sample_heads(w, n_heads)
        secs, fl = time_oracle(w, heads)
        line["cpu_baseline"] = {"value": fl / secs / 1e12, "unit": UNIT, "cores": ora.threads_available(), "kind": "oracle",
                                "seconds": secs,
                                "sample": f"every query row of the first {len(heads)} of {w.B * w.H} heads of {w.name}"}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
