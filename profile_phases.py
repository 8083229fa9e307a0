"""Per-phase SM-cycle breakdown of the attention kernel, from in-kernel clock stamps.

    python profile_phases.py [B H N d] [--causal] [--fp16] [--cyclic]

Builds a second copy of the library with -DSAW_PROFILE (libsawtooth_attn_profile.so, beside the normal one), runs one
warmed-up launch of the given shape (default 4 16 8192 128, bf16, non-causal, sawtooth order) and prints, for the
median CTA, the cycles per K/V step that the MMA-issuing lane of Q tile 0 and one softmax thread of Q tile 0 spend in
each phase.  The stamps cost about 45 cycles each, so the totals are a few per cent above an unprofiled run.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess

import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_16032_b200 import build as _build

PROFILE_LIB = os.path.join(_build.PKG, "libsawtooth_attn_profile.so")
MMA_PHASES = ["loop / decode", "wait Q", "wait K/V", "wait P (early part)", "issue P.V (early)", "wait P (rest)", "issue P.V (rest)",
              "issue Q.K + commit", "release K/V slots"]
SOFTMAX_PHASES = ["loop / decode", "wait S", "TMEM load", "mask + row max", "warp vote", "rescale test", "exp, convert, store (early part)",
                  "exp, convert, store (rest) + arrive", "epilogue: rest", "epilogue: wait O", "epilogue: wait staging slot",
                  "epilogue: stage + TMA store"]


def build_profile_library() -> str:
    newest = max(os.path.getmtime(f) for f in _build.DEPS)
    if not os.path.exists(PROFILE_LIB) or os.path.getmtime(PROFILE_LIB) < newest:
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.run([nvcc] + _build.NVCC_FLAGS + ["-DSAW_PROFILE", "-o", PROFILE_LIB] + _build.SOURCES, check=True)
    return PROFILE_LIB


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("shape", nargs="*", type=int, default=[4, 16, 8192, 128])
    ap.add_argument("--causal", action="store_true")
    ap.add_argument("--fp16", action="store_true")
    ap.add_argument("--cyclic", action="store_true")
    args = ap.parse_args()
    B, H, N, d = args.shape
    import torch

    lib = ctypes.CDLL(build_profile_library())
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.attn_fwd.argtypes = [vp] * 4 + [ci] * 4 + [cf, ci, ci, ci, vp]
    lib.attn_fwd.restype = ci
    lib.attn_debug_profile.argtypes = [vp]
    lib.attn_debug_profile.restype = ci
    lib.attn_last_kernel_cycles.argtypes = [ctypes.POINTER(ctypes.c_ulonglong)]
    lib.attn_last_error.restype = ctypes.c_char_p
    tdt = torch.float16 if args.fp16 else torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(1)
    q, k, v = (torch.randn((B, H, N, d), device="cuda", generator=g, dtype=torch.float32).to(tdt) for _ in range(3))
    o = torch.empty_like(q)
    stream = torch.cuda.current_stream().cuda_stream

    def launch():
        rc = lib.attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, 1.0 / float(np.sqrt(d)), int(args.causal),
                          0 if args.cyclic else 1, 0 if args.fp16 else 1, stream)
        if rc != 0:
            raise RuntimeError(lib.attn_last_error().decode())

    for _ in range(3):
        launch()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    launch()
    e1.record()
    torch.cuda.synchronize()
    table = (ctypes.c_ulonglong * (256 * 32))()
    if lib.attn_debug_profile(table) != 0:
        raise RuntimeError(lib.attn_last_error().decode())
    cycles = ctypes.c_ulonglong(0)
    lib.attn_last_kernel_cycles(ctypes.byref(cycles))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    # K/V steps per CTA from the host replay of the schedule (the normal library's; the schedule is the same).
    import paper_2601_16032_b200 as sa
    trace = sa.attn_schedule_trace(B, H, N, d, int(args.causal), sa.CYCLIC if args.cyclic else sa.SAWTOOTH,
                                   sa.F16 if args.fp16 else sa.BF16, None, sms)
    per_cta = {}
    for e in trace:
        per_cta[e.cta] = per_cta.get(e.cta, 0) + e.n_kv
    grid = len(per_cta)
    a = np.frombuffer(table, dtype=np.uint64).reshape(256, 32)[:min(grid, 256)].astype(np.float64)
    steps = float(np.median([per_cta[c] for c in range(min(grid, 256))]))  # K/V steps of the median CTA
    cycles.value = int(cycles.value * steps / per_cta[0])                  # CTA 0's cycle count, scaled to that many steps
    ms = e0.elapsed_time(e1)
    flops = 4.0 * B * H * float(N) ** 2 * d / (2 if args.causal else 1)
    print(f"B={B} H={H} N={N} d={d} {'fp16' if args.fp16 else 'bf16'} {'causal' if args.causal else 'non-causal'} "
          f"{'cyclic' if args.cyclic else 'sawtooth'}: {ms:.3f} ms, {flops / ms / 1e9:.0f} TFLOP/s with stamps, "
          f"{cycles.value / steps:.0f} cycles per K/V step, {cycles.value / ms / 1e3:.0f} MHz")
    med = np.median(a, axis=0) / steps
    print("MMA-issuing lane of Q tile 0, cycles per K/V step:")
    for i, n in enumerate(MMA_PHASES):
        print(f"  {n:42s} {med[i]:8.0f}")
    print(f"  {'sum':42s} {med[:len(MMA_PHASES)].sum():8.0f}")
    print("softmax thread (row 0 of Q tile 0), cycles per K/V step:")
    for i, n in enumerate(SOFTMAX_PHASES):
        print(f"  {n:42s} {med[12 + i]:8.0f}")
    print(f"  {'sum':42s} {med[12:12 + len(SOFTMAX_PHASES)].sum():8.0f}")


if __name__ == "__main__":
    main()
