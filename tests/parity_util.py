"""Shared helpers of the GPU parity tests: upload a seeded workload, run the CUDA path through the
C ABI, and compare sampled or full rows with the fp64 oracle."""
from __future__ import annotations

import numpy as np

import workloads as wl

MAX_ABS_TOL = 2e-2   # the bar stated for fp16 / bf16 outputs, against the fp64 oracle
MEAN_ABS_TOL = 2e-3


def torch_dtype(dtype: str):
    import torch
    return torch.bfloat16 if dtype == wl.BF16 else torch.float16


def upload(w: wl.Workload, device="cuda:0"):
    """q, k, v as [B, H, N, d] CUDA tensors holding exactly the workload's 16-bit patterns."""
    import torch
    out = []
    for name in ("q", "k", "v"):
        t = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.int16, device=device)
        for b, h in wl.all_heads(w):
            t[b, h].copy_(torch.from_numpy(wl.head_bits(w, name, b, h).view(np.int16)))
        out.append(t.view(torch_dtype(w.dtype)))
    return out


def run_cuda(w: wl.Workload, qkv, scan_order: int, opts=None):
    import torch
    import paper_2601_16032_b200 as sa
    q, k, v = qkv
    o = torch.full_like(q, float("nan"))
    sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal),
                   scan_order, sa.BF16 if w.dtype == wl.BF16 else sa.F16, torch.cuda.current_stream().cuda_stream, opts)
    sa.attn_device_status()  # synchronises; raises if a wait inside the kernel ran out
    return o


def output_bits(o, b: int, h: int, rows=None) -> np.ndarray:
    import torch
    t = o[b, h] if rows is None else o[b, h][torch.as_tensor(rows, device=o.device)]
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _head_f64(w: wl.Workload, b: int, h: int):
    return tuple(wl.bits_to_f64(wl.head_bits(w, n, b, h), w.dtype) for n in ("q", "k", "v"))


def oracle_rows(w: wl.Workload, plan) -> dict:
    """The oracle's output for the planned rows: {(b, h): (row indices, [n_rows, d] fp64)}."""
    from oracle import attention as ora
    want = {}
    for (b, h), rows in plan.items():
        q, k, v = _head_f64(w, b, h)
        idx = np.arange(w.N, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
        want[(b, h)] = (idx, ora.attention_rows(q[idx], idx, k, v, w.scale, w.causal))
    return want


def compare_rows(w: wl.Workload, o, plan, want):
    """(max_abs, mean_abs, n_rows) of the CUDA output `o` against precomputed oracle rows."""
    max_abs, total, count, n_rows = 0.0, 0.0, 0, 0
    for (b, h), rows in plan.items():
        idx, ref = want[(b, h)]
        got = wl.bits_to_f64(output_bits(o, b, h, None if rows is None else idx), w.dtype)
        assert np.isfinite(got).all(), f"non-finite output in head ({b},{h})"
        err = np.abs(got - ref)
        max_abs = max(max_abs, float(err.max()))
        total += float(err.sum())
        count += err.size
        n_rows += len(idx)
    return max_abs, total / count, n_rows


def compare_with_oracle(w: wl.Workload, o, plan=None):
    """Returns (max_abs, mean_abs, n_rows) of the CUDA output against the oracle on the planned rows."""
    plan = plan if plan is not None else wl.checked_rows(w)
    return compare_rows(w, o, plan, oracle_rows(w, plan))


def assert_parity(w: wl.Workload, o, plan=None):
    max_abs, mean_abs, n_rows = compare_with_oracle(w, o, plan)
    assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, \
        f"{w.name}: max_abs {max_abs:.3e} mean_abs {mean_abs:.3e} over {n_rows} rows"
    return max_abs, mean_abs
