"""ctypes binding of the C ABI declared in include/sawtooth_attn.h (same names, same arguments)."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

CYCLIC, SAWTOOTH = 0, 1
F16, BF16 = 0, 1
TILE_FASTEST, HEAD_FASTEST = 0, 1
PAIR_DEFAULT, PAIR_NONE, PAIR_MIRRORED, PAIR_ADJACENT = 0, 1, 2, 3
LAYOUT_BHND, LAYOUT_BNHD = 0, 1

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libsawtooth_attn.so")
_lib = None


class AttnError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"sawtooth_attn: {message} (status {status})")
        self.status = status


class Opts(ctypes.Structure):
    """attn_fwd_opts: 0 means 'library default' for every field."""
    _fields_ = [
        ("max_ctas", ctypes.c_int), ("kv_stages", ctypes.c_int), ("block_n", ctypes.c_int),
        ("q_tiles", ctypes.c_int), ("digit_order", ctypes.c_int), ("launch_mode", ctypes.c_int),
        ("l2_policy", ctypes.c_int), ("host_chunks", ctypes.c_int), ("lse", ctypes.c_void_p), ("pairing", ctypes.c_int), ("check_mode", ctypes.c_int),
        ("kv_heads", ctypes.c_int), ("layout", ctypes.c_int), ("reserved", ctypes.c_int * 2),
    ]


class Plan(ctypes.Structure):
    _fields_ = [
        ("block_m", ctypes.c_int), ("block_n", ctypes.c_int), ("q_tiles", ctypes.c_int),
        ("rows_per_item", ctypes.c_int), ("items_per_head", ctypes.c_int), ("n_work", ctypes.c_longlong),
        ("grid", ctypes.c_int), ("threads", ctypes.c_int), ("kv_stages", ctypes.c_int),
        ("smem_bytes", ctypes.c_int), ("sm_count", ctypes.c_int), ("pairing", ctypes.c_int), ("n_units", ctypes.c_longlong),
    ]


class TraceEntry(ctypes.Structure):
    _fields_ = [
        ("cta", ctypes.c_int), ("iteration", ctypes.c_int), ("k", ctypes.c_longlong),
        ("batch", ctypes.c_int), ("head", ctypes.c_int), ("q_item", ctypes.c_int),
        ("backward", ctypes.c_int), ("n_kv", ctypes.c_int), ("n_kv_q0", ctypes.c_int), ("n_kv_q1", ctypes.c_int),
        ("member", ctypes.c_int),
    ]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libsawtooth_attn.so; raises if it has not been built (there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise AttnError(-4, f"{_LIB_PATH} is missing: build it with `python -m paper_2601_16032_b200.build`")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    shape = [ci, ci, ci, ci]
    lib.attn_fwd.argtypes = [vp, vp, vp, vp] + shape + [cf, ci, ci, ci, vp]
    lib.attn_fwd_ex.argtypes = [vp, vp, vp, vp] + shape + [cf, ci, ci, ci, vp, ctypes.POINTER(Opts)]
    lib.attn_fwd_dynamic.argtypes = [vp, vp, vp, vp] + shape + [cf, ci, ci, ci, vp, ctypes.POINTER(Opts), vp, ctypes.c_size_t]
    lib.attn_fwd_dynamic.restype = ci
    lib.attn_fwd_dynamic_noalloc.argtypes = [vp, vp, vp, vp] + shape + [cf, ci, ci, ci, vp, ctypes.POINTER(Opts)]
    lib.attn_fwd_dynamic_noalloc.restype = ci
    lib.attn_dynamic_scratch_bytes.argtypes = [ci]
    lib.attn_dynamic_scratch_bytes.restype = ctypes.c_size_t
    lib.attn_fwd_host.argtypes = [vp] * 8 + shape + [cf, ci, ci, ci, vp, ctypes.POINTER(Opts)]
    lib.attn_query_plan.argtypes = shape + [ci, ci, ctypes.POINTER(Opts), ci, ctypes.POINTER(Plan)]
    lib.attn_schedule_trace.argtypes = shape + [ci, ci, ci, ctypes.POINTER(Opts), ci, ctypes.POINTER(TraceEntry),
                                                ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
    lib.attn_host_groups.argtypes = [ctypes.c_longlong, ctypes.c_size_t, ci, ctypes.POINTER(ctypes.c_longlong), ctypes.POINTER(ci)]
    lib.attn_host_groups.restype = ci
    lib.attn_dynamic_claim_trace.argtypes = lib.attn_schedule_trace.argtypes
    lib.attn_dynamic_claim_trace.restype = ci
    lib.attn_device_status.argtypes = [ctypes.POINTER(ci)]
    lib.attn_last_kernel_cycles.argtypes = [ctypes.POINTER(ctypes.c_ulonglong)]
    lib.attn_last_kernel_cycles.restype = ci
    for name in ("attn_fwd", "attn_fwd_ex", "attn_fwd_host", "attn_query_plan", "attn_schedule_trace", "attn_device_status"):
        getattr(lib, name).restype = ci
    lib.attn_status_string.argtypes = [ci]
    lib.attn_status_string.restype = ctypes.c_char_p
    lib.attn_last_error.argtypes = []
    lib.attn_last_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def attn_status_string(status: int) -> str:
    return load_library().attn_status_string(status).decode()


def attn_last_error() -> str:
    return load_library().attn_last_error().decode()


def _check(status: int) -> None:
    if status != 0:
        raise AttnError(status, attn_last_error() or attn_status_string(status))


def _opts_ptr(opts: Optional[Opts]):
    return ctypes.byref(opts) if opts is not None else None


def attn_fwd(q: int, k: int, v: int, o: int, B: int, H: int, N: int, d: int, scale: float, causal: int,
             scan_order: int, dtype: int, stream: int = 0) -> None:
    """q, k, v, o: device addresses of contiguous [B, H, N, d] 16-bit arrays; stream: a cudaStream_t handle."""
    _check(load_library().attn_fwd(q, k, v, o, B, H, N, d, scale, int(causal), scan_order, dtype, stream))


def attn_fwd_ex(q: int, k: int, v: int, o: int, B: int, H: int, N: int, d: int, scale: float, causal: int,
                scan_order: int, dtype: int, stream: int = 0, opts: Optional[Opts] = None) -> None:
    _check(load_library().attn_fwd_ex(q, k, v, o, B, H, N, d, scale, int(causal), scan_order, dtype, stream, _opts_ptr(opts)))


def attn_dynamic_scratch_bytes(ctas: int) -> int:
    return int(load_library().attn_dynamic_scratch_bytes(ctas))


def attn_fwd_dynamic(q: int, k: int, v: int, o: int, B: int, H: int, N: int, d: int, scale: float, causal: int,
                     scan_order: int, dtype: int, stream: int = 0, opts: Optional[Opts] = None, scratch: int = 0,
                     scratch_bytes: int = 0) -> None:
    """attn_fwd_ex with the dynamic tile schedule; scratch: device address of the caller's counter buffer."""
    _check(load_library().attn_fwd_dynamic(q, k, v, o, B, H, N, d, scale, int(causal), scan_order, dtype, stream,
                                           _opts_ptr(opts), scratch, scratch_bytes))


def attn_fwd_dynamic_noalloc(q: int, k: int, v: int, o: int, B: int, H: int, N: int, d: int, scale: float, causal: int,
                             scan_order: int, dtype: int, stream: int = 0, opts: Optional[Opts] = None) -> None:
    """The dynamic schedule without a scratch argument, for callers that may not allocate device memory: the
    counters live in a fixed array inside the library (at most 1024 CTAs; calls on one device share it, so calls
    that could overlap on the GPU must be serialised; make the first call on a device outside stream capture)."""
    _check(load_library().attn_fwd_dynamic_noalloc(q, k, v, o, B, H, N, d, scale, int(causal), scan_order, dtype, stream,
                                                   _opts_ptr(opts)))


def attn_fwd_host(q_host: int, k_host: int, v_host: int, o_host: int, q_dev: int, k_dev: int, v_dev: int, o_dev: int,
                  B: int, H: int, N: int, d: int, scale: float, causal: int, scan_order: int, dtype: int,
                  stream: int = 0, opts: Optional[Opts] = None) -> None:
    _check(load_library().attn_fwd_host(q_host, k_host, v_host, o_host, q_dev, k_dev, v_dev, o_dev, B, H, N, d, scale,
                                        int(causal), scan_order, dtype, stream, _opts_ptr(opts)))


def attn_query_plan(B: int, H: int, N: int, d: int, causal: int, dtype: int, opts: Optional[Opts] = None,
                    sm_count: int = 0) -> Plan:
    plan = Plan()
    _check(load_library().attn_query_plan(B, H, N, d, int(causal), dtype, _opts_ptr(opts), sm_count, ctypes.byref(plan)))
    return plan


def attn_schedule_trace(B: int, H: int, N: int, d: int, causal: int, scan_order: int, dtype: int,
                        opts: Optional[Opts] = None, sm_count: int = 0) -> list:
    lib = load_library()
    n = ctypes.c_size_t(0)
    _check(lib.attn_schedule_trace(B, H, N, d, int(causal), scan_order, dtype, _opts_ptr(opts), sm_count, None, 0, ctypes.byref(n)))
    buf = (TraceEntry * n.value)()
    _check(lib.attn_schedule_trace(B, H, N, d, int(causal), scan_order, dtype, _opts_ptr(opts), sm_count, buf, n.value, ctypes.byref(n)))
    return list(buf)


def attn_dynamic_claim_trace(B: int, H: int, N: int, d: int, causal: int, scan_order: int, dtype: int,
                             opts: Optional[Opts] = None, sm_count: int = 0) -> list:
    lib = load_library()
    n = ctypes.c_size_t(0)
    _check(lib.attn_dynamic_claim_trace(B, H, N, d, int(causal), scan_order, dtype, _opts_ptr(opts), sm_count, None, 0, ctypes.byref(n)))
    buf = (TraceEntry * n.value)()
    _check(lib.attn_dynamic_claim_trace(B, H, N, d, int(causal), scan_order, dtype, _opts_ptr(opts), sm_count, buf, n.value, ctypes.byref(n)))
    return list(buf)


def attn_host_groups(heads: int, head_bytes: int, host_chunks: int = 0) -> list:
    """The groups of heads attn_fwd_host cuts its work into (host-only)."""
    sizes = (ctypes.c_longlong * 32)()
    n = ctypes.c_int(0)
    _check(load_library().attn_host_groups(ctypes.c_longlong(heads), ctypes.c_size_t(head_bytes), host_chunks, sizes, ctypes.byref(n)))
    return [int(sizes[i]) for i in range(n.value)]


def attn_device_status() -> int:
    """Synchronises the device; returns 0, or raises AttnError if a kernel wait ran out since the last call."""
    code = ctypes.c_int(0)
    _check(load_library().attn_device_status(ctypes.byref(code)))
    return code.value


def attn_last_kernel_cycles() -> int:
    """Synchronises the device; SM cycles the first CTA of the most recent kernel spent on its work items."""
    c = ctypes.c_ulonglong(0)
    _check(load_library().attn_last_kernel_cycles(ctypes.byref(c)))
    return int(c.value)


def forward(q, k, v, causal: bool = False, scan_order: int = SAWTOOTH, scale: Optional[float] = None,
            opts: Optional[Opts] = None, out=None):
    """Convenience wrapper for torch CUDA tensors of shape [B, H, N, d] (fp16 or bf16, contiguous).

    Marshals pointers and the current stream into attn_fwd_ex; allocates `out` with torch if not given.
    """
    import torch

    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise AttnError(-1, "q, k and v must be CUDA tensors")
    if q.dtype not in (torch.float16, torch.bfloat16) or k.dtype != q.dtype or v.dtype != q.dtype:
        raise AttnError(-1, "q, k and v must share dtype float16 or bfloat16")
    if q.dim() != 4 or k.dim() != 4 or v.shape != k.shape or k.shape[0] != q.shape[0] or k.shape[2:] != q.shape[2:] or \
            q.shape[1] % k.shape[1] != 0:
        raise AttnError(-1, "q must be [B, H, N, d], k and v [B, H_kv, N, d] with H_kv dividing H")
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
        raise AttnError(-1, "q, k and v must be contiguous")
    B, H, N, d = q.shape
    if out is None:
        out = torch.empty_like(q)
    elif out.shape != q.shape or out.dtype != q.dtype or not out.is_contiguous() or not out.is_cuda:
        raise AttnError(-1, "out must match q")
    if scale is None:
        scale = 1.0 / float(d) ** 0.5
    if k.shape[1] != H:   # grouped-query attention: fewer K/V heads than query heads
        import copy
        opts = copy.copy(opts) if opts is not None else Opts()
        opts.kv_heads = int(k.shape[1])
    stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), B, H, N, d, float(scale), int(causal),
                    scan_order, BF16 if q.dtype == torch.bfloat16 else F16, stream, opts)
    return out
