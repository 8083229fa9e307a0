"""fp64 attention oracle (test infrastructure; the CUDA path never touches it).

Three statements of the same result (and, beside them, the logarithm of the softmax denominator per row,
`logsumexp_definition` / `logsumexp_rows`, which the CUDA path can emit as a second output):

* `attention_definition` -- Eq. 1 written out with numpy: the full N x N score matrix, a row
  softmax, a product with V.  It is the reference for small cases.
* `attention_rows` -- the same definition for a chosen set of query rows of one head, computed by
  the C routine in attn_ref.c (two passes per row, threaded over rows).  It is what the GPU output
  is compared with at every size, and what the benchmark times as its CPU baseline.
* `attention_online` -- Algorithm 1 step by step (resident Q tile, streamed K/V tiles, running
  max m, running sum l, rescaled accumulator O), with the order in which the K/V tiles are
  visited given by the caller.  It exists to show that the cyclic and the sawtooth scans of
  Algorithm 4 reach the result of the definition.

Inputs are fp64 arrays (16-bit patterns widened exactly by the workload module).  `scale` is the
factor Algorithm 1 multiplies S by; Eq. 1 fixes it to 1/sqrt(d).  Under the causal mask query i
sees keys 0..i.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

_lib = None


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        lib.attn_ref_rows.restype = ctypes.c_int
        lib.attn_ref_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_double, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
        ]
        lib.attn_ref_lse_rows.restype = ctypes.c_int
        lib.attn_ref_lse_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
            ctypes.c_double, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
        ]
        lib.attn_ref_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads_available() -> int:
    """Worker threads the C routine uses when asked for 'all'."""
    return int(_c().attn_ref_threads())


def attention_definition(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float, causal: bool) -> np.ndarray:
    """Eq. 1 for one head: O = softmax(scale * Q K^T) V, rows of Q against all (visible) keys."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    n_q, n_k = q.shape[0], k.shape[0]
    s = scale * (q @ k.T)
    if causal:
        i = np.arange(n_q)[:, None]
        j = np.arange(n_k)[None, :]
        s = np.where(j <= i, s, -np.inf)
    p = np.exp(s - s.max(axis=1, keepdims=True))
    return (p @ v) / p.sum(axis=1, keepdims=True)


def attention_rows(q_rows: np.ndarray, row_index: np.ndarray, k: np.ndarray, v: np.ndarray,
                   scale: float, causal: bool, threads: int = 0) -> np.ndarray:
    """Eq. 1 for the query rows `q_rows` (positions `row_index`) of one head, via attn_ref.c."""
    q_rows = np.ascontiguousarray(q_rows, np.float64)
    row_index = np.ascontiguousarray(row_index, np.int64)
    k = np.ascontiguousarray(k, np.float64)
    v = np.ascontiguousarray(v, np.float64)
    n_rows, d = q_rows.shape
    N = k.shape[0]
    if k.shape != (N, d) or v.shape != (N, d) or row_index.shape != (n_rows,):
        raise ValueError("shape mismatch")
    out = np.empty((n_rows, d), np.float64)
    rc = _c().attn_ref_rows(q_rows.ctypes.data, row_index.ctypes.data, n_rows, k.ctypes.data, v.ctypes.data,
                            N, d, float(scale), int(bool(causal)), int(threads), out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"attn_ref_rows failed ({rc})")
    return out


def logsumexp_definition(q: np.ndarray, k: np.ndarray, scale: float, causal: bool) -> np.ndarray:
    """ln of Eq. 1's softmax denominator per query row: ln sum_j exp(scale * q_i . k_j) over the visible keys."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    s = scale * (q @ k.T)
    if causal:
        i = np.arange(q.shape[0])[:, None]
        j = np.arange(k.shape[0])[None, :]
        s = np.where(j <= i, s, -np.inf)
    m = s.max(axis=1)
    return m + np.log(np.exp(s - m[:, None]).sum(axis=1))


def logsumexp_rows(q_rows: np.ndarray, row_index: np.ndarray, k: np.ndarray, scale: float, causal: bool,
                   threads: int = 0) -> np.ndarray:
    """The same per-row logarithm for chosen query rows of one head, via attn_ref.c."""
    q_rows = np.ascontiguousarray(q_rows, np.float64)
    row_index = np.ascontiguousarray(row_index, np.int64)
    k = np.ascontiguousarray(k, np.float64)
    n_rows, d = q_rows.shape
    N = k.shape[0]
    if k.shape != (N, d) or row_index.shape != (n_rows,):
        raise ValueError("shape mismatch")
    out = np.empty(n_rows, np.float64)
    rc = _c().attn_ref_lse_rows(q_rows.ctypes.data, row_index.ctypes.data, n_rows, k.ctypes.data, N, d, float(scale),
                                int(bool(causal)), int(threads), out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"attn_ref_lse_rows failed ({rc})")
    return out


def attention_head(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float, causal: bool, threads: int = 0) -> np.ndarray:
    """Every row of one head through the C routine."""
    return attention_rows(q, np.arange(q.shape[0], dtype=np.int64), k, v, scale, causal, threads)


def attention_online(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale: float, causal: bool,
                     T_r: int, T_c: int, kv_order) -> np.ndarray:
    """Algorithm 1 for one head, in fp64.

    The sequence is cut into Q tiles of T_r rows and K/V tiles of T_c rows (the paper uses
    T_r = T_c = T).  `kv_order(i, n_kv)` returns the order in which Q tile i visits the K/V tile
    indices 0..n_kv-1 it needs: Algorithm 4's forward or backward scan.  Under the causal mask a Q
    tile needs only the K/V tiles that hold a key some row of it may see.
    """
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    N, d = q.shape
    out = np.empty((N, d), np.float64)
    n_q_tiles = -(-N // T_r)
    for i in range(n_q_tiles):
        r0, r1 = i * T_r, min(N, (i + 1) * T_r)
        Qi = q[r0:r1]                                  # load Q_i (resident)
        Oi = np.zeros((r1 - r0, d))                    # O_i = 0
        li = np.zeros(r1 - r0)                         # l_i = 0
        mi = np.full(r1 - r0, -np.inf)                 # m_i = -inf
        n_kv = -(-N // T_c)
        if causal:
            n_kv = -(-r1 // T_c)                       # tiles holding keys 0 .. r1-1
        for j in kv_order(i, n_kv):
            c0, c1 = j * T_c, min(N, (j + 1) * T_c)
            Kj, Vj = k[c0:c1], v[c0:c1]                # load K_j, V_j
            S = (Qi @ Kj.T) * scale                    # S_ij = Q_i K_j^T, times scale
            if causal:
                rows = np.arange(r0, r1)[:, None]
                cols = np.arange(c0, c1)[None, :]
                S = np.where(cols <= rows, S, -np.inf)
            m_new = np.maximum(mi, S.max(axis=1))      # update the running max
            alpha = np.where(np.isneginf(m_new), 1.0, np.exp(mi - np.where(np.isneginf(m_new), 0.0, m_new)))
            P = np.exp(S - np.where(np.isneginf(m_new), 0.0, m_new)[:, None])
            P = np.where(np.isneginf(S), 0.0, P)
            li = li * alpha + P.sum(axis=1)            # update the running sum
            Oi = Oi * alpha[:, None] + P @ Vj          # O_i <- O_i + P_ij V_j, O_i rescaled first
            mi = m_new
        out[r0:r1] = Oi / li[:, None]                  # write O_i
    return out


def scan_forward(i: int, n_kv: int):
    """Cyclic order: every Q tile visits K/V tiles 0, 1, ..., n_kv-1."""
    return range(n_kv)


def scan_backward(i: int, n_kv: int):
    return range(n_kv - 1, -1, -1)
