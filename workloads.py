"""Seeded synthetic attention workloads (inputs only; no attention arithmetic lives here).

This module serves both the CPU oracle and the CUDA path: it draws the Q, K, V tensors as
16-bit patterns (IEEE fp16 or bfloat16, round-to-nearest-even from an fp32 normal draw), widens
such patterns exactly to fp64 for the oracle, and picks the query rows that are checked at sizes
where checking every row would take too long.  Nothing here computes a score, a softmax or an
output.

The shapes follow the paper's sweeps (batch 1..8, long sequences, head dimension 64; the studies
section and the CuTile validation) and add head dimension 128 and bf16, the shapes in which
present-day models run attention.  Each head of each tensor has its own random stream, keyed by
(seed, tensor, batch, head), so one head can be produced without producing the rest.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

import numpy as np

F16 = "f16"
BF16 = "bf16"
_TENSOR_ID = {"q": 0, "k": 1, "v": 2}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    dtype: str  # F16 or BF16
    causal: bool
    seed: int
    k_scale: float = 1.0  # multiplies K before rounding (a power of two, so exact)
    block_n: int = 128  # K/V rows per tile the configuration asks for

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d))

    @property
    def flops(self) -> float:
        """4*B*H*N^2*d, halved under the causal mask (the reporting convention)."""
        f = 4.0 * self.B * self.H * float(self.N) ** 2 * self.d
        return f / 2 if self.causal else f

    @property
    def compulsory_bytes(self) -> int:
        """Q, K, V read once and O written once."""
        return 4 * self.B * self.H * self.N * self.d * 2


CONFIGS = {
    "c1": Workload("c1", 1, 1, 1024, 64, F16, False, 1001),
    "c2": Workload("c2", 1, 8, 4096, 64, F16, False, 1002, block_n=64),
    "c3": Workload("c3", 4, 16, 8192, 128, BF16, False, 1003),
    "c4": Workload("c4", 1, 32, 32768, 128, BF16, True, 1004, k_scale=0.5),
    "c5": Workload("c5", 2, 16, 65536, 128, BF16, True, 1005),
}

# Smaller or differently shaped cases for profiler captures and scan-order studies (not parity
# configurations).  "long*" follow the paper's own studies: a single head whose K+V exceeds L2.
STUDY_CASES = {
    "c3-small": Workload("c3-small", 2, 16, 8192, 128, BF16, False, 2003),
    "c4-small": Workload("c4-small", 1, 8, 32768, 128, BF16, True, 2004, k_scale=0.5),
    # The paper's head dimension at a size that fills the GPU several times over, and a capture-sized half of it.
    "d64-n8k": Workload("d64-n8k", 4, 16, 8192, 64, F16, False, 2064),
    "d64-n8k-small": Workload("d64-n8k-small", 2, 16, 8192, 64, F16, False, 2065),
    "long-64k": Workload("long-64k", 1, 1, 65536, 128, BF16, False, 2010),
    "long-128k": Workload("long-128k", 1, 1, 131072, 128, BF16, False, 2011),
    "long-192k": Workload("long-192k", 1, 1, 196608, 128, BF16, False, 2012),
    "long-256k": Workload("long-256k", 1, 1, 262144, 128, BF16, False, 2006),
    "long-384k": Workload("long-384k", 1, 1, 393216, 128, BF16, False, 2013),
    "long-512k": Workload("long-512k", 1, 1, 524288, 128, BF16, False, 2007),
    "long-128k-b8": Workload("long-128k-b8", 8, 1, 131072, 64, F16, False, 2008),
}
# The batch sweep of the paper's CUDA results (batch 1, 2, 4, 8; one head; 128k keys), at the paper's head dimension
# and at 128.
for _b in (1, 2, 4, 8):
    STUDY_CASES[f"sweep-d64-b{_b}"] = Workload(f"sweep-d64-b{_b}", _b, 1, 131072, 64, F16, False, 2100 + _b)
    STUDY_CASES[f"sweep-d128-b{_b}"] = Workload(f"sweep-d128-b{_b}", _b, 1, 131072, 128, BF16, False, 2200 + _b)
# The same shape under the causal mask (the paper's second CuTile result).
STUDY_CASES["sweep-d64-b8-causal"] = Workload("sweep-d64-b8-causal", 8, 1, 131072, 64, F16, True, 2300)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = ((u + bias) >> np.uint32(16)).astype(np.uint16)
    nan = np.isnan(x)
    if nan.any():
        out[nan] = 0x7FC0
    return out


def f32_to_f16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to IEEE fp16 (nearest, ties to even) and return the 16-bit patterns."""
    return np.ascontiguousarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)


def to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == F16:
        return f32_to_f16_bits(x)
    if dtype == BF16:
        return f32_to_bf16_bits(x)
    raise ValueError(f"unknown dtype {dtype!r}")


def bits_to_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of 16-bit patterns to fp64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == F16:
        return bits.view(np.float16).astype(np.float64)
    if dtype == BF16:
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    raise ValueError(f"unknown dtype {dtype!r}")


def head_bits(w: Workload, tensor: str, b: int, h: int) -> np.ndarray:
    """The [N, d] 16-bit patterns of one head of q, k or v: i.i.d. N(0,1), K times k_scale."""
    rng = np.random.default_rng([w.seed, _TENSOR_ID[tensor], b, h])
    x = rng.standard_normal((w.N, w.d), dtype=np.float32)
    if tensor == "k" and w.k_scale != 1.0:
        x *= np.float32(w.k_scale)
    return to_bits(x, w.dtype)


def all_heads(w: Workload) -> Iterator[tuple[int, int]]:
    for b in range(w.B):
        for h in range(w.H):
            yield b, h


def tensor_bits(w: Workload, tensor: str) -> np.ndarray:
    """The whole [B, H, N, d] tensor as 16-bit patterns (contiguous, d fastest)."""
    out = np.empty((w.B, w.H, w.N, w.d), dtype=np.uint16)
    for b, h in all_heads(w):
        out[b, h] = head_bits(w, tensor, b, h)
    return out


def edge_rows(N: int, block: int = 128) -> list[int]:
    """Rows that sit on tile edges and on the ends of the sequence."""
    cand = [0, 1, block - 1, block, 2 * block - 1, 2 * block, N // 2, N - block - 1, N - block, N - 2, N - 1]
    return sorted({r for r in cand if 0 <= r < N})


def sampled_rows(w: Workload, b: int, h: int, n_random: int) -> np.ndarray:
    """Sorted, distinct query rows of head (b, h): the tile-edge rows plus n_random seeded ones."""
    rng = np.random.default_rng([w.seed + 1, b, h])
    rnd = rng.choice(w.N, size=min(n_random, w.N), replace=False) if n_random > 0 else np.empty(0, np.int64)
    rows = np.union1d(np.asarray(edge_rows(w.N), dtype=np.int64), rnd.astype(np.int64))
    return rows


def checked_rows(w: Workload) -> dict[tuple[int, int], np.ndarray | None]:
    """Which rows of which heads the parity tests compare.  None means every row of the head.

    c1, c2: every row of every head.  c3: every row of the first and the last head, and 1024
    seeded rows spread over the others.  c4: every row of the first and the last head, 512 seeded
    rows in each other head.  c5: 512 seeded rows in every head.
    """
    heads = list(all_heads(w))
    if w.name in ("c1", "c2"):
        return {bh: None for bh in heads}
    plan: dict[tuple[int, int], np.ndarray | None] = {}
    if w.name == "c3":
        others = heads[1:-1]
        per = -(-1024 // len(others))
        plan[heads[0]] = None
        plan[heads[-1]] = None
        for bh in others:
            plan[bh] = sampled_rows(w, bh[0], bh[1], per)
        return plan
    if w.name == "c4":
        plan[heads[0]] = None
        plan[heads[-1]] = None
        for bh in heads[1:-1]:
            plan[bh] = sampled_rows(w, bh[0], bh[1], 512)
        return plan
    for bh in heads:
        plan[bh] = sampled_rows(w, bh[0], bh[1], 512)
    return plan


def small_workload(name: str, B: int, H: int, N: int, d: int, dtype: str, causal: bool, seed: int,
                   k_scale: float = 1.0, block_n: int = 128) -> Workload:
    """A workload of any shape, for ragged and tiny parity cases."""
    return Workload(name, B, H, N, d, dtype, causal, seed, k_scale, block_n)
