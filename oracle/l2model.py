"""The paper's L2 sector model and an ideal-LRU trace simulator (test infrastructure).

Sector model (the section that models L2 sector access): with sequence length S, tile size T, head
dimension D, element size E and sector size C, a tile is T*D*E/C sectors.  Q and O tiles are
touched once each; without the causal mask every Q tile streams all of K and all of V.  Dropping the
ragged tail the paper writes M = 2*(S*D*E/C + S^2*D*E/(T*C)), which is 8*S*(1 + S/T) for
C = 32, E = 2, D = 64.

`sectors_per_head` is the same count without the approximation and for unequal tiles: W query rows
share one K/V stream, K/V tiles hold B_c rows, and under the causal mask Q tile t streams only the
K/V tiles that hold keys 0 .. min(S,(t+1)W)-1.  The paper's causal closed form,
8*S*(S/(2T) + 1/2), counts S/T*(S/T - 1)/2 K/V tile visits, i.e. it leaves out the tiles on the
diagonal; the exact count used here includes them, because a kernel has to load them.

The reuse-distance argument of the sawtooth section is the LRU stack-distance result: when n tiles
are traversed again and again through a fully associative LRU cache of c < n tiles, the cyclic order
misses n times per traversal and the sawtooth order n - c times (after the first).  `lru_misses`
replays any access sequence through such a cache; `wavefront_trace` interleaves the CTAs' scans the
way the paper describes them, in lockstep.
"""
from __future__ import annotations

from collections import OrderedDict
from typing import Iterable, Sequence

from .schedule import WorkItem, ceil_div


def sectors_paper_approx(S: int, T: int, D: int = 64, E: int = 2, C: int = 32) -> float:
    """M = 2*(S*D*E/C + S^2*D*E/(T*C)), the non-causal closed form."""
    return 2.0 * (S * D * E / C + S * S * D * E / (T * C))


def sectors_paper_approx_causal(S: int, T: int, D: int = 64, E: int = 2, C: int = 32) -> float:
    """The causal closed form as printed, 8*S*(S/(2T) + 1/2), for general D, E, C."""
    return 2.0 * (D * E / C) * S * (S / (2.0 * T) + 0.5)


def sectors_per_head(S: int, W: int, B_c: int, D: int, E: int = 2, C: int = 32, causal: bool = False) -> int:
    """Sectors one head moves between L2 and the SMs: Q and O once, K and V once per Q tile."""
    row = D * E
    if row % C:
        raise ValueError("a row must be a whole number of sectors")
    row_sectors = row // C
    total = 2 * S * row_sectors  # Q read, O written
    for t in range(ceil_div(S, W)):
        if causal:
            kv_rows = min(S, ceil_div(min(S, (t + 1) * W), B_c) * B_c)
        else:
            kv_rows = S
        total += 2 * kv_rows * row_sectors  # K and V
    return total


def cold_sectors(S: int, D: int, E: int = 2, C: int = 32) -> int:
    """Compulsory misses of one head: Q, K, V, O once each, 4*S*D*E/C (16*S in the paper's setting)."""
    return 4 * S * D * E // C


def lru_misses(accesses: Iterable, capacity: int) -> int:
    """Misses of a fully associative LRU cache holding `capacity` equal-sized lines."""
    cache: OrderedDict = OrderedDict()
    misses = 0
    for a in accesses:
        if a in cache:
            cache.move_to_end(a)
        else:
            misses += 1
            cache[a] = True
            if len(cache) > capacity:
                cache.popitem(last=False)
    return misses


def wavefront_trace(schedule: Sequence[Sequence[WorkItem]]):
    """K/V tile accesses of all CTAs interleaved in lockstep: step s of every CTA before step s+1.

    Each access is (batch, head, kv_tile); K and V of a tile move together, so one id stands for
    both.  A CTA whose current Q tile is finished moves on to its next one at the next step.
    """
    cursors = []
    for seq in schedule:
        steps = [(w.batch, w.head, j) for w in seq for j in w.kv_order()]
        cursors.append(steps)
    longest = max((len(s) for s in cursors), default=0)
    for s in range(longest):
        for steps in cursors:
            if s < len(steps):
                yield steps[s]
