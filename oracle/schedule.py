"""The paper's tile schedule, written out in plain Python (test infrastructure).

Algorithm 2 (persistent CTAs, grid-stride loop): G = min(N_tiles, N_SM) CTAs; CTA c handles the
linear work indices k = c, c + G, c + 2G, ... while k < N_tiles.  Each k names one
(batch, head, Q tile).  The paper does not say which of the three varies fastest; here the Q tile
does, then the head, then the batch ("tile_fastest"), so that CTAs running side by side stream
the K/V of the same head, which is the reuse between wavefronts that the paper observes.
"head_fastest" is the alternative order (head, then Q tile, then batch).

Algorithm 4 (sawtooth): every CTA counts the Q tiles it has handled so far (i_local).  On an even
count it scans its K/V tiles from the first to the last, on an odd count from the last to the
first.  The cyclic order always scans from the first to the last.

Causal mask: Q tile t (rows t*W .. min(N,(t+1)*W)-1) needs K/V tiles 0 .. hi-1 with
hi = ceil(min(N,(t+1)*W) / B_c); the tiles beyond are never visited, in either direction.

Pairs (the tile-based form of the sawtooth, where one trip of the persistent loop takes two Q tiles, the
first scanned forward and the second backward): with pairing the units that Algorithm 2's walk
hands out are pairs of Q tiles of one head, handled one after the other by the same CTA.
"adjacent" pairs are (2p, 2p+1).  "mirrored" pairs are (n_q-1-p, p): under the causal mask tile t
scans about t+1 tiles' worth of K/V, so the two members of a mirrored pair scan n_q+1 between them
whatever p is, and all units take the same time.  An odd middle tile forms a unit of its own.
i_local still counts Q tiles, so in the sawtooth order the first member of a pair is scanned
forward and the second backward.

Dynamic claims (a variant of Algorithm 2 in which a CTA takes the next unclaimed index from a shared
counter instead of adding G to its own): claim c = 0, 1, 2, ... names the Q tile that linear index c
names, except that under the causal mask the tiles of a head are handed out from the last (longest
scan) to the first.  Which CTA gets a claim is not determined; the scan direction is, by the round
of the claim, c // G: the value i_local would have if the CTAs took their claims in turn.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

CYCLIC = 0
SAWTOOTH = 1


@dataclass(frozen=True)
class WorkItem:
    cta: int
    i_local: int
    k: int
    batch: int
    head: int
    q_tile: int
    backward: bool
    n_kv: int  # K/V tiles this Q tile visits (0 .. n_kv-1)
    member: int = 0  # which Q tile of its pair this is (0 without pairing)

    def kv_order(self) -> range:
        return range(self.n_kv - 1, -1, -1) if self.backward else range(self.n_kv)


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def grid_size(n_tiles: int, n_sm: int) -> int:
    """Algorithm 2: one persistent CTA per SM, never more CTAs than Q tiles."""
    return min(n_tiles, n_sm)


def decode(k: int, B: int, H: int, n_q: int, digit_order: str = "tile_fastest") -> tuple[int, int, int]:
    """Linear work index -> (batch, head, Q tile)."""
    if digit_order == "tile_fastest":
        t = k % n_q
        h = (k // n_q) % H
        b = k // (n_q * H)
    elif digit_order == "head_fastest":
        h = k % H
        t = (k // H) % n_q
        b = k // (n_q * H)
    else:
        raise ValueError(digit_order)
    return b, h, t


def kv_tiles_needed(t: int, N: int, W: int, B_c: int, causal: bool) -> int:
    if not causal:
        return ceil_div(N, B_c)
    last_row_excl = min(N, (t + 1) * W)
    return ceil_div(last_row_excl, B_c)


def unit_members(p: int, n_q: int, pairing: str) -> list[int]:
    """The Q tiles of a head that unit p of the walk holds, in the order the CTA handles them."""
    if pairing == "none":
        return [p]
    if pairing == "mirrored":
        far, near = n_q - 1 - p, p
        return [far] if far == near else [far, near]
    if pairing == "adjacent":
        return [t for t in (2 * p, 2 * p + 1) if t < n_q]
    raise ValueError(pairing)


def units_per_head(n_q: int, pairing: str) -> int:
    return n_q if pairing == "none" else ceil_div(n_q, 2)


def cta_sequence(cta: int, G: int, B: int, H: int, N: int, W: int, B_c: int, causal: bool,
                 scan_order: int, digit_order: str = "tile_fastest", pairing: str = "none") -> Iterator[WorkItem]:
    """The Q tiles one CTA handles, in order, each with its K/V scan (Algorithms 2 and 4)."""
    n_q = ceil_div(N, W)
    n_u = units_per_head(n_q, pairing)
    n_units = B * H * n_u
    i_local = 0
    k = cta
    while k < n_units:
        b, h, p = decode(k, B, H, n_u, digit_order)
        for member, t in enumerate(unit_members(p, n_q, pairing)):
            backward = scan_order == SAWTOOTH and i_local % 2 == 1
            yield WorkItem(cta, i_local, k, b, h, t, backward, kv_tiles_needed(t, N, W, B_c, causal), member)
            i_local += 1
        k += G


def full_schedule(n_sm: int, B: int, H: int, N: int, W: int, B_c: int, causal: bool,
                  scan_order: int, digit_order: str = "tile_fastest", max_ctas: int = 0,
                  pairing: str = "none") -> list[list[WorkItem]]:
    n_units = B * H * units_per_head(ceil_div(N, W), pairing)
    G = grid_size(n_units, n_sm if max_ctas <= 0 else min(n_sm, max_ctas))
    return [list(cta_sequence(c, G, B, H, N, W, B_c, causal, scan_order, digit_order, pairing)) for c in range(G)]


def dynamic_claims(n_sm: int, B: int, H: int, N: int, W: int, B_c: int, causal: bool, scan_order: int,
                   digit_order: str = "tile_fastest", max_ctas: int = 0) -> list[WorkItem]:
    """The Q tiles in the order in which the dynamic schedule hands them out (cta = -1: not determined)."""
    n_q = ceil_div(N, W)
    n_work = B * H * n_q
    G = grid_size(n_work, n_sm if max_ctas <= 0 else min(n_sm, max_ctas))
    out = []
    for c in range(n_work):
        b, h, pos = decode(c, B, H, n_q, digit_order)
        t = n_q - 1 - pos if causal else pos
        rnd = c // G
        backward = scan_order == SAWTOOTH and rnd % 2 == 1
        out.append(WorkItem(-1, rnd, c, b, h, t, backward, kv_tiles_needed(t, N, W, B_c, causal)))
    return out
