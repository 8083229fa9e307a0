"""Pins of the schedule oracle (Algorithms 2 and 4): coverage, alternation, causal ranges."""
import itertools

import pytest

from oracle import schedule as sch

SHAPES = [
    # n_sm, B, H, N, W, B_c
    (4, 1, 1, 1024, 128, 128),
    (148, 1, 8, 4096, 128, 64),
    (5, 2, 3, 1000, 128, 64),
    (7, 1, 2, 777, 256, 128),
    (148, 1, 1, 130, 128, 128),
]


@pytest.mark.parametrize("n_sm,B,H,N,W,B_c", SHAPES)
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("order", [sch.CYCLIC, sch.SAWTOOTH])
@pytest.mark.parametrize("digits", ["tile_fastest", "head_fastest"])
def test_every_q_tile_exactly_once_and_grid_stride(n_sm, B, H, N, W, B_c, causal, order, digits):
    s = sch.full_schedule(n_sm, B, H, N, W, B_c, causal, order, digits)
    n_q = sch.ceil_div(N, W)
    n_tiles = B * H * n_q
    assert len(s) == min(n_tiles, n_sm)  # G = min(N_tiles, N_SM)
    seen = sorted((w.batch, w.head, w.q_tile) for seq in s for w in seq)
    assert seen == sorted(itertools.product(range(B), range(H), range(n_q)))
    for c, seq in enumerate(s):
        assert [w.k for w in seq] == list(range(c, n_tiles, len(s)))  # k = blockIdx, += G
        assert [w.i_local for w in seq] == list(range(len(seq)))
        for w in seq:
            if order == sch.CYCLIC:
                assert not w.backward
            else:
                assert w.backward == (w.i_local % 2 == 1)  # even forward, odd backward
            ks = list(w.kv_order())
            assert sorted(ks) == list(range(w.n_kv))  # each needed K/V tile once
            assert ks == (list(range(w.n_kv - 1, -1, -1)) if w.backward else list(range(w.n_kv)))


@pytest.mark.parametrize("N,W,B_c", [(1024, 128, 128), (1000, 128, 64), (777, 256, 128), (130, 128, 128), (1, 128, 128)])
def test_causal_range_is_exactly_the_tiles_holding_a_visible_key(N, W, B_c):
    for t in range(sch.ceil_div(N, W)):
        rows = range(t * W, min(N, (t + 1) * W))
        needed = {j // B_c for i in rows for j in range(i + 1)}  # brute force over (row, key) pairs
        assert needed == set(range(sch.kv_tiles_needed(t, N, W, B_c, True)))
        assert sch.kv_tiles_needed(t, N, W, B_c, False) == sch.ceil_div(N, B_c)


def test_digit_orders():
    assert sch.decode(0, 2, 3, 4) == (0, 0, 0)
    assert sch.decode(5, 2, 3, 4) == (0, 1, 1)       # tile fastest: k = (b*H + h)*n_q + t
    assert sch.decode(23, 2, 3, 4) == (1, 2, 3)
    assert sch.decode(5, 2, 3, 4, "head_fastest") == (0, 2, 1)  # k = (b*n_q + t)*H + h
    assert sch.decode(23, 2, 3, 4, "head_fastest") == (1, 2, 3)


def test_max_ctas_limits_the_grid():
    s = sch.full_schedule(148, 1, 1, 4096, 128, 128, False, sch.SAWTOOTH, max_ctas=3)
    assert len(s) == 3
    assert [w.q_tile for w in s[1]] == list(range(1, 32, 3))


@pytest.mark.parametrize("n_sm,B,H,N,W,B_c", SHAPES + [(3, 1, 2, 2305, 256, 128), (6, 2, 1, 4096, 256, 128)])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("order", [sch.CYCLIC, sch.SAWTOOTH])
@pytest.mark.parametrize("pairing", ["mirrored", "adjacent"])
def test_pairs_cover_every_q_tile_once_and_alternate(n_sm, B, H, N, W, B_c, causal, order, pairing):
    s = sch.full_schedule(n_sm, B, H, N, W, B_c, causal, order, "tile_fastest", pairing=pairing)
    n_q = sch.ceil_div(N, W)
    n_units = B * H * sch.ceil_div(n_q, 2)
    assert len(s) == min(n_units, n_sm)
    seen = sorted((w.batch, w.head, w.q_tile) for seq in s for w in seq)
    assert seen == sorted(itertools.product(range(B), range(H), range(n_q)))
    for c, seq in enumerate(s):
        assert sorted(set(w.k for w in seq)) == list(range(c, n_units, len(s)))   # units: k = blockIdx, += G
        assert [w.i_local for w in seq] == list(range(len(seq)))
        for w in seq:
            assert w.backward == (order == sch.SAWTOOTH and w.i_local % 2 == 1)
        for k, grp in itertools.groupby(seq, key=lambda w: w.k):
            grp = list(grp)
            assert [w.member for w in grp] == list(range(len(grp))) and 1 <= len(grp) <= 2
            assert len({(w.batch, w.head) for w in grp}) == 1                     # both tiles of a pair in one head
            p = k % sch.ceil_div(n_q, 2)
            if pairing == "mirrored":
                assert [w.q_tile for w in grp] == ([n_q - 1 - p, p] if n_q - 1 - p != p else [p])
            else:
                assert [w.q_tile for w in grp] == [t for t in (2 * p, 2 * p + 1) if t < n_q]


def test_mirrored_pairs_are_equally_long_under_the_causal_mask():
    """Tile t scans t+1 tiles' worth of K/V when W = B_c divides N, so the members of pair p scan (n-p) + (p+1) = n+1."""
    N, W = 4096, 128
    n_q = N // W
    s = sch.full_schedule(5, 1, 3, N, W, W, True, sch.SAWTOOTH, pairing="mirrored")
    for seq in s:
        for _, grp in itertools.groupby(seq, key=lambda w: w.k):
            assert sum(w.n_kv for w in grp) == n_q + 1
    # without pairs the items of one CTA differ in length by up to the whole sequence
    lengths = [w.n_kv for seq in sch.full_schedule(5, 1, 3, N, W, W, True, sch.SAWTOOTH) for w in seq]
    assert min(lengths) == 1 and max(lengths) == n_q
