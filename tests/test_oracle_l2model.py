"""Pins of the L2 sector model (the paper's tables) and of the LRU simulator (stack-distance law)."""
import os

import pytest

from oracle import l2model, schedule as sch


def read_table(path):
    rows = []
    for line in open(path):
        line = line.split("#")[0].strip()
        if line:
            rows.append([int(x) for x in line.split()])
    return rows


def test_model_reproduces_table2_exactly(golden_dir):
    for S, T, D, E, C, sectors in read_table(os.path.join(golden_dir, "table2_l2_sectors.txt")):
        assert l2model.sectors_per_head(S, T, T, D, E, C, causal=False) == sectors


def test_model_close_to_table1(golden_dir):
    for S, T, D, E, C, sectors in read_table(os.path.join(golden_dir, "table1_l2_sectors.txt")):
        got = l2model.sectors_per_head(S, T, T, D, E, C, causal=False)
        assert abs(got - sectors) / sectors < 0.0025


def test_closed_forms():
    S, T = 32768, 80
    assert l2model.sectors_paper_approx(S, T) == pytest.approx(8 * S * (1 + S / T))
    assert l2model.sectors_paper_approx_causal(S, T) == pytest.approx(8 * S * (S / (2 * T) + 0.5))
    assert l2model.cold_sectors(S, 64) == 16 * S
    # exact count when T divides S: n Q tiles, each streaming all of K and V
    S, T = 4096, 128
    assert l2model.sectors_per_head(S, T, T, 64) == l2model.sectors_paper_approx(S, T)
    # causal, T | S: n(n+1)/2 K/V tile visits (the diagonal tiles are loaded)
    n = S // T
    tile = T * 64 * 2 // 32
    assert l2model.sectors_per_head(S, T, T, 64, causal=True) == 2 * n * tile + 2 * tile * n * (n + 1) // 2
    # the printed causal form counts n(n-1)/2 visits: it is below the exact count by the diagonal
    assert l2model.sectors_per_head(S, T, T, 64, causal=True) - l2model.sectors_paper_approx_causal(S, T) == \
        pytest.approx(2 * tile * n)


def test_wider_q_tiles_share_one_kv_stream():
    a = l2model.sectors_per_head(8192, 128, 128, 128)
    b = l2model.sectors_per_head(8192, 256, 128, 128)
    qo = 2 * 8192 * 8
    assert (a - qo) == 2 * (b - qo)


@pytest.mark.parametrize("n,c", [(10, 4), (16, 15), (7, 1), (12, 6)])
def test_lru_stack_distance_law(n, c):
    """n tiles re-traversed through an LRU cache of c < n tiles: cyclic misses n per pass,
    sawtooth n - c per pass after the first."""
    passes = 6
    cyclic = [j for _ in range(passes) for j in range(n)]
    saw = [j for p in range(passes) for j in (range(n) if p % 2 == 0 else range(n - 1, -1, -1))]
    assert l2model.lru_misses(cyclic, c) == passes * n
    assert l2model.lru_misses(saw, c) == n + (passes - 1) * (n - c)
    assert l2model.lru_misses(cyclic, n) == n  # everything fits: cold misses only
    assert l2model.lru_misses(saw, n) == n


def test_wavefront_trace_of_a_schedule():
    """Two CTAs, one head of 4 Q tiles and 4 K/V tiles: CTA 0 gets tiles 0, 2; CTA 1 gets 1, 3."""
    s = sch.full_schedule(2, 1, 1, 512, 128, 128, False, sch.SAWTOOTH)
    tr = list(l2model.wavefront_trace(s))
    kv = [t[2] for t in tr]
    assert kv == [0, 0, 1, 1, 2, 2, 3, 3, 3, 3, 2, 2, 1, 1, 0, 0]
    # with a cache of 2 tiles the backward pass finds tiles 3 and 2 still resident
    assert l2model.lru_misses(tr, 2) == 4 + 2
    s = sch.full_schedule(2, 1, 1, 512, 128, 128, False, sch.CYCLIC)
    assert l2model.lru_misses(l2model.wavefront_trace(s), 2) == 8


def causal_misses(n_sm, H, N, capacity_tiles, order, pairing):
    s = sch.full_schedule(n_sm, 1, H, N, 256, 128, True, order, pairing=pairing)
    return l2model.lru_misses(l2model.wavefront_trace(s), capacity_tiles)


@pytest.mark.parametrize("heads_in_cache", [0.5, 2])
def test_lru_on_causal_schedules_unpaired_sawtooth_loses_and_mirrored_pairs_win(heads_in_cache):
    """A scaled-down causal workload (16 CTAs, 8 heads of 64 K/V tiles, 256-row items) through an ideal LRU cache.
    Without pairs the items of a wave differ in length, the CTAs drift apart, and backward scans that start at each
    item's own diagonal make it worse: the sawtooth order misses more than the cyclic one.  With mirrored pairs every
    unit is equally long, the wave stays on a few tiles, and the sawtooth order is never the worse one."""
    n_sm, H, N = 16, 8, 8192
    cap = int(heads_in_cache * N // 128)
    compulsory = H * N // 128
    none_cyc = causal_misses(n_sm, H, N, cap, sch.CYCLIC, "none")
    none_saw = causal_misses(n_sm, H, N, cap, sch.SAWTOOTH, "none")
    mir_cyc = causal_misses(n_sm, H, N, cap, sch.CYCLIC, "mirrored")
    mir_saw = causal_misses(n_sm, H, N, cap, sch.SAWTOOTH, "mirrored")
    assert none_saw > none_cyc > 4 * compulsory
    assert compulsory <= mir_saw <= mir_cyc <= 2 * compulsory
    assert mir_saw * 4 < none_cyc


def test_mirrored_sawtooth_wave_reads_two_tiles_at_a_time():
    """One head, W = B_c, CTAs in lockstep: a CTA on pair p reads tile t at step t < n-p (first member, forward) and tile
    n - t afterwards (second member, backward), whatever p is, so the whole wave touches at most two tiles per step."""
    N, W, n_sm = 4096, 128, 8
    n = N // W
    s = sch.full_schedule(n_sm, 1, 1, N, W, W, True, sch.SAWTOOTH, pairing="mirrored")
    per_cta = [[j for w in seq[:2] for j in w.kv_order()] for seq in s]     # every CTA's first unit
    assert all(len(steps) == n + 1 for steps in per_cta)
    for t in range(n + 1):
        tiles = {steps[t] for steps in per_cta}
        assert tiles <= {t, n - t}
    # the cyclic order spreads the second members over as many tiles as there are CTAs
    c = sch.full_schedule(n_sm, 1, 1, N, W, W, True, sch.CYCLIC, pairing="mirrored")
    per_cta = [[j for w in seq[:2] for j in w.kv_order()] for seq in c]
    assert len({steps[n - 1] for steps in per_cta}) == n_sm
