"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, validates
arguments, and its host-side schedule replay agrees entry by entry with the schedule oracle."""
import ctypes
import os
import re

import pytest

import paper_2601_16032_b200 as sa
from oracle import schedule as sch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    from conftest import nvcc_available
    from paper_2601_16032_b200 import build
    if not nvcc_available() and not os.path.exists(sa.library_path()):
        pytest.skip("the C-ABI library is not built and there is no nvcc to build it with")
    if nvcc_available():
        build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sawtooth_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(attn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(sa.library_path())
    names = declared_functions()
    assert {"attn_fwd", "attn_fwd_ex", "attn_fwd_host", "attn_query_plan", "attn_schedule_trace",
            "attn_device_status", "attn_status_string", "attn_last_error"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None


def test_status_strings():
    assert sa.attn_status_string(0) == "ok"
    for s in range(-6, 0):
        assert sa.attn_status_string(s) not in ("ok", "unknown status")
    assert sa.attn_status_string(-99) == "unknown status"


def test_plan_matches_algorithm_2():
    p = sa.attn_query_plan(4, 16, 8192, 128, 0, sa.BF16, sm_count=148)
    assert (p.block_m, p.block_n, p.q_tiles, p.rows_per_item) == (128, 128, 2, 256)
    assert p.items_per_head == 32 and p.n_work == 2048 and p.grid == 148  # G = min(N_tiles, N_SM)
    assert p.smem_bytes <= 232448 and p.kv_stages >= 2
    p = sa.attn_query_plan(1, 1, 1024, 64, 0, sa.F16, sm_count=148)
    assert p.n_work == 4 and p.grid == 4
    o = sa.Opts()
    o.q_tiles, o.block_n, o.max_ctas = 1, 64, 5
    p = sa.attn_query_plan(1, 8, 4096, 64, 0, sa.F16, o, sm_count=148)
    assert (p.rows_per_item, p.block_n, p.n_work, p.grid) == (128, 64, 256, 5)
    o = sa.Opts()
    o.launch_mode = 1  # Algorithm 3: one CTA per work item
    assert sa.attn_query_plan(1, 8, 4096, 64, 0, sa.F16, o, sm_count=148).grid == 128


def test_argument_validation_without_a_device():
    cases = [
        (dict(B=0), -1), (dict(N=-3), -1), (dict(d=80), -2), (dict(causal=3), -1), (dict(dtype=9), -1),
    ]
    for change, status in cases:
        a = dict(B=1, H=1, N=128, d=64, causal=0, dtype=0)
        a.update(change)
        with pytest.raises(sa.AttnError) as e:
            sa.attn_query_plan(a["B"], a["H"], a["N"], a["d"], a["causal"], a["dtype"], sm_count=148)
        assert e.value.status == status
    bad = sa.Opts()
    bad.block_n = 96
    with pytest.raises(sa.AttnError):
        sa.attn_query_plan(1, 1, 128, 64, 0, 0, bad, sm_count=148)
    bad = sa.Opts()
    bad.kv_stages = 99
    with pytest.raises(sa.AttnError):
        sa.attn_query_plan(1, 1, 128, 128, 0, 0, bad, sm_count=148)
    with pytest.raises(sa.AttnError) as e:
        sa.attn_fwd(0, 0, 0, 0, 1, 1, 128, 64, 0.125, 0, 0, 0)
    assert e.value.status == -1 and "non-null" in str(e.value)


SHAPES = [
    # n_sm, B, H, N, d, q_tiles, block_n
    (4, 1, 1, 1024, 64, 2, 128),
    (148, 1, 8, 4096, 64, 2, 64),
    (5, 2, 3, 1000, 128, 1, 64),
    (7, 1, 2, 777, 128, 2, 128),
    (148, 1, 1, 130, 64, 2, 128),
    (3, 2, 2, 2049, 128, 2, 64),
]


@pytest.mark.parametrize("n_sm,B,H,N,d,q_tiles,block_n", SHAPES)
@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("order", [sa.CYCLIC, sa.SAWTOOTH])
@pytest.mark.parametrize("digits", [sa.TILE_FASTEST, sa.HEAD_FASTEST])
def test_schedule_replay_equals_the_schedule_oracle(n_sm, B, H, N, d, q_tiles, block_n, causal, order, digits):
    check_replay(n_sm, B, H, N, d, q_tiles, block_n, causal, order, digits, sa.PAIR_NONE, "none")


@pytest.mark.parametrize("n_sm,B,H,N,d,q_tiles,block_n", SHAPES + [(5, 1, 3, 2305, 128, 2, 128)])
@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("order", [sa.CYCLIC, sa.SAWTOOTH])
@pytest.mark.parametrize("pairing", [(sa.PAIR_MIRRORED, "mirrored"), (sa.PAIR_ADJACENT, "adjacent")])
def test_paired_schedule_replay_equals_the_schedule_oracle(n_sm, B, H, N, d, q_tiles, block_n, causal, order, pairing):
    check_replay(n_sm, B, H, N, d, q_tiles, block_n, causal, order, sa.TILE_FASTEST, pairing[0], pairing[1])
    check_replay(n_sm, B, H, N, d, q_tiles, block_n, causal, order, sa.HEAD_FASTEST, pairing[0], pairing[1])


def test_default_pairing_is_mirrored_under_the_causal_mask_only():
    assert sa.attn_query_plan(1, 32, 32768, 128, 1, sa.BF16, sm_count=148).pairing == sa.PAIR_MIRRORED
    assert sa.attn_query_plan(1, 32, 32768, 128, 0, sa.BF16, sm_count=148).pairing == sa.PAIR_NONE
    p = sa.attn_query_plan(1, 32, 32768, 128, 1, sa.BF16, sm_count=148)
    assert p.n_units == 32 * 64 and p.grid == 148
    o = sa.Opts()
    o.pairing = sa.PAIR_NONE
    assert sa.attn_query_plan(1, 32, 32768, 128, 1, sa.BF16, o, sm_count=148).n_units == 32 * 128


def check_replay(n_sm, B, H, N, d, q_tiles, block_n, causal, order, digits, pairing, pairing_name):
    o = sa.Opts()
    o.q_tiles, o.block_n, o.digit_order, o.pairing = q_tiles, block_n, digits, pairing
    got = sa.attn_schedule_trace(B, H, N, d, causal, order, sa.F16, o, sm_count=n_sm)
    W = 128 * q_tiles
    want = [w for seq in sch.full_schedule(n_sm, B, H, N, W, block_n, bool(causal), order,
                                           "head_fastest" if digits else "tile_fastest", pairing=pairing_name) for w in seq]
    assert len(got) == len(want)
    for g, w in zip(got, want):
        assert (g.cta, g.iteration, g.k, g.batch, g.head, g.q_item, bool(g.backward), g.n_kv, g.member) == \
            (w.cta, w.i_local, w.k, w.batch, w.head, w.q_tile, w.backward, w.n_kv, w.member)
        # per 128-row tile ranges: what an item of W = 128 rows at that position would need
        for qi, n_q in enumerate((g.n_kv_q0, g.n_kv_q1)):
            r = g.q_item * W + qi * 128
            if qi >= q_tiles or r >= N:
                assert n_q == 0
            else:
                assert n_q == sch.kv_tiles_needed(r // 128, N, 128, block_n, bool(causal))
        assert max(g.n_kv_q0, g.n_kv_q1) == g.n_kv


@pytest.mark.parametrize("n_sm,max_ctas", [(148, 0), (148, 3), (5, 0)])
@pytest.mark.parametrize("B,H,N,q_tiles,block_n", [(2, 3, 1330, 2, 128), (1, 5, 700, 1, 64), (3, 1, 256, 2, 128), (1, 2, 4096, 2, 128)])
@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("digits", [0, 1])
def test_dynamic_claim_replay_equals_the_schedule_oracle(n_sm, max_ctas, B, H, N, q_tiles, block_n, causal, order, digits):
    """The dynamic schedule's order of claims: the linear order of Algorithm 2, the Q blocks of a head from the longest
    scan to the shortest under the causal mask, the direction of a block from the round of its claim."""
    o = sa.Opts()
    o.q_tiles, o.block_n, o.digit_order, o.max_ctas = q_tiles, block_n, digits, max_ctas
    got = sa.attn_dynamic_claim_trace(B, H, N, 128, causal, order, sa.BF16, o, sm_count=n_sm)
    W = 128 * q_tiles
    want = sch.dynamic_claims(n_sm, B, H, N, W, block_n, bool(causal), order, "head_fastest" if digits else "tile_fastest", max_ctas)
    assert len(got) == len(want) == B * H * -(-N // W)
    for g, w in zip(got, want):
        assert (g.cta, g.iteration, g.k, g.batch, g.head, g.q_item, bool(g.backward), g.n_kv, g.member) == \
            (-1, w.i_local, w.k, w.batch, w.head, w.q_tile, w.backward, w.n_kv, 0)
    assert sorted((g.batch, g.head, g.q_item) for g in got) == sorted((b, h, t) for b in range(B) for h in range(H) for t in range(-(-N // W)))
    if causal and not digits:   # within a head the scans never get longer
        for a, b in zip(got, got[1:]):
            if (a.batch, a.head) == (b.batch, b.head):
                assert a.n_kv >= b.n_kv
    if not causal and max_ctas == 0:   # the static, unpaired walk hands out the same blocks with the same directions
        o.pairing = sa.PAIR_NONE
        static = {(e.batch, e.head, e.q_item): bool(e.backward) for e in sa.attn_schedule_trace(B, H, N, 128, 0, order, sa.BF16, o, sm_count=n_sm)}
        assert static == {(g.batch, g.head, g.q_item): bool(g.backward) for g in got}


def test_host_groups():
    """attn_fwd_host's groups of heads: equal ones on request; left to the library, one group for small tensors and
    otherwise one per 16 MiB of a tensor, 32 at most, a head at least."""
    mib = 1 << 20
    assert sa.attn_host_groups(32, 16 * mib) == [1] * 32                           # c5: 32 heads of 16 MiB
    assert sa.attn_host_groups(32, 8 * mib) == [2] * 16                            # c4
    assert sa.attn_host_groups(64, 2 * mib) == [8] * 8                             # c3
    assert sa.attn_host_groups(5, 64 * mib) == [1] * 5
    assert sa.attn_host_groups(1, 64 * mib) == [1]
    assert sa.attn_host_groups(8, 1 * mib) == [8]                                  # 8 MiB: not worth a pipeline
    assert sa.attn_host_groups(8, 4 * mib) == [8]                                  # 32 MiB: not yet
    assert sa.attn_host_groups(10, 16 * mib, 3) == [4, 3, 3]
    assert sa.attn_host_groups(2, 16 * mib, 16) == [1, 1]
    for heads in list(range(1, 200)) + [1000, 4096, 100000]:
        for chunks in (0, 1, 7, 32):
            g = sa.attn_host_groups(heads, 3 * mib, chunks)
            assert sum(g) == heads and len(g) <= 32 and min(g) >= 1 and max(g) - min(g) <= 1
            assert g == sorted(g, reverse=True)
    with pytest.raises(sa.AttnError):
        sa.attn_host_groups(0, mib)
    with pytest.raises(sa.AttnError):
        sa.attn_host_groups(4, mib, 33)


def test_measuring_aids_compile():
    """The two stand-alone measuring aids at the repository root compile for sm_100a against the in-tree headers and
    library (they are run on a GPU by hand or by bench.py, never here)."""
    import subprocess
    import tempfile
    from conftest import nvcc_available
    if not nvcc_available():
        pytest.skip("nvcc not found")
    from paper_2601_16032_b200 import build as lib_build
    assert os.path.exists(lib_build.build_host_call_probe())
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with tempfile.TemporaryDirectory() as tmp:
        subprocess.run([os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc"), "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a",
                        "-o", os.path.join(tmp, "profile_mma_rate"), os.path.join(root, "profile_mma_rate.cu")], check=True, cwd=root)
