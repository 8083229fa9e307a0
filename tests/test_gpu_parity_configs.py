"""GPU parity on the five benchmark configurations at full size, through the C ABI, in the launch
configuration the benchmark times (library defaults), both scan orders; for c3, c4 and c5 also on the dynamic schedule
of the benchmark's second leg, for c5 also through attn_fwd_host, its end-to-end leg.

The oracle result of the checked rows is computed once per configuration and both orders are
compared with it: every row of every head for c1 and c2, every row of two heads plus seeded rows
elsewhere for c3 and c4, 512 seeded rows plus the tile-edge rows in every head for c5."""
import numpy as np
import pytest

import workloads as wl
from parity_util import MAX_ABS_TOL, MEAN_ABS_TOL, oracle_rows, compare_rows, run_cuda, upload, output_bits

pytestmark = pytest.mark.gpu


def check_config(name, opts_list, also_dynamic=False, also_host=False):
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.CONFIGS[name]
    plan = wl.checked_rows(w)
    want = oracle_rows(w, plan)
    qkv = upload(w)
    outs = {}
    for label, opts in opts_list:
        for order in (sa.CYCLIC, sa.SAWTOOTH):
            o = run_cuda(w, qkv, order, opts)
            max_abs, mean_abs, n_rows = compare_rows(w, o, plan, want)
            assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, \
                f"{name} {label} order {order}: max_abs {max_abs:.3e} mean_abs {mean_abs:.3e} over {n_rows} rows"
            outs[(label, order)] = o if w.compulsory_bytes <= (64 << 20) else None
            del o
    if also_dynamic or also_host:
        q, k, v = qkv
        adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
        stream = torch.cuda.current_stream().cuda_stream
        o = torch.empty_like(q)
    if also_dynamic:   # the schedule of the benchmark's second leg
        single = sa.Opts()
        single.pairing = sa.PAIR_NONE
        n_bytes = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, single).grid)
        scratch = torch.zeros(n_bytes // 4, dtype=torch.int32, device=q.device)
        for order in (sa.CYCLIC, sa.SAWTOOTH):
            o.fill_(float("nan"))
            sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal), order, adt,
                                stream, None, scratch.data_ptr(), n_bytes)
            sa.attn_device_status()
            max_abs, mean_abs, n_rows = compare_rows(w, o, plan, want)
            assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, f"{name} dynamic order {order}: max_abs {max_abs:.3e} mean_abs {mean_abs:.3e}"
    if also_host:      # the benchmark's end-to-end leg: host buffers in and out, the library's own groups of heads
        host = [t.view(torch.int16).cpu().pin_memory() for t in (q, k, v)]
        o_host = torch.full(q.shape, -1, dtype=torch.int16).pin_memory()
        staging = [torch.empty_like(q) for _ in range(3)]
        o.fill_(float("nan"))
        sa.attn_fwd_host(host[0].data_ptr(), host[1].data_ptr(), host[2].data_ptr(), o_host.data_ptr(), staging[0].data_ptr(),
                         staging[1].data_ptr(), staging[2].data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal), sa.SAWTOOTH,
                         adt, stream, None)
        torch.cuda.synchronize()
        sa.attn_device_status()
        got = o_host.view(q.dtype).cuda()
        max_abs, mean_abs, n_rows = compare_rows(w, got, plan, want)
        assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, f"{name} host entry point: max_abs {max_abs:.3e} mean_abs {mean_abs:.3e}"
        del host, o_host, staging, got
    torch.cuda.empty_cache()
    return w, outs


def test_c1_all_rows_both_tile_shapes():
    import paper_2601_16032_b200 as sa
    o64 = sa.Opts()
    o64.block_n = 64
    w, outs = check_config("c1", [("default", None), ("128x64", o64)])
    a = wl.bits_to_f64(output_bits(outs[("default", sa.CYCLIC)], 0, 0), w.dtype)
    b = wl.bits_to_f64(output_bits(outs[("default", sa.SAWTOOTH)], 0, 0), w.dtype)
    assert np.abs(a - b).max() <= 1e-2


def test_c2_all_rows_128x64_tiles_and_default():
    import paper_2601_16032_b200 as sa
    o64 = sa.Opts()
    o64.block_n = 64  # the 128 x 64 Q / K tiles this configuration names
    check_config("c2", [("128x64", o64), ("default", None)])


def test_c3_two_heads_plus_sampled_rows():
    check_config("c3", [("default", None)], also_dynamic=True)


def test_c4_causal_two_heads_plus_sampled_rows():
    check_config("c4", [("default", None)], also_dynamic=True)


def test_c5_causal_sampled_rows_every_head():
    check_config("c5", [("default", None)], also_dynamic=True, also_host=True)


def test_long_single_head_beyond_l2_sampled_rows():
    """One head of 262,144 keys (K+V = 128 MiB, more than the L2): 256 seeded rows plus the tile-edge rows, both scan
    orders and the dynamic schedule, against the oracle."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.STUDY_CASES["long-256k"]
    plan = {(0, 0): wl.sampled_rows(w, 0, 0, 256)}
    want = oracle_rows(w, plan)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        o = run_cuda(w, qkv, order)
        max_abs, mean_abs, n_rows = compare_rows(w, o, plan, want)
        assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, (order, max_abs, mean_abs, n_rows)
    q, k, v = qkv
    n_bytes = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(w.B, w.H, w.N, w.d, 0, sa.BF16).grid)
    scratch = torch.zeros(n_bytes // 4, dtype=torch.int32, device=q.device)
    o = torch.full_like(q, float("nan"))
    sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 0, sa.SAWTOOTH, sa.BF16,
                        torch.cuda.current_stream().cuda_stream, None, scratch.data_ptr(), n_bytes)
    sa.attn_device_status()
    max_abs, mean_abs, n_rows = compare_rows(w, o, plan, want)
    assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, ("dynamic", max_abs, mean_abs, n_rows)


@pytest.mark.parametrize("name", ["d64-n8k", "sweep-d64-b8", "sweep-d64-b8-causal"])
def test_d64_benchmark_shapes_sampled_rows(name):
    """The d = 64 shapes the benchmark also times (a shape that fills the GPU, and the paper's own sweep shape with and
    without the causal mask: 512 K/V steps per work item through three S buffers): seeded rows of every head, both orders."""
    import paper_2601_16032_b200 as sa
    w = wl.STUDY_CASES[name]
    plan = {bh: wl.sampled_rows(w, bh[0], bh[1], 96 if w.N > 10000 else 24) for bh in wl.all_heads(w)}
    want = oracle_rows(w, plan)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        o = run_cuda(w, qkv, order)
        max_abs, mean_abs, n_rows = compare_rows(w, o, plan, want)
        assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, (name, order, max_abs, mean_abs, n_rows)


def test_many_small_heads():
    """1,500 heads of 300 keys: many more (batch, head) pairs than SMs, ragged length, both tile shapes."""
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("many-heads", 25, 60, 300, 64, wl.F16, True, 7900)
    plan = {(b, h): None for (b, h) in [(0, 0), (7, 31), (24, 59)]}
    want = oracle_rows(w, plan)
    qkv = upload(w)
    for block_n in (128, 64):
        opts = sa.Opts()
        opts.block_n = block_n
        o = run_cuda(w, qkv, sa.SAWTOOTH, opts)
        max_abs, mean_abs, _ = compare_rows(w, o, plan, want)
        assert max_abs <= MAX_ABS_TOL and mean_abs <= MEAN_ABS_TOL, (block_n, max_abs, mean_abs)
