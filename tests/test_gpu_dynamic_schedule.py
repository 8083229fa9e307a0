"""GPU tests of attn_fwd_dynamic: the persistent CTAs claim their work items from a counter in caller-provided
scratch memory instead of walking Algorithm 2's fixed grid-stride sequence.  The result must be the oracle's, every
item must be handled exactly once, the output must be the same launch after launch, and in the cyclic order it must
equal the static schedule's bit for bit."""
import numpy as np
import pytest

import workloads as wl
from parity_util import assert_parity, upload

pytestmark = pytest.mark.gpu


def run_dynamic(w, qkv, order, opts=None, ctas_for_scratch=None):
    import torch
    import paper_2601_16032_b200 as sa
    q, k, v = qkv
    adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
    opts = opts or sa.Opts()
    opts.pairing = sa.PAIR_NONE   # the dynamic schedule claims single items: the plan that sizes its scratch has no pairs
    plan = sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, opts)
    n_bytes = sa.attn_dynamic_scratch_bytes(plan.grid if ctas_for_scratch is None else ctas_for_scratch)
    scratch = torch.full((n_bytes // 4,), 0x5a5a5a5a, dtype=torch.int32, device=q.device)  # stale contents on purpose
    o = torch.full_like(q, float("nan"))
    sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal),
                        order, adt, torch.cuda.current_stream().cuda_stream, opts, scratch.data_ptr(), n_bytes)
    sa.attn_device_status()
    return o, scratch.cpu().numpy(), plan


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d,dtype", [(128, wl.BF16), (64, wl.F16)])
@pytest.mark.parametrize("max_ctas", [0, 3])
def test_dynamic_schedule_parity_and_coverage(causal, d, dtype, max_ctas):
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("dyn", 2, 3, 1330, d, dtype, causal, 7400 + d)
    qkv = upload(w)
    opts = sa.Opts()
    opts.max_ctas = max_ctas
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        o, scratch, plan = run_dynamic(w, qkv, order, opts)
        assert_parity(w, o)
        per_cta = scratch[64:64 + plan.grid]
        assert per_cta.sum() == plan.n_work and (per_cta >= 0).all()   # every item handled exactly once
        assert scratch[0] == plan.n_work + plan.grid                      # plus one failed claim per CTA


@pytest.mark.parametrize("block_n,q_tiles", [(64, 2), (128, 1), (64, 1)])
@pytest.mark.parametrize("N", [1, 129, 1000])
def test_dynamic_schedule_other_tile_shapes_and_sizes(block_n, q_tiles, N):
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("dyn-shapes", 1, 5, N, 128, wl.BF16, True, 7450 + N)
    qkv = upload(w)
    opts = sa.Opts()
    opts.block_n, opts.q_tiles, opts.max_ctas = block_n, q_tiles, 2
    o, scratch, plan = run_dynamic(w, qkv, sa.SAWTOOTH, opts)
    assert_parity(w, o)
    assert scratch[64:64 + plan.grid].sum() == plan.n_work


def test_dynamic_cyclic_equals_static_bitwise():
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("dyn-eq", 1, 4, 2000, 128, wl.BF16, True, 7500)
    q, k, v = qkv = upload(w)
    o_dyn, _, _ = run_dynamic(w, qkv, sa.CYCLIC)
    o_sta = torch.empty_like(q)
    sa.attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o_sta.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1, sa.CYCLIC, sa.BF16,
                torch.cuda.current_stream().cuda_stream)
    sa.attn_device_status()
    assert torch.equal(o_dyn.view(torch.int16), o_sta.view(torch.int16))


@pytest.mark.parametrize("causal", [False, True])
def test_dynamic_sawtooth_is_reproducible(causal):
    """Which CTA wins a claim is a race, but an item's scan direction follows the round of its claim, not the winner's own
    count: launch after launch gives the same bits, with few CTAs (many claims each) and with one per item's worth of SMs;
    without the causal mask they are the bits of the static, unpaired schedule."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("dyn-repro", 2, 3, 1700, 128, wl.BF16, causal, 7550)
    q, k, v = qkv = upload(w)
    for max_ctas in (3, 0):
        opts = sa.Opts()
        opts.max_ctas = max_ctas
        first, _, _ = run_dynamic(w, qkv, sa.SAWTOOTH, opts)
        assert_parity(w, first)
        for _ in range(5):
            again, _, _ = run_dynamic(w, qkv, sa.SAWTOOTH, opts)
            assert torch.equal(again.view(torch.int16), first.view(torch.int16))
        if not causal:
            sta = sa.Opts()
            sta.max_ctas, sta.pairing = max_ctas, sa.PAIR_NONE
            o_sta = torch.empty_like(q)
            sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o_sta.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 0, sa.SAWTOOTH, sa.BF16,
                           torch.cuda.current_stream().cuda_stream, sta)
            sa.attn_device_status()
            assert torch.equal(first.view(torch.int16), o_sta.view(torch.int16))


def test_dynamic_rejects_bad_scratch_and_launch_mode():
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("dyn-bad", 1, 2, 512, 64, wl.F16, False, 7600)
    qkv = upload(w)
    with pytest.raises(sa.AttnError) as e:
        run_dynamic(w, qkv, sa.CYCLIC, ctas_for_scratch=1)   # 4 work items -> 4 CTAs, room for one
    assert e.value.status == -1
    q = qkv[0]
    with pytest.raises(sa.AttnError):
        sa.attn_fwd_dynamic(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), 1, 2, 512, 64, 0.125, 0, 0, sa.F16, 0, None, 0, 4096)
    opts = sa.Opts()
    opts.launch_mode = 1
    with pytest.raises(sa.AttnError):
        run_dynamic(w, qkv, sa.CYCLIC, opts)
    opts = sa.Opts()
    opts.pairing = sa.PAIR_MIRRORED
    with pytest.raises(sa.AttnError):
        sa.attn_fwd_dynamic(q.data_ptr(), q.data_ptr(), q.data_ptr(), q.data_ptr(), 1, 2, 512, 64, 0.125, 1, 0, sa.F16, 0, opts, q.data_ptr(), 4096)
