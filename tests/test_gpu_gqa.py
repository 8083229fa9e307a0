"""GPU: grouped-query attention (fewer K/V heads than query heads) against the fp64 oracle, which is given, head by
head, the K/V head that the query head's group shares."""
import numpy as np
import pytest

import workloads as wl
from parity_util import MAX_ABS_TOL, MEAN_ABS_TOL

pytestmark = pytest.mark.gpu


def run_case(B, H, kv_heads, N, d, dtype, causal, order, seed, dynamic=False, opts=None):
    import torch
    import paper_2601_16032_b200 as sa
    from oracle import attention as ora
    wq = wl.small_workload("gqa-q", B, H, N, d, dtype, causal, seed)
    wkv = wl.small_workload("gqa-kv", B, kv_heads, N, d, dtype, causal, seed + 1)
    tdt = torch.bfloat16 if dtype == wl.BF16 else torch.float16

    def up(w, name):
        t = torch.empty((w.B, w.H, w.N, w.d), dtype=torch.int16, device="cuda:0")
        for b, h in wl.all_heads(w):
            t[b, h].copy_(torch.from_numpy(wl.head_bits(w, name, b, h).view(np.int16)))
        return t.view(tdt)

    q, k, v = up(wq, "q"), up(wkv, "k"), up(wkv, "v")
    o = torch.full_like(q, float("nan"))
    opts = opts or sa.Opts()
    opts.kv_heads = kv_heads
    adt = sa.BF16 if dtype == wl.BF16 else sa.F16
    st = torch.cuda.current_stream().cuda_stream
    if dynamic:
        opts.pairing = sa.PAIR_NONE
        nb = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(B, H, N, d, int(causal), adt, opts).grid)
        scratch = torch.zeros(nb // 4, dtype=torch.int32, device="cuda:0")
        sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, wq.scale, int(causal), order, adt, st,
                            opts, scratch.data_ptr(), nb)
    else:
        sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, wq.scale, int(causal), order, adt, st, opts)
    sa.attn_device_status()
    group = H // kv_heads
    worst, total, count = 0.0, 0.0, 0
    for b, h in wl.all_heads(wq):
        qq = wl.bits_to_f64(wl.head_bits(wq, "q", b, h), dtype)
        kk = wl.bits_to_f64(wl.head_bits(wkv, "k", b, h // group), dtype)
        vv = wl.bits_to_f64(wl.head_bits(wkv, "v", b, h // group), dtype)
        want = ora.attention_head(qq, kk, vv, wq.scale, causal)
        got = wl.bits_to_f64(o[b, h].contiguous().view(torch.int16).cpu().numpy().view(np.uint16), dtype)
        assert np.isfinite(got).all()
        err = np.abs(got - want)
        worst, total, count = max(worst, float(err.max())), total + float(err.sum()), count + err.size
    assert worst <= MAX_ABS_TOL and total / count <= MEAN_ABS_TOL, (worst, total / count)


@pytest.mark.parametrize("kv_heads", [1, 2, 4])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d,dtype", [(128, wl.BF16), (64, wl.F16)])
def test_grouped_query_attention(kv_heads, causal, d, dtype):
    import paper_2601_16032_b200 as sa
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        run_case(2, 4, kv_heads, 900, d, dtype, causal, order, 7800 + kv_heads)


def test_grouped_query_attention_other_plans():
    import paper_2601_16032_b200 as sa
    o = sa.Opts()
    o.max_ctas, o.digit_order = 3, sa.HEAD_FASTEST
    run_case(1, 6, 2, 1330, 128, wl.BF16, True, sa.SAWTOOTH, 7810, opts=o)
    run_case(1, 6, 3, 1330, 128, wl.BF16, True, sa.SAWTOOTH, 7811, dynamic=True)
    o = sa.Opts()
    o.launch_mode, o.block_n, o.q_tiles = 1, 64, 1
    run_case(2, 4, 2, 700, 64, wl.F16, False, sa.CYCLIC, 7812, opts=o)


def test_kv_heads_must_divide_heads_and_the_wrapper_infers_them():
    import torch
    import paper_2601_16032_b200 as sa
    q = torch.randn(1, 4, 256, 64, device="cuda:0").to(torch.float16)
    k = torch.randn(1, 2, 256, 64, device="cuda:0").to(torch.float16)
    o = sa.Opts()
    o.kv_heads = 3
    with pytest.raises(sa.AttnError) as e:
        sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), k.data_ptr(), q.data_ptr(), 1, 4, 256, 64, 0.125, 0, 0, sa.F16, 0, o)
    assert e.value.status == -1
    out = sa.forward(q, k, k, causal=True)          # K/V with two heads: groups of two query heads
    sa.attn_device_status()
    ref = torch.nn.functional.scaled_dot_product_attention(q.float(), k.float().repeat_interleave(2, dim=1), k.float().repeat_interleave(2, dim=1),
                                                           is_causal=True)
    assert (out.float() - ref).abs().max() < 2e-2


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("kv_heads", [0, 2])
@pytest.mark.parametrize("d,dtype,N", [(128, wl.BF16, 1330), (64, wl.F16, 257)])
def test_bnhd_layout(causal, kv_heads, d, dtype, N):
    """q, k, v and o stored as [B, N, heads, d]: same result as the oracle head by head, log-sum-exp still [B, H, N]."""
    import torch
    import paper_2601_16032_b200 as sa
    from oracle import attention as ora
    B, H = 2, 4
    Hkv = kv_heads or H
    wq = wl.small_workload("bnhd-q", B, H, N, d, dtype, causal, 7900)
    wkv = wl.small_workload("bnhd-kv", B, Hkv, N, d, dtype, causal, 7901)
    tdt = torch.bfloat16 if dtype == wl.BF16 else torch.float16

    def up(w, name):   # [B, N, heads, d]
        t = torch.empty((w.B, w.N, w.H, w.d), dtype=torch.int16, device="cuda:0")
        for b, h in wl.all_heads(w):
            t[b, :, h].copy_(torch.from_numpy(wl.head_bits(w, name, b, h).view(np.int16)))
        return t.view(tdt)

    q, k, v = up(wq, "q"), up(wkv, "k"), up(wkv, "v")
    o = torch.full_like(q, float("nan"))
    lse = torch.full((B, H, N), float("nan"), dtype=torch.float32, device="cuda:0")
    opts = sa.Opts()
    opts.layout, opts.kv_heads, opts.max_ctas, opts.lse = sa.LAYOUT_BNHD, kv_heads, 3, lse.data_ptr()
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), B, H, N, d, wq.scale, int(causal), order,
                       sa.BF16 if dtype == wl.BF16 else sa.F16, torch.cuda.current_stream().cuda_stream, opts)
        sa.attn_device_status()
        worst, total, count = 0.0, 0.0, 0
        for b, h in wl.all_heads(wq):
            g = h // (H // Hkv)
            qq = wl.bits_to_f64(wl.head_bits(wq, "q", b, h), dtype)
            kk = wl.bits_to_f64(wl.head_bits(wkv, "k", b, g), dtype)
            vv = wl.bits_to_f64(wl.head_bits(wkv, "v", b, g), dtype)
            got = wl.bits_to_f64(o[b, :, h].contiguous().view(torch.int16).cpu().numpy().view(np.uint16), dtype)
            err = np.abs(got - ora.attention_head(qq, kk, vv, wq.scale, causal))
            worst, total, count = max(worst, float(err.max())), total + float(err.sum()), count + err.size
            want_lse = ora.logsumexp_rows(qq, np.arange(N, dtype=np.int64), kk, wq.scale, causal)
            assert np.abs(lse[b, h].double().cpu().numpy() - want_lse).max() <= 5e-4
        assert worst <= MAX_ABS_TOL and total / count <= MEAN_ABS_TOL, (worst, total / count)
