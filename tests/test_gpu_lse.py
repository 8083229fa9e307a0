"""GPU: the optional log-sum-exp output (ln of the softmax denominator per query row) against the fp64 oracle,
element by element, through the C ABI."""
import numpy as np
import pytest

import workloads as wl
from parity_util import assert_parity, upload

pytestmark = pytest.mark.gpu

# fp32 running sums of probabilities whose exponents come from the MUFU (rel. error about 2^-22) or from a cubic with
# relative error 7.5e-5; a sum of N such terms keeps that relative error, so ln of it is off by about 1e-4 at most.
LSE_ABS_TOL = 5e-4


def run_with_lse(w, qkv, order, opts=None):
    import torch
    import paper_2601_16032_b200 as sa
    q, k, v = qkv
    o = torch.full_like(q, float("nan"))
    lse = torch.full((w.B, w.H, w.N), float("nan"), dtype=torch.float32, device=q.device)
    opts = opts or sa.Opts()
    opts.lse = lse.data_ptr()
    sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal),
                   order, sa.BF16 if w.dtype == wl.BF16 else sa.F16, torch.cuda.current_stream().cuda_stream, opts)
    sa.attn_device_status()
    return o, lse


def oracle_lse(w, b, h):
    from oracle import attention as ora
    q = wl.bits_to_f64(wl.head_bits(w, "q", b, h), w.dtype)
    k = wl.bits_to_f64(wl.head_bits(w, "k", b, h), w.dtype)
    return ora.logsumexp_rows(q, np.arange(w.N, dtype=np.int64), k, w.scale, w.causal)


@pytest.mark.parametrize("N", [1, 129, 257, 1000, 2500])
@pytest.mark.parametrize("d,dtype", [(64, wl.F16), (128, wl.BF16)])
@pytest.mark.parametrize("causal", [False, True])
def test_lse_matches_oracle(N, d, dtype, causal):
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("lse", 2, 2, N, d, dtype, causal, 7600 + N)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        opts = sa.Opts()
        opts.max_ctas = 3
        o, lse = run_with_lse(w, qkv, order, opts)
        assert_parity(w, o)
        for b, h in wl.all_heads(w):
            got = lse[b, h].double().cpu().numpy()
            assert np.isfinite(got).all()
            assert np.abs(got - oracle_lse(w, b, h)).max() <= LSE_ABS_TOL


def test_lse_with_wide_scores_and_tile_options():
    """Scores spread over hundreds of units (the lazy rescale path) and the 64-row K/V tiles, one Q tile per item."""
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("lse-wide", 1, 2, 1330, 128, wl.BF16, True, 7650, k_scale=8.0)
    qkv = upload(w)
    opts = sa.Opts()
    opts.block_n, opts.q_tiles, opts.max_ctas = 64, 1, 2
    o, lse = run_with_lse(w, qkv, sa.SAWTOOTH, opts)
    assert_parity(w, o)
    for b, h in wl.all_heads(w):
        want = oracle_lse(w, b, h)
        got = lse[b, h].double().cpu().numpy()
        assert np.abs(got - want).max() <= LSE_ABS_TOL * max(1.0, np.abs(want).max() / 16.0)


def test_lse_pointer_is_optional_and_checked():
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("lse-opt", 1, 1, 300, 64, wl.F16, False, 7660)
    q, k, v = upload(w)
    o = torch.empty_like(q)
    lse = torch.zeros(w.N + 1, dtype=torch.float32, device=q.device)
    opts = sa.Opts()
    opts.lse = lse.data_ptr() + 2          # not 4-byte aligned
    with pytest.raises(sa.AttnError) as e:
        sa.attn_fwd_ex(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), 1, 1, w.N, w.d, w.scale, 0, sa.SAWTOOTH, sa.F16, 0, opts)
    assert e.value.status == -3
