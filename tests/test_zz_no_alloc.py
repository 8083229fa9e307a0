"""attn_fwd_dynamic_noalloc: the dynamic-schedule forward pass for callers that are not allowed to allocate device
memory (code running under stream capture, inside an allocator hook, in a no-allocation real-time loop, or as a guest
in an application that owns all device memory).  Its counters sit in a fixed array inside the library instead of in a
caller-provided buffer.  The check: through the C ABI, two calls in a row, each compared with attn_fwd_dynamic (which
takes the scratch from the caller) within the parity tolerance of the other tests; the second call finds the first
call's counters still in the array and must not be disturbed by them.  This file sorts last on purpose, so that a run
that stops at the first failure has already run everything else."""
import numpy as np
import pytest

import workloads as wl
from parity_util import MAX_ABS_TOL, MEAN_ABS_TOL, upload, output_bits

pytestmark = pytest.mark.gpu


def test_no_alloc_entry_matches_the_scratch_taking_entry_twice_in_a_row():
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("noalloc", 2, 3, 1500, 128, wl.BF16, True, 7700)
    q, k, v = upload(w)
    stream = torch.cuda.current_stream().cuda_stream
    opts = sa.Opts()
    opts.max_ctas = 5   # several items per CTA, so the counters are really used
    opts.pairing = sa.PAIR_NONE   # the dynamic schedule claims single items
    plan = sa.attn_query_plan(w.B, w.H, w.N, w.d, 1, sa.BF16, opts)
    n_bytes = sa.attn_dynamic_scratch_bytes(plan.grid)
    scratch = torch.zeros(n_bytes // 4, dtype=torch.int32, device=q.device)
    want = torch.empty_like(q)
    sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), want.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1, sa.SAWTOOTH,
                        sa.BF16, stream, opts, scratch.data_ptr(), n_bytes)
    sa.attn_device_status()
    for call in range(2):
        got = torch.full_like(q, float("nan"))
        sa.attn_fwd_dynamic_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), got.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1,
                                    sa.SAWTOOTH, sa.BF16, stream, opts)
        sa.attn_device_status()
        for b, h in wl.all_heads(w):
            a = wl.bits_to_f64(output_bits(got, b, h), w.dtype)
            r = wl.bits_to_f64(output_bits(want, b, h), w.dtype)
            assert np.isfinite(a).all(), f"call {call}: non-finite output in head ({b},{h})"
            err = np.abs(a - r)
            assert err.max() <= MAX_ABS_TOL and err.mean() <= MEAN_ABS_TOL, (call, b, h, err.max(), err.mean())


def test_no_alloc_entry_validates_arguments_and_runs_other_shapes():
    """Same argument checks as the other entry points (nothing is enqueued on a bad call), and a second shape and
    type on the same shared array.  The 1024-CTA limit itself cannot be reached on a GPU with fewer SMs than that:
    the persistent grid never exceeds the SM count."""
    import torch
    import paper_2601_16032_b200 as sa
    from parity_util import assert_parity
    w = wl.small_workload("noalloc-f16", 1, 2, 700, 64, wl.F16, False, 7800)
    q, k, v = upload(w)
    o = torch.full_like(q, float("nan"))
    stream = torch.cuda.current_stream().cuda_stream
    with pytest.raises(sa.AttnError) as e:
        sa.attn_fwd_dynamic_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, 96, w.scale, 0,
                                    sa.CYCLIC, sa.F16, stream, None)
    assert e.value.status == -2
    sa.attn_fwd_dynamic_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 0,
                                sa.CYCLIC, sa.F16, stream, None)
    sa.attn_device_status()
    assert_parity(w, o)
