"""Seeded random sweep over shapes and options: every case is checked against the fp64 oracle on all of its rows
(or the sampled plan for longer ones), through the static and the dynamic schedule."""
import numpy as np
import pytest

import workloads as wl
from parity_util import assert_parity, run_cuda, upload

pytestmark = pytest.mark.gpu


def _cases(n=48, seed=20260116):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        d = int(rng.choice([64, 128]))
        out.append(dict(
            B=int(rng.integers(1, 4)), H=int(rng.integers(1, 5)), N=int(rng.choice([1, 2, 63, 64, 65, 127, 128, 129, 255, 256, 257, 384, 511, 640, 777, 1025, 1500])),
            d=d, dtype=str(rng.choice([wl.F16, wl.BF16])), causal=bool(rng.integers(0, 2)), order=int(rng.integers(0, 2)),
            block_n=int(rng.choice([0, 64, 128])), q_tiles=int(rng.choice([0, 1, 2])), kv_stages=int(rng.choice([0, 2, 3, 4])),
            max_ctas=int(rng.choice([0, 1, 2, 5])), digit_order=int(rng.integers(0, 2)), dynamic=bool(rng.integers(0, 2)), pairing=int(rng.integers(0, 4)), seed=9000 + i))
    return out


@pytest.mark.parametrize("c", _cases(), ids=lambda c: f"B{c['B']}H{c['H']}N{c['N']}d{c['d']}{c['dtype']}{'c' if c['causal'] else 'f'}o{c['order']}bn{c['block_n']}q{c['q_tiles']}s{c['kv_stages']}m{c['max_ctas']}g{c['digit_order']}{'dyn' if c['dynamic'] else 'sta'}p{c['pairing']}")
def test_random_case(c):
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("rand", c["B"], c["H"], c["N"], c["d"], c["dtype"], c["causal"], c["seed"])
    qkv = upload(w)
    opts = sa.Opts()
    opts.block_n, opts.q_tiles, opts.kv_stages, opts.max_ctas, opts.digit_order = c["block_n"], c["q_tiles"], c["kv_stages"], c["max_ctas"], c["digit_order"]
    if not c["dynamic"]:
        opts.pairing = c["pairing"]
        o = run_cuda(w, qkv, c["order"], opts)
    else:
        q, k, v = qkv
        adt = sa.BF16 if w.dtype == wl.BF16 else sa.F16
        opts.pairing = sa.PAIR_NONE   # the plan of the dynamic schedule: single items
        plan = sa.attn_query_plan(w.B, w.H, w.N, w.d, int(w.causal), adt, opts)
        n_bytes = sa.attn_dynamic_scratch_bytes(plan.grid)
        scratch = torch.full((n_bytes // 4,), -7, dtype=torch.int32, device=q.device)
        o = torch.full_like(q, float("nan"))
        sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(w.causal), c["order"],
                            adt, torch.cuda.current_stream().cuda_stream, opts, scratch.data_ptr(), n_bytes)
        sa.attn_device_status()
        assert int(scratch[64:64 + plan.grid].sum()) == plan.n_work
    assert_parity(w, o)
