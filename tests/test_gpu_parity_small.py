"""GPU parity at small and ragged sizes: every row of every head against the fp64 oracle, through
the C ABI, for both scan orders, both tile shapes, one or two Q tiles per work item."""
import numpy as np
import pytest

import workloads as wl
from parity_util import assert_parity, run_cuda, upload, output_bits

pytestmark = pytest.mark.gpu


def opts_for(block_n=0, q_tiles=0, **kw):
    import paper_2601_16032_b200 as sa
    o = sa.Opts()
    o.block_n, o.q_tiles = block_n, q_tiles
    for k, v in kw.items():
        setattr(o, k, v)
    return o


@pytest.mark.parametrize("N", [1, 17, 128, 129, 200, 256, 257, 1000])
@pytest.mark.parametrize("d,dtype", [(64, wl.F16), (128, wl.BF16), (64, wl.BF16), (128, wl.F16)])
@pytest.mark.parametrize("causal", [False, True])
def test_ragged_sizes(N, d, dtype, causal):
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("ragged", 2, 3, N, d, dtype, causal, 7000 + N)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        assert_parity(w, run_cuda(w, qkv, order))


@pytest.mark.parametrize("block_n", [64, 128])
@pytest.mark.parametrize("q_tiles", [1, 2])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d,dtype", [(64, wl.F16), (128, wl.BF16)])
def test_tile_shapes_and_scan_orders(block_n, q_tiles, causal, d, dtype):
    """Few SMs' worth of CTAs (max_ctas) so that every CTA runs several items and alternates direction."""
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("tiles", 1, 2, 1330, d, dtype, causal, 7100 + block_n + q_tiles)
    qkv = upload(w)
    outs = []
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        o = run_cuda(w, qkv, order, opts_for(block_n, q_tiles, max_ctas=3))
        assert_parity(w, o)
        outs.append(o)
    a = wl.bits_to_f64(output_bits(outs[0], 0, 1), dtype)
    b = wl.bits_to_f64(output_bits(outs[1], 0, 1), dtype)
    assert np.abs(a - b).max() <= 1e-2  # the two orders agree to rounding


@pytest.mark.parametrize("opt", [dict(kv_stages=2), dict(kv_stages=3), dict(digit_order=1), dict(launch_mode=1),
                                 dict(l2_policy=1), dict(max_ctas=1), dict(pairing=1), dict(pairing=2), dict(pairing=3),
                                 dict(pairing=2, launch_mode=1), dict(pairing=3, digit_order=1, max_ctas=2), dict(check_mode=1)])
def test_options_do_not_change_the_result(opt):
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("opts", 2, 2, 900, 128, wl.BF16, True, 7200)
    qkv = upload(w)
    assert_parity(w, run_cuda(w, qkv, sa.SAWTOOTH, opts_for(**opt)))


def test_bitwise_reproducible_and_guard_bands_untouched():
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("repro", 1, 2, 777, 128, wl.BF16, True, 7300)
    q, k, v = upload(w)
    n = q.numel()
    guard = 4096
    buf = torch.full((n + 2 * guard,), -1, dtype=torch.int16, device="cuda:0")
    o = buf[guard:guard + n].view(torch.bfloat16).view(q.shape)
    outs = []
    for _ in range(2):
        o.view(torch.int16).fill_(-1)
        sa.attn_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1,
                    sa.SAWTOOTH, sa.BF16, torch.cuda.current_stream().cuda_stream)
        sa.attn_device_status()
        outs.append(o.view(torch.int16).clone())
        assert (buf[:guard] == -1).all() and (buf[guard + n:] == -1).all()
    assert torch.equal(outs[0], outs[1])
    assert_parity(w, o)


def test_invariants_on_gpu():
    """V = ones gives ones; causal row 0 returns V row 0; a dominant score selects its V row."""
    import torch
    import paper_2601_16032_b200 as sa
    B, H, N, d = 1, 2, 300, 64
    g = torch.Generator(device="cpu").manual_seed(5)
    q = torch.randn(B, H, N, d, generator=g).to(torch.float16).cuda()
    k = torch.randn(B, H, N, d, generator=g).to(torch.float16).cuda()
    v = torch.randn(B, H, N, d, generator=g).to(torch.float16).cuda()
    ones = torch.ones_like(v)
    for causal in (False, True):
        o = sa.forward(q, k, ones, causal=causal)
        sa.attn_device_status()
        assert (o == 1).all()
    o = sa.forward(q, k, v, causal=True)
    sa.attn_device_status()
    assert torch.equal(o[:, :, 0], v[:, :, 0])
    kn = torch.nn.functional.normalize(k.float(), dim=-1)
    q_hot = (60.0 * kn[:, :, 123:124]).expand(B, H, N, d).to(torch.float16).contiguous()
    o = sa.forward(q_hot, kn.to(torch.float16), v, causal=False, scale=1.0)
    sa.attn_device_status()
    assert (o - v[:, :, 123:124]).abs().max() < 2e-2


def test_cycle_counter_reports_a_plausible_clock():
    """attn_last_kernel_cycles / elapsed time is an SM clock between 0.5 and 2.2 GHz for a launch that fills the GPU."""
    import torch
    import paper_2601_16032_b200 as sa
    q = torch.randn(2, 16, 4096, 128, device="cuda:0").to(torch.bfloat16)
    o = torch.empty_like(q)
    st = torch.cuda.current_stream().cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(3):
        if i == 2:
            e0.record()
        sa.attn_fwd(q.data_ptr(), q.data_ptr(), q.data_ptr(), o.data_ptr(), 2, 16, 4096, 128, 0.088, 0, sa.SAWTOOTH, sa.BF16, st)
    e1.record()
    cycles = sa.attn_last_kernel_cycles()
    sa.attn_device_status()
    mhz = cycles / (e0.elapsed_time(e1) * 1e3)
    assert 500 < mhz < 2200, (cycles, e0.elapsed_time(e1))


def test_bad_arguments_are_rejected_before_launch():
    import torch
    import paper_2601_16032_b200 as sa
    t = torch.zeros(1, 1, 128, 64, dtype=torch.float16, device="cuda:0")
    p = t.data_ptr()
    st = 0
    cases = [
        (dict(q=0), -1), (dict(N=0), -1), (dict(d=96), -2), (dict(scale=float("nan")), -1), (dict(scale=float("inf")), -1),
        (dict(scan_order=5), -1), (dict(dtype=7), -1), (dict(causal=2), -1), (dict(q=p + 2), -3),
    ]
    for change, status in cases:
        a = dict(q=p, k=p, v=p, o=p, B=1, H=1, N=128, d=64, scale=0.125, causal=0, scan_order=0, dtype=0)
        a.update(change)
        with pytest.raises(sa.AttnError) as e:
            sa.attn_fwd(a["q"], a["k"], a["v"], a["o"], a["B"], a["H"], a["N"], a["d"], a["scale"], a["causal"],
                        a["scan_order"], a["dtype"], st)
        assert e.value.status == status, (change, e.value)


@pytest.mark.parametrize("host_chunks", [1, 3, 32])
def test_host_entry_point_pipeline_matches_device_entry_point(host_chunks):
    """attn_fwd_host (pinned host buffers in and out, heads cut into groups that are uploaded, computed and
    downloaded as a pipeline) gives the device entry point's result bit for bit in the cyclic order."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("host", 1, 5, 700, 128, wl.BF16, True, 7350)
    q, k, v = upload(w)
    want = run_cuda(w, (q, k, v), sa.CYCLIC)
    host = [t.view(torch.int16).cpu().pin_memory() for t in (q, k, v)]
    o_host = torch.full(q.shape, -1, dtype=torch.int16).pin_memory()
    dev = [torch.empty_like(q) for _ in range(4)]
    opts = sa.Opts()
    opts.host_chunks = host_chunks
    stream = torch.cuda.Stream()
    for _ in range(2):   # twice: the second call reuses the pipeline's events
        o_host.fill_(-1)
        sa.attn_fwd_host(host[0].data_ptr(), host[1].data_ptr(), host[2].data_ptr(), o_host.data_ptr(), dev[0].data_ptr(),
                         dev[1].data_ptr(), dev[2].data_ptr(), dev[3].data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1, sa.CYCLIC,
                         sa.BF16, stream.cuda_stream, opts)
        stream.synchronize()
        sa.attn_device_status()
        assert torch.equal(o_host, want.view(torch.int16).cpu())
    assert_parity(w, o_host.view(torch.bfloat16).cuda())


def test_host_entry_point_with_the_library_own_groups():
    """A tensor above 32 MiB, host_chunks left at 0: attn_fwd_host cuts the nine heads into two groups and runs their
    kernels on two streams in turn; the result is the device entry point's up to the scan directions."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("host-ramp", 1, 9, 16384, 128, wl.BF16, True, 7355)
    assert sa.attn_host_groups(w.B * w.H, w.N * w.d * 2) == [5, 4]
    q, k, v = upload(w)
    want = run_cuda(w, (q, k, v), sa.SAWTOOTH)
    host = [t.view(torch.int16).cpu().pin_memory() for t in (q, k, v)]
    o_host = torch.full(q.shape, -1, dtype=torch.int16).pin_memory()
    dev = [torch.empty_like(q) for _ in range(4)]
    stream = torch.cuda.Stream()
    for _ in range(2):
        o_host.fill_(-1)
        sa.attn_fwd_host(host[0].data_ptr(), host[1].data_ptr(), host[2].data_ptr(), o_host.data_ptr(), dev[0].data_ptr(),
                         dev[1].data_ptr(), dev[2].data_ptr(), dev[3].data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1, sa.SAWTOOTH,
                         sa.BF16, stream.cuda_stream, None)
        stream.synchronize()
        sa.attn_device_status()
        # a group is a launch of its own: its heads' items land on other CTAs, with other scan directions, than in one launch
        got = o_host.view(torch.bfloat16).cuda()
        assert (got.float() - want.float()).abs().max().item() < 2e-2
    assert_parity(w, got, {bh: wl.sampled_rows(w, bh[0], bh[1], 48) for bh in wl.all_heads(w)})


@pytest.mark.parametrize("causal", [False, True])
def test_large_score_range_exercises_the_lazy_rescale(causal):
    """K scaled by 8: scores spread over +-35 in log2 units, so the running maximum jumps by more than the rescale
    threshold between tiles again and again, and the softmax is close to one-hot."""
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("peaky", 1, 3, 1500, 128, wl.BF16, causal, 7360, k_scale=8.0)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        assert_parity(w, run_cuda(w, qkv, order))


def test_monotonically_growing_scores_and_uniform_scores():
    """Scores that grow with the key index (every tile raises the row maximum in a forward scan, none in a backward
    one) and scores that are all equal (K = 0: O is the mean, or prefix mean, of V), against the oracle."""
    import torch
    import paper_2601_16032_b200 as sa
    from oracle import attention as ora
    N, d = 1100, 64
    g = torch.Generator(device="cpu").manual_seed(11)
    v = torch.randn(1, 1, N, d, generator=g).to(torch.float16)
    q = torch.full((1, 1, N, d), 0.5, dtype=torch.float16)
    ramp = (torch.arange(N, dtype=torch.float32) * (1.0 / 16.0)).view(1, 1, N, 1).expand(1, 1, N, d).contiguous().to(torch.float16)
    for k, causal in ((ramp, False), (ramp, True), (torch.zeros_like(q), True)):
        want = ora.attention_head(q[0, 0].double().numpy(), k[0, 0].double().numpy(), v[0, 0].double().numpy(), 0.125, causal)
        opts = sa.Opts()
        opts.max_ctas = 2
        for order in (sa.CYCLIC, sa.SAWTOOTH):
            o = sa.forward(q.cuda(), k.cuda(), v.cuda(), causal=causal, scan_order=order, scale=0.125, opts=opts)
            sa.attn_device_status()
            err = np.abs(o[0, 0].double().cpu().numpy() - want)
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, (causal, order, err.max(), err.mean())


@pytest.mark.parametrize("pairing", [1, 2, 3])
@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("N,q_tiles", [(2305, 2), (1330, 1), (256, 2), (300, 2)])
def test_pairings_cover_every_row(pairing, causal, N, q_tiles):
    """One item per unit, mirrored pairs and adjacent pairs (odd and even numbers of Q blocks, a head of one block),
    few CTAs so that every CTA walks several units: every row of every head against the oracle, both scan orders."""
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("pairs", 1, 3, N, 128, wl.BF16, causal, 7400 + N)
    qkv = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        assert_parity(w, run_cuda(w, qkv, order, opts_for(q_tiles=q_tiles, pairing=pairing, max_ctas=2)))


@pytest.mark.parametrize("scale", [-0.11, 0.0, -2.5])
@pytest.mark.parametrize("causal", [False, True])
def test_negative_and_zero_scale(scale, causal):
    """Any finite scale: a negative one turns the softmax towards the smallest scores, zero weighs every visible key
    alike (O is the mean, or prefix mean, of V).  Against the oracle, which takes the scale as it is."""
    import torch
    import paper_2601_16032_b200 as sa
    from oracle import attention as ora
    w = wl.small_workload("scale", 1, 2, 900, 64, wl.F16, causal, 7450)
    q, k, v = upload(w)
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        o = sa.forward(q, k, v, causal=causal, scan_order=order, scale=scale)
        sa.attn_device_status()
        for h in range(w.H):
            want = ora.attention_head(*(wl.bits_to_f64(wl.head_bits(w, n, 0, h), w.dtype) for n in ("q", "k", "v")), scale, causal)
            err = np.abs(o[0, h].double().cpu().numpy() - want)
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, (scale, causal, order, err.max(), err.mean())


def test_host_entry_point_refuses_before_copying_and_leaves_the_stream_usable():
    """A bad option makes attn_fwd_host fail before anything is enqueued (the device staging buffers keep their
    contents); a good call on the same stream afterwards gives the device entry point's result bit for bit."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("host-bad", 1, 5, 700, 128, wl.BF16, True, 7351)
    q, k, v = upload(w)
    want = run_cuda(w, (q, k, v), sa.CYCLIC)
    host = [t.view(torch.int16).cpu().pin_memory() for t in (q, k, v)]
    o_host = torch.full(q.shape, -1, dtype=torch.int16).pin_memory()
    dev = [torch.full_like(q.view(torch.int16), 77) for _ in range(4)]
    stream = torch.cuda.Stream()

    def call(opts, scan_order=sa.CYCLIC):
        sa.attn_fwd_host(host[0].data_ptr(), host[1].data_ptr(), host[2].data_ptr(), o_host.data_ptr(), dev[0].data_ptr(),
                         dev[1].data_ptr(), dev[2].data_ptr(), dev[3].data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1, scan_order,
                         sa.BF16, stream.cuda_stream, opts)

    for bad in (dict(block_n=96), dict(kv_stages=99), dict(pairing=9), dict(check_mode=1)):
        opts = sa.Opts()
        opts.host_chunks = 3
        for name, val in bad.items():
            setattr(opts, name, val)
        with pytest.raises(sa.AttnError):
            call(opts)
    opts = sa.Opts()
    opts.host_chunks = 3
    with pytest.raises(sa.AttnError):
        call(opts, scan_order=7)
    stream.synchronize()
    assert all((d == 77).all() for d in dev)        # nothing was copied
    call(opts)
    stream.synchronize()
    sa.attn_device_status()
    assert torch.equal(o_host, want.view(torch.int16).cpu())


def test_repeated_calls_reuse_cached_tensor_maps_correctly():
    """The library keeps the tensor maps of the last few (pointers, shape) combinations a thread used: alternating between
    two sets of buffers, and reusing one buffer with another shape, must keep giving each call its own result."""
    import torch
    import paper_2601_16032_b200 as sa
    wa = wl.small_workload("maps-a", 1, 2, 640, 128, wl.BF16, False, 7500)
    wb = wl.small_workload("maps-b", 1, 2, 640, 128, wl.BF16, False, 7501)
    a, b = upload(wa), upload(wb)
    want_a, want_b = run_cuda(wa, a, sa.CYCLIC), run_cuda(wb, b, sa.CYCLIC)
    for _ in range(3):
        assert torch.equal(run_cuda(wa, a, sa.CYCLIC), want_a)
        assert torch.equal(run_cuda(wb, b, sa.CYCLIC), want_b)
    # same buffers read as one head of twice the length
    wc = wl.small_workload("maps-c", 1, 1, 1280, 128, wl.BF16, True, 7502)
    qc, kc, vc = (t.view(1, 1, 1280, 128) for t in a)
    o = torch.empty_like(qc)
    sa.attn_fwd(qc.data_ptr(), kc.data_ptr(), vc.data_ptr(), o.data_ptr(), 1, 1, 1280, 128, wc.scale, 1, sa.CYCLIC, sa.BF16,
                torch.cuda.current_stream().cuda_stream)
    sa.attn_device_status()
    from oracle import attention as ora
    f = lambda t: t[0, 0].double().cpu().numpy()
    err = np.abs(f(o) - ora.attention_head(f(qc), f(kc), f(vc), wc.scale, True))
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    assert torch.equal(run_cuda(wa, a, sa.CYCLIC), want_a)


@pytest.mark.parametrize("N", [1, 100, 128])
@pytest.mark.parametrize("kv_stages", [0, 3])
def test_many_one_tile_items_per_cta(N, kv_stages):
    """Heads of at most 128 rows: the second Q tile of every work item lies beyond N, so its MMA lane has nothing to wait for
    and runs ahead of the softmax warps, item after item.  Few CTAs, many items each, repeated launches, static and
    dynamic schedule: the staging slot of the ring must be handed back by the warps that used it, not by that lane."""
    import torch
    import paper_2601_16032_b200 as sa
    w = wl.small_workload("tiny-items", 4, 8, N, 64, wl.BF16, False, 7700 + N)
    qkv = upload(w)
    q, k, v = qkv
    opts = opts_for(kv_stages=kv_stages, max_ctas=2, block_n=64)
    want = None
    for rep in range(10):
        o = run_cuda(w, qkv, sa.CYCLIC, opts)
        if want is None:
            assert_parity(w, o)
            want = o
        else:
            assert torch.equal(o.view(torch.int16), want.view(torch.int16))
    dyn = opts_for(kv_stages=kv_stages, max_ctas=2, block_n=64, pairing=1)
    nb = sa.attn_dynamic_scratch_bytes(2)
    scratch = torch.zeros(nb // 4, dtype=torch.int32, device=q.device)
    for rep in range(10):
        o = torch.full_like(q, float("nan"))
        sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 0, sa.CYCLIC, sa.BF16,
                            torch.cuda.current_stream().cuda_stream, dyn, scratch.data_ptr(), nb)
        sa.attn_device_status()
        assert torch.equal(o.view(torch.int16), want.view(torch.int16))


@pytest.mark.parametrize("shape", [(64, 128, 2), (64, 64, 2), (64, 128, 1), (128, 128, 1), (128, 64, 2), (128, 64, 1)],
                         ids=lambda t: f"d{t[0]}bn{t[1]}q{t[2]}")
@pytest.mark.parametrize("N,causal", [(129, False), (257, False), (385, True), (641, True), (900, False)])
@pytest.mark.parametrize("kv_stages,max_ctas", [(0, 1), (2, 2), (3, 3)])
def test_s_buffers_handed_round_in_product_order(shape, N, causal, kv_stages, max_ctas):
    """The tile shapes that leave tensor memory room for more S buffers than Q tiles (d = 64, a single Q tile, 64-row K/V
    tiles): S of a tile's next step is issued before its present P is waited for, and the buffers go round in the order
    of the products of both tiles.  Ragged heads make that order irregular: second tiles that lie beyond N for whole
    items (their MMA lane skips those products and runs ahead), diagonals that end one tile's products a step before the
    other's, backward scans that start with such a step.  Few CTAs with many items each, shallow K/V rings, static and
    dynamic schedule, both orders, launches repeated: the result stays the oracle's, and the static one bit for bit."""
    import torch
    import paper_2601_16032_b200 as sa
    d, block_n, q_tiles = shape
    w = wl.small_workload("s-buffers", 2, 3, N, d, wl.BF16 if d == 128 else wl.F16, causal, 7800 + N)
    qkv = upload(w)
    q, k, v = qkv
    adt = sa.BF16 if d == 128 else sa.F16
    for order in (sa.CYCLIC, sa.SAWTOOTH):
        opts = opts_for(block_n, q_tiles, kv_stages=kv_stages, max_ctas=max_ctas)
        first = run_cuda(w, qkv, order, opts)
        assert_parity(w, first)
        for _ in range(3):
            assert torch.equal(run_cuda(w, qkv, order, opts).view(torch.int16), first.view(torch.int16))
        dyn = opts_for(block_n, q_tiles, kv_stages=kv_stages, max_ctas=max_ctas, pairing=1)
        nb = sa.attn_dynamic_scratch_bytes(max_ctas)
        scratch = torch.zeros(nb // 4, dtype=torch.int32, device=q.device)
        for _ in range(2):
            o = torch.full_like(q, float("nan"))
            sa.attn_fwd_dynamic(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, int(causal), order,
                                adt, torch.cuda.current_stream().cuda_stream, dyn, scratch.data_ptr(), nb)
            sa.attn_device_status()
            assert_parity(w, o)


def test_calls_captured_in_a_cuda_graph_replay_bit_for_bit():
    """After one call outside any capture (the library looks its device symbols up and raises the kernel's shared-memory
    limit on a device's first call), attn_fwd, attn_fwd_ex with a log-sum-exp output and attn_fwd_dynamic only enqueue
    work on the stream they are given: captured into a CUDA graph and replayed on new inputs in the same buffers, they
    give what the direct calls give."""
    import torch
    import paper_2601_16032_b200 as sa
    wa = wl.small_workload("graph-a", 1, 3, 1100, 128, wl.BF16, True, 7950)
    wb = wl.small_workload("graph-b", 1, 3, 1100, 128, wl.BF16, True, 7951)
    a, b = upload(wa), upload(wb)
    q, k, v = (torch.empty_like(t) for t in a)
    o1, o2, o3 = (torch.empty_like(q) for _ in range(3))
    lse = torch.empty((wa.B, wa.H, wa.N), dtype=torch.float32, device=q.device)
    opts = sa.Opts()
    opts.lse = lse.data_ptr()
    single = sa.Opts()
    single.pairing = sa.PAIR_NONE
    nb = sa.attn_dynamic_scratch_bytes(sa.attn_query_plan(wa.B, wa.H, wa.N, wa.d, 1, sa.BF16, single).grid)
    scratch = torch.zeros(nb // 4, dtype=torch.int32, device=q.device)

    def calls(stream):
        args = (q.data_ptr(), k.data_ptr(), v.data_ptr())
        shape = (wa.B, wa.H, wa.N, wa.d, wa.scale, 1, sa.SAWTOOTH, sa.BF16, stream)
        sa.attn_fwd(*args, o1.data_ptr(), *shape)
        sa.attn_fwd_ex(*args, o2.data_ptr(), *shape, opts)
        sa.attn_fwd_dynamic(*args, o3.data_ptr(), *shape, None, scratch.data_ptr(), nb)

    for dst, src in zip((q, k, v), a):
        dst.copy_(src)
    calls(torch.cuda.current_stream().cuda_stream)     # the first calls on the device, outside the capture
    torch.cuda.synchronize()
    sa.attn_device_status()
    want_a = [t.clone() for t in (o1, o2, o3, lse)]
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            calls(torch.cuda.current_stream().cuda_stream)
    torch.cuda.current_stream().wait_stream(side)
    for inputs, want in ((b, None), (a, want_a)):
        for dst, src in zip((q, k, v), inputs):
            dst.copy_(src)
        for t in (o1, o2, o3):
            t.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        sa.attn_device_status()
        if want is None:
            assert_parity(wb, o1)
            assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
            assert_parity(wb, o3)
        else:
            for got, w_ in zip((o1, o2, o3), want[:3]):
                assert torch.equal(got.view(torch.int16), w_.view(torch.int16))
            assert torch.equal(lse, want[3])


def test_host_entry_point_from_two_threads():
    """Two host threads, each with its own stream and buffers, call attn_fwd_host at the same time (ctypes drops the
    interpreter lock during the call): the device's one pipeline is handed from call to call under its lock, and both
    get the device entry point's result bit for bit.  The device entry point is called from both threads as well (its
    tensor-map cache is per thread, the per-device state behind a lock)."""
    import threading
    import torch
    import paper_2601_16032_b200 as sa
    jobs = []
    for i in range(2):
        w = wl.small_workload(f"host-thread-{i}", 1, 6, 600 + 100 * i, 128, wl.BF16, True, 7360 + i)
        q, k, v = upload(w)
        want = run_cuda(w, (q, k, v), sa.CYCLIC)
        host = [t.view(torch.int16).cpu().pin_memory() for t in (q, k, v)]
        o_host = torch.full(q.shape, -1, dtype=torch.int16).pin_memory()
        dev = [torch.empty_like(q) for _ in range(4)]
        jobs.append(dict(w=w, q=q, k=k, v=v, want=want, host=host, o_host=o_host, dev=dev, stream=torch.cuda.Stream(), errors=[]))

    def work(j):
        try:
            torch.cuda.set_device(0)
            w = j["w"]
            opts = sa.Opts()
            opts.host_chunks = 3
            for _ in range(5):
                j["o_host"].fill_(-1)
                sa.attn_fwd_host(j["host"][0].data_ptr(), j["host"][1].data_ptr(), j["host"][2].data_ptr(), j["o_host"].data_ptr(),
                                 j["dev"][0].data_ptr(), j["dev"][1].data_ptr(), j["dev"][2].data_ptr(), j["dev"][3].data_ptr(),
                                 w.B, w.H, w.N, w.d, w.scale, 1, sa.CYCLIC, sa.BF16, j["stream"].cuda_stream, opts)
                j["stream"].synchronize()
                if not torch.equal(j["o_host"], j["want"].view(torch.int16).cpu()):
                    j["errors"].append("host result differs")
                o = torch.empty_like(j["q"])
                sa.attn_fwd(j["q"].data_ptr(), j["k"].data_ptr(), j["v"].data_ptr(), o.data_ptr(), w.B, w.H, w.N, w.d, w.scale, 1,
                            sa.CYCLIC, sa.BF16, j["stream"].cuda_stream)
                j["stream"].synchronize()
                if not torch.equal(o, j["want"]):
                    j["errors"].append("device result differs")
        except Exception as e:   # surfaces in the main thread below
            j["errors"].append(repr(e))

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    sa.attn_device_status()
    assert all(not j["errors"] for j in jobs), [j["errors"] for j in jobs]
