"""The seeded input generators: reproducible, correctly rounded, exactly widened."""
import numpy as np
import torch

import workloads as wl


def test_bf16_rounding_matches_torch_and_widening_is_exact():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    x[:4] = [1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -0.0, 65504.0]  # two ties, a signed zero
    bits = wl.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16)
    assert (torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16) == want).all()
    np.testing.assert_array_equal(wl.bits_to_f64(bits, wl.BF16), want.to(torch.float64).numpy())


def test_f16_rounding_matches_torch_and_widening_is_exact():
    x = np.random.default_rng(1).standard_normal(100000).astype(np.float32)
    bits = wl.f32_to_f16_bits(x)
    want = torch.from_numpy(x).to(torch.float16)
    assert (torch.from_numpy(bits.view(np.int16)).view(torch.float16) == want).all()
    np.testing.assert_array_equal(wl.bits_to_f64(bits, wl.F16), want.to(torch.float64).numpy())


def test_heads_are_reproducible_and_distinct():
    w = wl.CONFIGS["c2"]
    a = wl.head_bits(w, "k", 0, 3)
    assert a.shape == (w.N, w.d) and a.dtype == np.uint16
    np.testing.assert_array_equal(a, wl.head_bits(w, "k", 0, 3))
    assert (a != wl.head_bits(w, "k", 0, 4)).mean() > 0.9
    assert (a != wl.head_bits(w, "v", 0, 3)).mean() > 0.9
    x = wl.bits_to_f64(a, w.dtype)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01


def test_k_scale_is_exact():
    w = wl.CONFIGS["c4"]
    small = wl.small_workload("t", 1, 1, 256, 128, wl.BF16, True, w.seed, k_scale=0.5)
    plain = wl.small_workload("t", 1, 1, 256, 128, wl.BF16, True, w.seed, k_scale=1.0)
    np.testing.assert_array_equal(wl.bits_to_f64(wl.head_bits(small, "k", 0, 0), wl.BF16) * 2,
                                  wl.bits_to_f64(wl.head_bits(plain, "k", 0, 0), wl.BF16))


def test_checked_rows_plan():
    for name, w in wl.CONFIGS.items():
        plan = wl.checked_rows(w)
        assert set(plan) == set(wl.all_heads(w))
        for rows in plan.values():
            if rows is not None:
                assert (np.diff(rows) > 0).all() and rows[0] == 0 and rows[-1] == w.N - 1
    c3 = wl.checked_rows(wl.CONFIGS["c3"])
    assert c3[(0, 0)] is None and c3[(3, 15)] is None
    assert sum(len(r) for r in c3.values() if r is not None) >= 1024
    c5 = wl.checked_rows(wl.CONFIGS["c5"])
    assert all(r is not None and len(r) >= 512 for r in c5.values())


def test_flops_and_bytes():
    assert wl.CONFIGS["c3"].flops == 4 * 4 * 16 * 8192 ** 2 * 128
    assert wl.CONFIGS["c4"].flops == 2 * 32 * 32768 ** 2 * 128
    assert wl.CONFIGS["c5"].compulsory_bytes == 2 * 1024 ** 3
