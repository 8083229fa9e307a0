"""Pins of the attention oracle against things other than itself: library routines, closed forms,
exact rational arithmetic and the invariants of softmax attention.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch

from oracle import attention as ora


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


CASES = [(7, 5, 3), (33, 33, 8), (64, 64, 16), (50, 50, 64), (130, 130, 32)]


@pytest.mark.parametrize("n,_,d", CASES)
@pytest.mark.parametrize("causal", [False, True])
def test_matches_scipy_softmax_times_v(n, _, d, causal):
    """Library routine: scipy's softmax over masked scores, then a matrix product."""
    q, k, v = rnd((n, d), 1), rnd((n, d), 2), rnd((n, d), 3)
    scale = 0.37
    s = scale * np.einsum("id,jd->ij", q, k)
    if causal:
        s[np.triu_indices(n, 1)] = -np.inf
    want = scipy.special.softmax(s, axis=1) @ v
    np.testing.assert_allclose(ora.attention_head(q, k, v, scale, causal), want, rtol=0, atol=1e-13)
    np.testing.assert_allclose(ora.attention_definition(q, k, v, scale, causal), want, rtol=0, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_matches_torch_sdpa_fp64(causal):
    """Library routine: torch's scaled_dot_product_attention on CPU in fp64 (scale and mask its own)."""
    n, d = 96, 24
    q, k, v = rnd((n, d), 4), rnd((n, d), 5), rnd((n, d), 6)
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (q, k, v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal)[0, 0].numpy()
    scale = 1.0 / np.sqrt(d)
    np.testing.assert_allclose(ora.attention_head(q, k, v, scale, causal), want, rtol=0, atol=1e-13)
    np.testing.assert_allclose(ora.attention_definition(q, k, v, scale, causal), want, rtol=0, atol=1e-13)


def test_two_keys_closed_form():
    """Two keys: softmax is the logistic function, o = v1 + (v0 - v1) * sigmoid(scale * q.(k0 - k1))."""
    d = 6
    q, k, v = rnd((1, d), 7), rnd((2, d), 8), rnd((2, d), 9)
    scale = 1.7
    w0 = scipy.special.expit(scale * float(q[0] @ (k[0] - k[1])))
    want = v[1] + (v[0] - v[1]) * w0
    got = ora.attention_rows(q, np.array([1]), k, v, scale, False)
    np.testing.assert_allclose(got[0], want, rtol=0, atol=1e-14)
    # dropping the scale, or putting it on the wrong side of the exponent, fails this
    assert abs(scipy.special.expit(float(q[0] @ (k[0] - k[1]))) - w0) > 1e-3


def test_exact_rational_brute_force():
    """Integer-valued q, k and scale = ln 2 make every weight a power of two, so the result is an
    exact rational number; compare with Fractions on a tiny case."""
    rng = np.random.default_rng(10)
    n, d = 9, 4
    q = rng.integers(-2, 3, (n, d)).astype(float)
    k = rng.integers(-2, 3, (n, d)).astype(float)
    v = rng.integers(-8, 9, (n, d)).astype(float)
    for causal in (False, True):
        got = ora.attention_head(q, k, v, np.log(2.0), causal)
        got_def = ora.attention_definition(q, k, v, np.log(2.0), causal)
        for i in range(n):
            keys = range(i + 1) if causal else range(n)
            e = {j: int(sum(int(q[i, t]) * int(k[j, t]) for t in range(d))) for j in keys}
            lo = min(e.values())
            w = {j: Fraction(2) ** (e[j] - lo) for j in keys}
            den = sum(w.values())
            for t in range(d):
                want = sum(w[j] * int(v[j, t]) for j in keys) / den
                assert abs(got[i, t] - float(want)) < 1e-13
                assert abs(got_def[i, t] - float(want)) < 1e-13


@pytest.mark.parametrize("causal", [False, True])
def test_v_identity_returns_the_softmax_matrix_and_rows_sum_to_one(causal):
    """With V = I the output is the probability matrix itself: rows sum to 1, masked entries are 0."""
    n = 40
    q, k = rnd((n, n), 11), rnd((n, n), 12)
    p = ora.attention_head(q, k, np.eye(n), 0.2, causal)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-14)
    assert (p >= 0).all()
    if causal:
        assert (p[np.triu_indices(n, 1)] == 0).all()
        assert (np.diag(p) > 0).all()  # the diagonal key is visible


@pytest.mark.parametrize("causal", [False, True])
def test_v_ones_gives_ones(causal):
    n, d = 70, 8
    o = ora.attention_head(rnd((n, d), 13), rnd((n, d), 14), np.ones((n, d)), 0.5, causal)
    np.testing.assert_allclose(o, 1.0, rtol=0, atol=1e-14)


def test_one_hot_score_row_selects_that_v_row():
    n, d = 32, 8
    k, v = rnd((n, d), 15), rnd((n, d), 16)
    k /= np.linalg.norm(k, axis=1, keepdims=True)
    target = 19
    q = 400.0 * k[target][None, :]  # score of the target exceeds every other by a wide margin
    gaps = 400.0 * (1.0 - k @ k[target])
    assert np.sort(gaps)[1] > 60
    got = ora.attention_rows(q, np.array([n - 1]), k, v, 1.0, False)
    np.testing.assert_allclose(got[0], v[target], rtol=0, atol=1e-12)
    # a flipped sign in the exponent would pick the most negative score instead
    assert np.argmin(k @ k[target]) != target


def test_zero_keys_give_means_of_visible_values():
    """K = 0: uniform weights.  Non-causal: the mean of V.  Causal: the running mean of V rows 0..i."""
    n, d = 57, 5
    q, v = rnd((n, d), 17), rnd((n, d), 18)
    k = np.zeros((n, d))
    np.testing.assert_allclose(ora.attention_head(q, k, v, 0.3, False), np.tile(v.mean(0), (n, 1)), atol=1e-14)
    prefix = np.cumsum(v, axis=0) / np.arange(1, n + 1)[:, None]
    np.testing.assert_allclose(ora.attention_head(q, k, v, 0.3, True), prefix, atol=1e-14)


def test_causal_first_row_is_first_value_row_and_last_row_sees_everything():
    n, d = 21, 7
    q, k, v = rnd((n, d), 19), rnd((n, d), 20), rnd((n, d), 21)
    c = ora.attention_head(q, k, v, 0.4, True)
    f = ora.attention_head(q, k, v, 0.4, False)
    np.testing.assert_array_equal(c[0], v[0])
    np.testing.assert_allclose(c[-1], f[-1], atol=1e-15)
    assert np.abs(c[:-1] - f[:-1]).max() > 1e-3


def test_shift_invariance():
    """A constant added to every score of a row (an extra feature equal in all keys) changes nothing."""
    n, d = 30, 6
    q, k, v = rnd((n, d), 22), rnd((n, d), 23), rnd((n, d), 24)
    q2 = np.concatenate([q, rnd((n, 1), 25)], axis=1)
    k2 = np.concatenate([k, np.full((n, 1), 3.25)], axis=1)
    v_pad = np.concatenate([v, np.zeros((n, 1))], axis=1)
    a = ora.attention_head(q, k, v, 0.5, False)
    b = ora.attention_head(q2, k2, v_pad, 0.5, False)[:, :d]
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_sampled_rows_equal_full_rows():
    n, d = 200, 16
    q, k, v = rnd((n, d), 26), rnd((n, d), 27), rnd((n, d), 28)
    rows = np.array([0, 3, 127, 128, 199])
    for causal in (False, True):
        full = ora.attention_head(q, k, v, 0.25, causal)
        part = ora.attention_rows(q[rows], rows, k, v, 0.25, causal)
        np.testing.assert_array_equal(part, full[rows])
        one = ora.attention_rows(q[rows], rows, k, v, 0.25, causal, threads=1)
        np.testing.assert_array_equal(one, part)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("T_r,T_c", [(16, 16), (32, 8), (16, 48), (128, 64)])
def test_algorithm1_online_update_reaches_the_definition_in_any_scan_order(causal, T_r, T_c):
    """Algorithm 1 with forward, backward and alternating (sawtooth) K/V scans equals Eq. 1."""
    n, d = 150, 12  # ragged against every tile size above
    q, k, v = rnd((n, d), 29), rnd((n, d), 30, 2.0), rnd((n, d), 31)
    want = ora.attention_head(q, k, v, 0.6, causal)

    def sawtooth(i, n_kv):
        return ora.scan_backward(i, n_kv) if i % 2 else ora.scan_forward(i, n_kv)

    for order in (ora.scan_forward, ora.scan_backward, sawtooth):
        got = ora.attention_online(q, k, v, 0.6, causal, T_r, T_c, order)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)


def test_rejects_bad_arguments():
    q = rnd((2, 4), 1)
    with pytest.raises(RuntimeError):
        ora.attention_rows(q, np.array([0, 9]), rnd((3, 4), 2), rnd((3, 4), 3), 1.0, False)
    with pytest.raises(ValueError):
        ora.attention_rows(q, np.array([0, 1]), rnd((3, 5), 2), rnd((3, 4), 3), 1.0, False)


@pytest.mark.parametrize("n,_,d", CASES)
@pytest.mark.parametrize("causal", [False, True])
def test_logsumexp_matches_scipy(n, _, d, causal):
    """Library routine: scipy's logsumexp over the masked score rows."""
    q, k = rnd((n, d), 21), rnd((n, d), 22)
    scale = 0.41
    s = scale * np.einsum("id,jd->ij", q, k)
    if causal:
        s[np.triu_indices(n, 1)] = -np.inf
    want = scipy.special.logsumexp(s, axis=1)
    rows = np.arange(n, dtype=np.int64)
    np.testing.assert_allclose(ora.logsumexp_rows(q, rows, k, scale, causal), want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(ora.logsumexp_definition(q, k, scale, causal), want, rtol=0, atol=1e-12)


def test_logsumexp_closed_forms():
    """K = 0 makes every score 0: the row sees c keys and lse = ln c (c = N, or i + 1 under the causal mask).  One
    score far above the rest gives lse = that score.  Shifting every score of a row by a constant shifts lse by it."""
    n, d = 37, 5
    q, k0 = rnd((n, d), 23), np.zeros((n, d))
    rows = np.arange(n, dtype=np.int64)
    np.testing.assert_allclose(ora.logsumexp_rows(q, rows, k0, 0.7, False), np.full(n, np.log(n)), rtol=0, atol=1e-13)
    np.testing.assert_allclose(ora.logsumexp_rows(q, rows, k0, 0.7, True), np.log(rows + 1.0), rtol=0, atol=1e-13)
    k = rnd((n, d), 24) * 0.01
    k[11] = 50.0 * q[3] / np.dot(q[3], q[3])          # q[3] . k[11] = 50
    got = ora.logsumexp_rows(q[3:4], np.array([3]), k, 2.0, False)
    assert abs(got[0] - 100.0) < 1e-12
    # appending a constant feature c to q and 1 to every k adds c to every score of the row
    q1 = np.concatenate([q, np.full((n, 1), 3.25)], axis=1)
    k1 = np.concatenate([k, np.ones((n, 1))], axis=1)
    np.testing.assert_allclose(ora.logsumexp_rows(q1, rows, k1, 1.0, True) - ora.logsumexp_rows(q, rows, k, 1.0, True),
                               np.full(n, 3.25), rtol=0, atol=1e-12)


def test_logsumexp_normalises_the_definition():
    """exp(s - lse) are the softmax weights: they sum to 1 and reproduce the attention output."""
    n, d = 45, 9
    q, k, v = rnd((n, d), 25), rnd((n, d), 26), rnd((n, d), 27)
    scale = 0.5
    lse = ora.logsumexp_rows(q, np.arange(n, dtype=np.int64), k, scale, True)
    s = scale * (q @ k.T)
    s[np.triu_indices(n, 1)] = -np.inf
    w = np.exp(s - lse[:, None])
    np.testing.assert_allclose(w.sum(axis=1), np.ones(n), rtol=0, atol=1e-13)
    np.testing.assert_allclose(w @ v, ora.attention_head(q, k, v, scale, True), rtol=0, atol=1e-13)
