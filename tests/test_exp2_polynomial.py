"""The cubic the kernel uses for 2^f on the FMA pipe (a quarter of the exponentials at d = 64): its coefficients are read from
the CUDA header and checked on the host against 2^f in fp64, evaluated in fp32 Horner form as the kernel does, and the
range reduction (floor taken from the low mantissa bits of x + 1.5 * 2^23) is replayed with numpy integers."""
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def coefficients():
    text = open(os.path.join(ROOT, "paper_2601_16032_b200", "csrc", "ptx.cuh")).read()
    body = text[text.index("exp2_poly_pair"):]
    body = body[:body.index("y1 =")]
    vals = [np.float32(x) for x in re.findall(r"pack_f32x2\((0\.\d+)f, 0\.\d+f\)", body)]
    assert len(vals) == 4
    c3, c2, c1, c0 = vals
    return c0, c1, c2, c3


def test_cubic_is_within_1e_4_of_two_to_the_f():
    c0, c1, c2, c3 = coefficients()
    f = np.linspace(0.0, 1.0, 200001, dtype=np.float32)
    p = np.float32(c3) * f + np.float32(c2)
    p = p * f + np.float32(c1)
    p = p * f + np.float32(c0)
    rel = np.abs(p.astype(np.float64) / np.exp2(f.astype(np.float64)) - 1.0)
    assert rel.max() < 1e-4          # far below the 2^-9 rounding of a bf16 probability
    assert 0.99 < p.min() and p.max() < 2.001


def test_range_reduction_and_exponent_insertion():
    c0, c1, c2, c3 = coefficients()
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.uniform(-126.0, 8.0, 100000), [-126.0, -125.999, -1.0, -0.5, 0.0, 7.999, -300.0, -np.inf]]).astype(np.float32)
    xc = np.maximum(x, np.float32(-126.0))
    magic = np.float32(12582912.0)
    # x + magic rounded toward minus infinity: at this magnitude one ulp is 1, so the sum is magic + floor(x)
    t = (magic.astype(np.float64) + np.floor(xc.astype(np.float64))).astype(np.float32)
    fl = t - magic
    assert np.array_equal(fl, np.floor(xc))
    f = xc - fl
    p = ((c3 * f + c2) * f + c1) * f + c0
    bits = p.view(np.int32) + (t.view(np.int32) << 23)
    y = bits.view(np.float32)
    want = np.exp2(xc.astype(np.float64))
    ok = want > 1e-37
    assert np.abs(y[ok].astype(np.float64) / want[ok] - 1.0).max() < 1.5e-4
    assert (y[~ok] >= 0).all() and (y[~ok] < 1e-36).all()   # clamped inputs give (nearly) zero, never garbage
