"""Pins of the oracle's averageGradients() + updateWeights() step (Algorithm 1, after unpack()).

What fixes it without reference to itself: a hand-worked example (tests/golden/worked_bins.txt), the
special cases that reduce to a subtraction or to nothing, and the definition of IEEE binary32
round-to-nearest-even applied to each of the four operations with exact rational arithmetic (which
a fused multiply-add, a multiplication by 1/k or a different operation order would fail).
"""
from fractions import Fraction

import numpy as np

from tests.helpers import f32, read_sections
from oracle import cref

SEC = read_sections("worked_bins.txt")
L_T = int(SEC[""]["L_T"][0])
N = int(SEC[""]["n"][0])


def _two_streams():
    s1, s2 = SEC["step1"], SEC["step2"]
    residue = f32(s1["residue"]).copy()
    p1 = cref.pack(f32(s1["dW"]), residue, L_T)
    p2 = cref.pack(f32(s2["dW"]), residue, L_T)
    return [p1.raw, p2.raw]


def test_hand_worked_update():
    a = SEC["average_sgd"]
    w, v = cref.average_sgd(_two_streams(), N, f32(a["w_in"]), f32(a["v_in"]), float(a["lr"][0]), float(a["mu"][0]))
    np.testing.assert_array_equal(v, f32(a["v_out"]))
    np.testing.assert_array_equal(w, f32(a["w_out"]))
    # the mean itself: with zero momentum and weights, lr = -1 returns it
    w0, v0 = cref.average_sgd(_two_streams(), N, np.zeros(N, np.float32), np.zeros(N, np.float32), -1.0, 0.0)
    np.testing.assert_array_equal(v0, f32(a["mean"]))
    np.testing.assert_array_equal(w0, f32(a["mean"]))


def test_special_cases_reduce_to_textbook_operations():
    rng = np.random.default_rng(5)
    n, L = 3001, 50
    streams = []
    for l in range(3):
        streams.append(cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L).raw)
    w = rng.normal(0, 1, n).astype(np.float32)
    v = rng.normal(0, 1e-2, n).astype(np.float32)
    dense = cref.unpack_sum(streams, n)
    # one learner, no momentum, lr = 1: plain w - gradient
    w1, v1 = cref.average_sgd(streams[:1], n, w, v, 1.0, 0.0)
    d1 = cref.unpack_sum(streams[:1], n)
    np.testing.assert_array_equal(v1, d1)
    np.testing.assert_array_equal(w1, w - d1)
    # lr = 0: the weights do not move, the momentum still does
    w2, v2 = cref.average_sgd(streams, n, w, v, 0.0, 0.9)
    np.testing.assert_array_equal(w2, w)
    assert not np.array_equal(v2, v)
    # where nobody sent anything the mean is +0: v' = mu v there, exactly
    idle = dense == 0
    assert idle.any()
    np.testing.assert_array_equal(v2[idle], (np.float32(0.9) * v)[idle])
    # inputs are left alone
    w_copy, v_copy = w.copy(), v.copy()
    cref.average_sgd(streams, n, w, v, 0.1, 0.9)
    np.testing.assert_array_equal(w, w_copy)
    np.testing.assert_array_equal(v, v_copy)


def _fl32(x: Fraction) -> Fraction:
    """x rounded to the nearest binary32 value, ties to even (exact rational arithmetic; normal and
    subnormal range, no overflow handling: the test stays far from it)."""
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    x = abs(x)
    e = x.numerator.bit_length() - x.denominator.bit_length()
    if Fraction(2) ** e > x:
        e -= 1                                  # 2^e <= x < 2^(e+1)
    e = max(e, -126)                            # subnormals share the exponent of the smallest normal
    ulp = Fraction(2) ** (e - 23)
    q = x / ulp
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * lo * ulp


def test_every_operation_is_rounded_on_its_own():
    rng = np.random.default_rng(11)
    n, L, k = 400, 50, 3
    streams = [cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), rng.normal(0, 1e-3, n).astype(np.float32), L).raw
               for _ in range(k)]
    w = rng.normal(0, 1, n).astype(np.float32)
    v = rng.normal(0, 1e-2, n).astype(np.float32)
    lr, mu = np.float32(0.1), np.float32(0.9)
    w_new, v_new = cref.average_sgd(streams, n, w, v, float(lr), float(mu))
    dense = cref.unpack_sum(streams, n)
    fused_differs = 0
    for i in range(n):
        s = Fraction(float(dense[i]))
        mean = _fl32(s / k)
        mv = _fl32(Fraction(float(mu)) * Fraction(float(v[i])))
        vv = _fl32(mv + mean)
        lv = _fl32(Fraction(float(lr)) * vv)
        ww = _fl32(Fraction(float(w[i])) - lv)
        assert Fraction(float(v_new[i])) == vv, i
        assert Fraction(float(w_new[i])) == ww, i
        # the same with a fused multiply-add, or with a multiplication by fl(1/k), is a different number
        # often enough that the exact match above means something
        fused_v = _fl32(Fraction(float(mu)) * Fraction(float(v[i])) + mean)
        recip = _fl32(s * _fl32(Fraction(1, k)))
        fused_differs += (fused_v != vv) or (recip != mean)
    assert fused_differs > 0
