"""Pins of the oracle's averageGradients() + Adam step: a hand-worked exact example, special cases, and the
definition of IEEE binary32 rounding applied to each operation with exact rational arithmetic (square root
included: the rounded root is checked by squaring its neighbours)."""
from fractions import Fraction

import numpy as np

from oracle import cref
from tests.helpers import f32, read_sections
from tests.test_oracle_average_sgd import _fl32, _two_streams

SEC = read_sections("worked_bins.txt")
A = SEC["average_adam"]


def test_hand_worked_adam_step():
    n = int(A["an"][0])
    streams = _two_streams()
    # the fixture covers the first bin: run the whole layer, compare its first four elements
    N = int(SEC[""]["n"][0])
    pad = lambda v, fill: np.concatenate([f32(v), np.full(N - n, fill, np.float32)])
    w, m, v = cref.average_adam(streams, N, pad(A["w_in"], 1), pad(A["m_in"], 0), pad(A["v_in"], 1),
                                float(A["step_size"][0]), float(A["beta1"][0]), float(A["beta2"][0]), float(A["eps"][0]))
    np.testing.assert_array_equal(m[:n], f32(A["m_out"]))
    np.testing.assert_array_equal(v[:n], f32(A["v_out"]))
    np.testing.assert_array_equal(w[:n], f32(A["w_out"]))


def test_special_cases():
    rng = np.random.default_rng(41)
    n, L = 2003, 50
    streams = [cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L).raw for _ in range(2)]
    w = rng.normal(0, 1, n).astype(np.float32)
    m = rng.normal(0, 1e-3, n).astype(np.float32)
    v = (rng.normal(0, 1e-3, n).astype(np.float32)) ** 2
    # step_size 0: the weights stay, the moments move
    w1, m1, v1 = cref.average_adam(streams, n, w, m, v, 0.0, 0.9, 0.999, 1e-8)
    np.testing.assert_array_equal(w1, w)
    assert not np.array_equal(m1, m) and not np.array_equal(v1, v)
    # beta1 = beta2 = 0: m' is the mean, v' its square, the step is step_size * mean / (|mean| + eps)
    dense = cref.unpack_sum(streams, n) / np.float32(2)
    w2, m2, v2 = cref.average_adam(streams, n, w, m, v, 0.5, 0.0, 0.0, 1e-8)
    np.testing.assert_array_equal(m2, dense)
    np.testing.assert_array_equal(v2, dense * dense)
    idle = dense == 0
    np.testing.assert_array_equal(w2[idle], w[idle])          # 0 / eps = 0: nothing moves where nobody sent
    assert np.all(np.abs(w2[~idle] - w[~idle]) <= 0.5 * (1 + 1e-6))


def _sqrt32(x: Fraction) -> Fraction:
    """Correctly rounded binary32 square root of a non-negative binary32 value, by exact comparison of squares."""
    if x == 0:
        return Fraction(0)
    guess = Fraction(float(np.sqrt(np.float64(float(x)))))        # close; refined below
    r = _fl32(guess)
    f = np.float32(float(r))
    cands = [Fraction(float(c)) for c in (np.nextafter(f, np.float32(0)), f, np.nextafter(f, np.float32(np.inf)))]
    # the rounded root is the candidate nearest to the true root: compare midpoints' squares with x
    best = cands[0]
    for lo, hi in zip(cands, cands[1:]):
        mid = (lo + hi) / 2
        if mid * mid < x or (mid * mid == x and (int(hi / (hi - lo)) % 2 == 0)):
            best = hi
    return best


def test_every_operation_is_rounded_on_its_own():
    rng = np.random.default_rng(42)
    n, L, k = 300, 50, 3
    streams = [cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), rng.normal(0, 1e-3, n).astype(np.float32), L).raw
               for _ in range(k)]
    w = rng.normal(0, 1, n).astype(np.float32)
    m = rng.normal(0, 1e-3, n).astype(np.float32)
    v = (rng.normal(0, 1e-3, n).astype(np.float32)) ** 2
    ss, b1, b2, eps = np.float32(1e-3), np.float32(0.9), np.float32(0.999), np.float32(1e-8)
    w_new, m_new, v_new = cref.average_adam(streams, n, w, m, v, float(ss), float(b1), float(b2), float(eps))
    dense = cref.unpack_sum(streams, n)
    F = lambda x: Fraction(float(x))
    c1, c2 = _fl32(1 - F(b1)), _fl32(1 - F(b2))
    for i in range(n):
        mean = _fl32(F(dense[i]) / k)
        mm = _fl32(_fl32(F(b1) * F(m[i])) + _fl32(c1 * mean))
        vv = _fl32(_fl32(F(b2) * F(v[i])) + _fl32(c2 * _fl32(mean * mean)))
        den = _fl32(_sqrt32(vv) + F(eps))
        ww = _fl32(F(w[i]) - _fl32(_fl32(F(ss) * mm) / den))
        assert F(m_new[i]) == mm, i
        assert F(v_new[i]) == vv, i
        assert F(w_new[i]) == ww, i
