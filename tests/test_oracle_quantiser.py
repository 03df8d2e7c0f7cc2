"""Pins of the oracle's second quantiser (Section 2.5 leaves the quantisation function open): sign(G) times the
mean |G| of the sent elements in place of the mean of the bin maxima.  The selection, the word format and the
residue rule (G - Gq where sent) are Algorithm 2's; only the one value per layer changes."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import cref, scalar


def nearest_f32(q: Fraction) -> np.float32:
    """The binary32 value nearest to an exact rational, ties to even (checked by exact comparison of the two
    neighbours, so this helper shares nothing with the code under test)."""
    x = np.float32(float(q))
    lo, hi = np.nextafter(x, np.float32(-np.inf)), np.nextafter(x, np.float32(np.inf))
    best = min((lo, x, hi), key=lambda c: (abs(Fraction(float(c)) - q), int(np.float32(c).view(np.uint32)) & 1))
    return np.float32(best)


def test_hand_worked_bins_with_the_sent_mean():
    """The worked example of the main fixture (L_T = 4, n = 14): bin 0 sends places 0, 1, 3 (|G| .5, .25, .25),
    bin 1 places 0 and 3 (.75, .75), bin 2 nothing, bin 3 both (.25, .5).  Seven sent elements, sum 3.25:
    scale = 3.25 / 7 rounded to binary32; every sent residue is G -/+ that, rounded once."""
    residue = np.array([0, 0, 0, 0, 1, 0, 0, .5, .25, 0, 0, 0, 1, .25], np.float32)
    dW = np.array([.5, -.25, .125, .25, -.25, .125, -.125, .25, -.25, 0, 0, 0, -.75, .25], np.float32)
    G = residue + dW
    r = residue.copy()
    p = cref.pack(dW, r, 4, quantiser=1)
    assert p.n_sel == 7 and list(p.bin_cnt) == [3, 2, 0, 2]
    assert bytes(p.words) == bytes([0x01, 0x07, 0x0D, 0x01, 0x0D, 0x01, 0x05])       # the words do not change
    assert p.flags == 4
    want_scale = nearest_f32(Fraction(13, 4) / 7)
    assert p.scale.view(np.uint32) == want_scale.view(np.uint32)
    sent = [0, 1, 3, 4, 7, 12, 13]
    for i in range(14):
        if i in sent:
            q = Fraction(float(want_scale)) * (-1 if np.signbit(G[i]) else 1)
            assert r[i].view(np.uint32) == nearest_f32(Fraction(float(G[i])) - q).view(np.uint32), i
        else:
            assert r[i] == G[i]
    # the paper's quantiser on the same data: same selection, scale 1.75 / 4
    r0 = residue.copy()
    p0 = cref.pack(dW, r0, 4)
    assert bytes(p0.words) == bytes(p.words) and float(p0.scale) == 0.4375 and p0.flags == 0


def test_closed_forms():
    rng = np.random.default_rng(5)
    n = 5000
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    res = rng.normal(0, 2e-3, n).astype(np.float32)
    # local selection alone (factor 1) on continuous data: exactly the bin maxima are sent, so the mean |G| of the
    # sent elements IS the mean of the bin maxima: the two quantisers give the same scale, residue and words
    a, b = res.copy(), res.copy()
    pa = cref.pack(dW, a, 50, factor=1.0)
    pb = cref.pack(dW, b, 50, factor=1.0, quantiser=1)
    assert pa.n_sel == pa.n_bins == pb.n_sel
    assert pa.scale_bits == pb.scale_bits and bytes(pa.words) == bytes(pb.words) and np.array_equal(a, b)
    assert pa.flags == 2 and pb.flags == 6
    # L_T = 1: every non-zero element is sent: the scale is the mean |G|, by either definition
    a, b = res.copy(), res.copy()
    pa, pb = cref.pack(dW, a, 1), cref.pack(dW, b, 1, quantiser=1)
    assert pa.n_sel == n and pa.scale_bits == pb.scale_bits and np.array_equal(a, b)
    # nothing sent: scale 0
    z = np.zeros(100, np.float32)
    p = cref.pack(z, z.copy(), 50, quantiser=1)
    assert p.n_sel == 0 and p.scale_bits == 0


def test_the_sent_mean_is_the_exactly_rounded_mean_and_lowers_the_squared_error():
    rng = np.random.default_rng(6)
    for L_T, n in ((50, 20011), (500, 30000), (7, 999)):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        res = rng.normal(0, 2e-3, n).astype(np.float32)
        G = res + dW
        r0, r1 = res.copy(), res.copy()
        p0 = cref.pack(dW, r0, L_T)
        p1 = cref.pack(dW, r1, L_T, quantiser=1)
        assert bytes(p0.words) == bytes(p1.words) and np.array_equal(p0.bin_cnt, p1.bin_cnt)   # same selection
        pos, _ = p1.positions_and_codes()
        total = sum((Fraction(float(abs(G[i]))) for i in pos), Fraction(0))
        want = np.float32(float(total) / float(len(pos)))
        assert p1.scale_bits == int(want.view(np.uint32))
        assert min(abs(G[pos])) <= p1.scale <= max(abs(G[pos]))
        # residues: G - sign * scale, one rounded subtraction; and a smaller squared error on the sent elements
        q = np.where(np.signbit(G[pos]), -p1.scale, p1.scale).astype(np.float32)
        assert np.array_equal(r1[pos], G[pos] - q)
        err0 = float(np.sum(r0[pos].astype(np.float64) ** 2))
        err1 = float(np.sum(r1[pos].astype(np.float64) ** 2))
        assert err1 <= err0


@pytest.mark.parametrize("L_T", [1, 2, 3, 4, 8])
def test_brute_force_against_the_scalar_restatement(L_T):
    rng = np.random.default_rng(100 + L_T)
    values = np.array([0, .125, -.125, .25, -.25, .5, -.5, 1, -1], np.float32)
    for _ in range(400):
        n = int(rng.integers(1, 9))
        dW = rng.choice(values, n)
        res = rng.choice(values, n)
        literal = bool(rng.integers(0, 2))
        factor = float(rng.choice([0.0, 1.0, 1.5]))
        r = res.copy()
        p = cref.pack(dW, r, L_T, flags=int(literal), factor=factor, quantiser=1)
        bc, words, scale, new_r, _ = scalar.pack(dW, res, L_T, literal=literal, factor=factor, quantiser=1)
        assert bytes(p.raw) == scalar.to_stream(n, L_T, bc, words, scale, literal=literal, factor=factor, quantiser=1)
        assert np.array_equal(r.view(np.uint32), np.array(new_r, np.float32).view(np.uint32))
