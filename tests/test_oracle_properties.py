"""Pins for the oracle that need no second implementation of its formulae:
closed-form special cases, invariants, metamorphic relations, brute force
against the independent scalar restatement, and the exact sum against
rational arithmetic.  CPU only."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import cref, scalar

RNG = np.random.default_rng(20171202)


def _gauss(n, sigma=1e-3, rng=RNG):
    return rng.normal(0.0, sigma, n).astype(np.float32)


# --------------------------------------------------------------------------
# exact sum (the scale must not depend on summation order)
# --------------------------------------------------------------------------

def _wide_values(count, rng):
    e = rng.integers(-149, 128, count)
    m = rng.integers(1, 1 << 24, count)
    v = np.ldexp(m.astype(np.float64), e - 23)
    v = v[np.isfinite(v) & (v < 3.4e38)].astype(np.float32)
    return np.concatenate([v, np.float32([0.0, 1e-45, 3e38, 3e38, 1.17549435e-38])])


def test_exact_sum_against_fractions_and_fsum_over_60_decades():
    v = _wide_values(20000, np.random.default_rng(1))
    exact = sum((Fraction(float(x)) for x in v), Fraction(0))
    want = float(exact)                       # correctly rounded big-int division
    assert cref.exact_sum(v) == want == math.fsum(float(x) for x in v)
    assert cref.exact_sum(v[::-1].copy()) == want


def test_exact_sum_rounding_ties_to_even_and_sticky():
    one, ulp = 1.0, 2.0 ** -52
    # 2^60 + 2^7 is a tie between two doubles (spacing 2^8): ties-to-even keeps 2^60
    assert cref.exact_sum(np.float32([2.0 ** 60, 2.0 ** 7])) == 2.0 ** 60
    # one more unit below the tie makes it sticky -> rounds up
    assert cref.exact_sum(np.float32([2.0 ** 60, 2.0 ** 7, 2.0 ** -100])) == 2.0 ** 60 + 2.0 ** 8
    # odd mantissa + tie rounds up to even
    assert cref.exact_sum(np.float32([2.0 ** 60, 2.0 ** 8, 2.0 ** 7])) == 2.0 ** 60 + 2.0 ** 9
    assert cref.exact_sum(np.float32([])) == 0.0
    assert cref.exact_sum(np.float32([1e-45] * 3)) == 3 * 2.0 ** -149
    assert one + ulp > one


def test_sequential_float32_sum_would_not_do():
    # why the scale is defined through an exact sum: fp32 accumulation drifts
    g = np.abs(_gauss(2_000_000, 1e-3, np.random.default_rng(5))) + np.float32(2e-3)
    seq = np.float32(0)
    for chunk in np.array_split(g, 2000):
        seq = np.float32(seq + np.float32(chunk.sum(dtype=np.float32)))
    exact = cref.exact_sum(g)
    assert exact == math.fsum(g.astype(np.float64))
    assert exact == float(np.sum(g.astype(np.float64)[::-1]))  # spread of 2 binades: fp64 is exact
    assert abs(float(seq) - exact) / exact > 1e-8


# --------------------------------------------------------------------------
# special cases with a textbook closed form
# --------------------------------------------------------------------------

@pytest.mark.parametrize("L_T,n", [(50, 100352), (500, 200000), (7, 1000), (64, 6400), (65, 6500)])
def test_zero_residue_first_step_closed_form(L_T, n):
    # residue == 0: G = dW and H = 2*dW exactly, so an element is sent iff
    # 2|dW| >= max_bin|dW|, and residue' = dW - sign(dW) * mean(bin maxima)
    dW = _gauss(n)
    residue = np.zeros(n, dtype=np.float32)
    p = cref.pack(dW, residue, L_T, want_gmax=True)
    B = -(-n // L_T)
    pad = np.zeros(B * L_T, dtype=np.float32)
    pad[:n] = np.abs(dW)
    gmax = pad.reshape(B, L_T).max(axis=1)
    np.testing.assert_array_equal(p.g_max, gmax)
    sel = (2.0 * np.abs(dW) >= np.repeat(gmax, L_T)[:n]) & (dW != 0)
    pos, code = p.positions_and_codes()
    np.testing.assert_array_equal(pos, np.flatnonzero(sel))
    np.testing.assert_array_equal(code == 3, dW[sel] < 0)
    scale = np.float32(math.fsum(gmax.astype(np.float64)) / B)
    assert p.scale == scale
    want = dW.copy()
    want[sel] = dW[sel] - np.where(dW[sel] < 0, -scale, scale).astype(np.float32)
    np.testing.assert_array_equal(residue, want)
    np.testing.assert_array_equal(p.bin_cnt, np.add.reduceat(
        np.concatenate([sel, np.zeros(B * L_T - n, bool)]).astype(np.int64), np.arange(0, B * L_T, L_T)))


def test_bin_length_one_is_one_bit_quantisation_with_error_feedback():
    # L_T = 1: every non-zero element is its own bin maximum -> all sent,
    # scale = mean|G| : the 1-bit scheme with mean reconstruction the paper's
    # Background section describes.
    n = 3000
    dW, r0 = _gauss(n), _gauss(n, 5e-3)
    dW[7] = 0.0
    r0[7] = 0.0
    residue = r0.copy()
    p = cref.pack(dW, residue, 1)
    G = r0 + dW
    assert p.n_sel == n - 1 and p.n_bins == n and p.tile_bins == 4000
    scale = np.float32(math.fsum(np.abs(G).astype(np.float64)) / n)
    assert p.scale == scale
    want = (G - np.where(np.signbit(G), -scale, scale).astype(np.float32)).astype(np.float32)
    want[7] = 0.0
    np.testing.assert_array_equal(residue, want)
    assert set(np.unique(p.words)) <= {1, 3}


def test_single_bin_zero_gradient_sends_only_the_global_maximum():
    # L_T >= n and dW == 0: H = G, so only |G| == max is sent (the "local
    # selection" scheme of the Discussions section); its residue becomes exactly 0.
    n = 400
    r0 = _gauss(n, 1.0)
    residue = r0.copy()
    p = cref.pack(np.zeros(n, np.float32), residue, 500)
    k = int(np.argmax(np.abs(r0)))
    assert p.n_sel == 1 and int(p.words[0]) >> 2 == k
    assert p.scale == np.abs(r0[k]) and residue[k] == 0.0
    keep = np.arange(n) != k
    np.testing.assert_array_equal(residue[keep], r0[keep])


def test_zero_gradient_selects_exactly_the_bin_maxima():
    n, L_T = 5000, 50
    r0 = _gauss(n, 1.0)
    r0[100:150] = 0.0                                   # a zero bin
    residue = r0.copy()
    p = cref.pack(np.zeros(n, np.float32), residue, L_T, want_gmax=True)
    assert p.n_sel == p.n_bins - 1 and p.bin_cnt[2] == 0
    assert np.all(np.delete(p.bin_cnt, 2) == 1)


def test_quantise_uses_sign_of_G_not_H():
    # residue 1.0, dW -0.75 -> G = +0.25, H = -0.5: sent with code '+'
    residue = np.float32([1.0, 0.0])
    p = cref.pack(np.float32([-0.75, 0.0]), residue, 2)
    assert p.words.tolist() == [1] and p.scale == np.float32(0.25) and residue[0] == 0.0


def test_empty_and_tiny_inputs():
    p = cref.pack(np.zeros(0, np.float32), np.zeros(0, np.float32), 50)
    assert (p.n, p.n_bins, p.n_tiles, p.n_sel, p.bytes_used) == (0, 0, 0, 0, 80)
    assert p.scale == 0 and p.tile_off.tolist() == [0]
    r = np.float32([0.5])
    p = cref.pack(np.float32([0.25]), r, 16384)
    assert p.n_sel == 1 and p.w == 2 and p.tile_bins == 1 and p.scale == np.float32(0.75)
    assert r[0] == 0.0
    assert cref.unpack_sum([p.raw], 1).tolist() == [0.75]


# --------------------------------------------------------------------------
# invariants on random multi-step runs
# --------------------------------------------------------------------------

@pytest.mark.parametrize("L_T,n,literal", [(50, 100352, 0), (500, 60010, 0), (3, 1001, 0),
                                           (1000, 9999, 0), (1001, 9999, 0), (50, 20000, 1)])
def test_invariants_over_steps(L_T, n, literal):
    rng = np.random.default_rng(L_T * 7919 + n)
    residue = np.zeros(n, np.float32)
    decoded_total = np.zeros(n, np.float64)
    dW_total = np.zeros(n, np.float64)
    steps = 6
    for _ in range(steps):
        dW = _gauss(n, 1e-3, rng)
        if n > 600:
            dW[500:500 + min(L_T, 50)] = 0.0
        r_before = residue.copy()
        p = cref.pack(dW, residue, L_T, flags=literal, want_gmax=True)
        G = r_before + dW
        H = G + dW
        gm = np.repeat(p.g_max, L_T)[:n]
        pos, code = p.positions_and_codes()
        sel = np.zeros(n, bool)
        sel[pos] = True
        # a bin sends something iff its maximum is non-zero (default reading)
        if not literal:
            np.testing.assert_array_equal(p.bin_cnt >= 1, p.g_max > 0)
        # sent <=> passes the soft threshold or is the maximum
        passes = (np.abs(H) >= gm) | ((np.abs(G) == gm) & (literal == 0))
        np.testing.assert_array_equal(sel, passes & (gm > 0) & (G != 0))
        # residue: untouched elements carry G bit for bit; sent ones G -+ scale
        np.testing.assert_array_equal(residue[~sel], G[~sel])
        q = np.where(code == 3, -p.scale, p.scale).astype(np.float32)
        np.testing.assert_array_equal(residue[pos], (G[pos] - q).astype(np.float32))
        np.testing.assert_array_equal(code == 3, np.signbit(G[pos]))
        # ascending positions, counts add up, directory is the exclusive scan
        assert np.all(np.diff(pos) > 0)
        assert int(p.bin_cnt.sum()) == p.n_sel == len(p.words)
        tiles = np.add.reduceat(p.bin_cnt.astype(np.int64), np.arange(0, p.n_bins, p.tile_bins))
        np.testing.assert_array_equal(p.tile_off, np.concatenate([[0], np.cumsum(tiles)]))
        assert p.g_max.min() <= p.scale <= p.g_max.max()
        # decoding returns +-scale exactly where something was sent, zero elsewhere
        dst = cref.unpack_sum([p.raw], n)
        assert np.all(dst[~sel] == 0)
        np.testing.assert_array_equal(dst[pos], q)
        decoded_total += dst
        dW_total += dW
    # error feedback telescopes: what was sent plus what is left is what came in
    err = np.abs(decoded_total + residue - dW_total).max()
    assert err <= steps * 2.0 ** -22 * max(np.abs(dW_total).max(), np.abs(residue).max(), 1e-3)


def test_determinism_same_inputs_same_bytes():
    dW, r = _gauss(20000), _gauss(20000, 3e-3)
    a = cref.pack(dW, r.copy(), 50)
    b = cref.pack(dW, r.copy(), 50)
    assert a.raw.tobytes() == b.raw.tobytes()


# --------------------------------------------------------------------------
# metamorphic relations (exact in binary32)
# --------------------------------------------------------------------------

def test_negation_flips_codes_only():
    dW, r = _gauss(10000), _gauss(10000, 3e-3)
    ra, rb = r.copy(), (-r).copy()
    a = cref.pack(dW, ra, 50)
    b = cref.pack(-dW, rb, 50)
    assert a.scale_bits == b.scale_bits
    np.testing.assert_array_equal(a.bin_cnt, b.bin_cnt)
    np.testing.assert_array_equal(a.words >> 2, b.words >> 2)
    np.testing.assert_array_equal(a.words & 3, 4 - (b.words & 3))
    np.testing.assert_array_equal(ra, -rb)


@pytest.mark.parametrize("k", [-20, 9])
def test_power_of_two_scaling_leaves_the_stream_alone(k):
    dW, r = _gauss(10000), _gauss(10000, 3e-3)
    s = np.float32(2.0 ** k)
    ra, rb = r.copy(), (r * s).copy()
    a = cref.pack(dW, ra, 500)
    b = cref.pack(dW * s, rb, 500)
    assert b.scale == a.scale * s
    np.testing.assert_array_equal(a.words, b.words)
    np.testing.assert_array_equal(a.bin_cnt, b.bin_cnt)
    np.testing.assert_array_equal(ra * s, rb)


def test_permuting_bins_permutes_the_stream_and_keeps_the_scale():
    L_T, B = 50, 400
    dW, r = _gauss(L_T * B), _gauss(L_T * B, 3e-3)
    r[::977] *= np.float32(1e4)       # wide exponent spread: order would matter in fp32/fp64
    perm = np.random.default_rng(3).permutation(B)
    dWp = dW.reshape(B, L_T)[perm].ravel().copy()
    rp = r.reshape(B, L_T)[perm].ravel().copy()
    ra = r.copy()
    a = cref.pack(dW, ra, L_T)
    b = cref.pack(dWp, rp, L_T)
    assert a.scale_bits == b.scale_bits
    np.testing.assert_array_equal(a.bin_cnt[perm], b.bin_cnt)
    np.testing.assert_array_equal(ra.reshape(B, L_T)[perm].ravel(), rp)


def test_appending_a_zero_bin_rescales_by_the_bin_count():
    L_T, B = 50, 99
    dW, r = _gauss(L_T * B), _gauss(L_T * B, 3e-3)
    a = cref.pack(dW, r.copy(), L_T, want_gmax=True)
    z = np.zeros(L_T, np.float32)
    b = cref.pack(np.concatenate([dW, z]), np.concatenate([r, z]), L_T)
    S = math.fsum(a.g_max.astype(np.float64))
    assert a.scale == np.float32(S / B) and b.scale == np.float32(S / (B + 1))
    np.testing.assert_array_equal(a.words, b.words)


# --------------------------------------------------------------------------
# brute force: C oracle vs the scalar Python restatement, byte for byte
# --------------------------------------------------------------------------

VALUES = [0.0, 0.125, -0.125, 0.25, -0.25, 0.5, -0.5, 1.0, -1.0]


@pytest.mark.parametrize("L_T", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("literal", [False, True])
def test_brute_force_tiny_tensors(L_T, literal):
    rng = np.random.default_rng(100 + L_T)
    cases = []
    # exhaustive for n = 2 over the 9-value alphabet (dW and residue): 9^4 = 6561 cases
    if L_T <= 2:
        for combo in itertools.product(VALUES, repeat=4):
            cases.append((combo[:2], combo[2:]))
    for _ in range(3000):
        n = int(rng.integers(1, 9))
        cases.append((rng.choice(VALUES, n), rng.choice(VALUES, n)))
    for dW, r in cases:
        dW = np.asarray(dW, np.float32)
        r = np.asarray(r, np.float32)
        rc = r.copy()
        p = cref.pack(dW, rc, L_T, flags=int(literal))
        cnt, words, scale, res, _ = scalar.pack(dW, r, L_T, literal)
        ref = scalar.to_stream(len(dW), L_T, cnt, words, scale, literal)
        assert p.raw.tobytes() == ref, (dW, r)
        assert rc.tobytes() == np.array(res, np.float32).tobytes(), (dW, r)


def test_brute_force_random_floats_multi_step_and_decode():
    rng = np.random.default_rng(77)
    for L_T, n in [(5, 23), (64, 200), (65, 200), (50, 152)]:
        streams_c, streams_s = [], []
        for learner in range(3):
            r_c = np.zeros(n, np.float32)
            r_s = [np.float32(0)] * n
            for _ in range(3):
                dW = rng.normal(0, 1e-3, n).astype(np.float32)
                p = cref.pack(dW, r_c, L_T)
                cnt, words, scale, r_s, _ = scalar.pack(dW, r_s, L_T)
                assert p.raw.tobytes() == scalar.to_stream(n, L_T, cnt, words, scale)
                assert r_c.tobytes() == np.array(r_s, np.float32).tobytes()
            streams_c.append(p.raw)
            streams_s.append((cnt, words, scale))
        dst = cref.unpack_sum(streams_c, n)
        ref = np.array(scalar.unpack_sum(streams_s, n, L_T), np.float32)
        assert dst.tobytes() == ref.tobytes()


def test_decoder_rejects_reserved_code_and_mismatched_streams():
    dW = _gauss(200)
    p = cref.pack(dW, np.zeros(200, np.float32), 50)
    bad = p.raw.copy()
    bad[p.bytes_used - 16 * ((p.n_sel + 15) // 16)] = 0b10      # first payload word -> code 10
    with pytest.raises(RuntimeError, match="-5"):
        cref.unpack_sum([bad], 200)
    q = cref.pack(_gauss(250), np.zeros(250, np.float32), 50)
    with pytest.raises(RuntimeError, match="-4"):
        cref.unpack_sum([p.raw, q.raw], 200)


def test_pack_on_several_threads_gives_the_same_bytes():
    """The all-cores mode of the oracle (used only as a timed baseline) spreads pack()'s loops over
    threads; bins are independent and the scale's sum is exact, so nothing may change."""
    rng = np.random.default_rng(99)
    assert cref.get_threads() == 1
    try:
        for L_T, n, flags, factor in [(50, 100352, 0, 0.0), (500, 147456 + 3, 0, 0.0), (7, 30011, 1, 0.0),
                                      (5000, 123457, 0, 1.5), (64, 64 * 33 + 1, 0, 0.0), (50, 0, 0, 0.0)]:
            dW = rng.normal(0, 1e-3, n).astype(np.float32)
            r0 = rng.normal(0, 2e-3, n).astype(np.float32)
            cref.set_threads(1)
            r1 = r0.copy()
            one = cref.pack(dW, r1, L_T, flags=flags, factor=factor)
            cref.set_threads(5)
            r5 = r0.copy()
            many = cref.pack(dW, r5, L_T, flags=flags, factor=factor)
            assert np.array_equal(one.raw, many.raw), (L_T, n)
            assert np.array_equal(r1.view(np.uint32), r5.view(np.uint32)), (L_T, n)
    finally:
        cref.set_threads(1)

