"""Pins of the oracle's scale-factor variant of the selection test (Section 2.4): a hand-worked
example, the factor-1 case against its closed form (only bin maxima are sent: the paper's "LS"), the
factor-2 case against the default on exactly representable data, and the C oracle against the
independent scalar restatement on random tiny inputs."""
import numpy as np
import pytest

from oracle import cref, scalar
from tests.helpers import f32, read_sections

SEC = read_sections("worked_bins.txt")
F = SEC["scale_factor"]


@pytest.mark.parametrize("factor", ["1", "1.5", "2", "8"])
def test_hand_worked_factors(factor):
    L_T, n = int(F["fL_T"][0]), int(F["fn"][0])
    residue = f32(F["residue"]).copy()
    p = cref.pack(f32(F["dW"]), residue, L_T, factor=float(factor), want_gmax=True)
    np.testing.assert_array_equal(p.g_max, f32(F["g_max"]))
    assert p.scale == np.float32(float(F["scale"][0]))
    np.testing.assert_array_equal(p.bin_cnt, [int(v) for v in F[f"f{factor}_bin_cnt"]])
    np.testing.assert_array_equal(p.words, [int(v, 16) for v in F[f"f{factor}_payload_hex"]])
    np.testing.assert_array_equal(residue, f32(F[f"f{factor}_residue_out"]))
    assert p.raw[7] == 2 and n == residue.size           # header flags: bit 1 = made with a factor
    # the scalar restatement agrees
    cnt, words, scale, res, _ = scalar.pack(f32(F["dW"]), f32(F["residue"]), L_T, factor=float(factor))
    assert cnt == [int(v) for v in F[f"f{factor}_bin_cnt"]]
    assert words == [int(v, 16) for v in F[f"f{factor}_payload_hex"]]
    np.testing.assert_array_equal(np.array(res, dtype=np.float32), f32(F[f"f{factor}_residue_out"]))


def test_factor_one_sends_exactly_the_bin_maxima():
    rng = np.random.default_rng(21)
    for L_T, n in ((50, 10007), (500, 20011), (7, 1000)):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        r = rng.normal(0, 3e-3, n).astype(np.float32)
        r[:L_T] = 0
        dW[:L_T] = 0                                   # a zero bin: nothing is sent from it
        res = r.copy()
        p = cref.pack(dW, res, L_T, factor=1.0)
        G = r + dW
        pad = (-n) % L_T
        absG = np.abs(np.concatenate([G, np.zeros(pad, np.float32)])).reshape(-1, L_T)
        gmax = absG.max(axis=1)
        want = ((absG == gmax[:, None]) & (gmax[:, None] > 0)).reshape(-1)[:n]
        pos, codes = p.positions_and_codes()
        got = np.zeros(n, bool)
        got[pos] = True
        np.testing.assert_array_equal(got, want)
        assert p.bin_cnt[0] == 0 and (p.bin_cnt[1:] >= 1).all()
        # residue: G - sign(G) * scale where sent, G elsewhere
        q = np.where(G < 0, -p.scale, p.scale).astype(np.float32)
        np.testing.assert_array_equal(res, np.where(want, G - q, G))


def test_factor_two_is_the_default_where_the_arithmetic_is_exact():
    s1 = SEC["step1"]
    L_T = int(SEC[""]["L_T"][0])
    r0, r2 = f32(s1["residue"]).copy(), f32(s1["residue"]).copy()
    p0 = cref.pack(f32(s1["dW"]), r0, L_T)
    p2 = cref.pack(f32(s1["dW"]), r2, L_T, factor=2.0)
    np.testing.assert_array_equal(p0.bin_cnt, p2.bin_cnt)
    np.testing.assert_array_equal(p0.words, p2.words)
    np.testing.assert_array_equal(r0, r2)
    assert p0.scale == p2.scale and p0.raw[7] == 0 and p2.raw[7] == 2


def test_c_oracle_and_scalar_restatement_agree_for_any_factor():
    rng = np.random.default_rng(22)
    vals = np.array([0, 2.0 ** -3, -2.0 ** -3, 0.3, -0.7, 1.0, -1.0, 1e-3], np.float32)
    for trial in range(300):
        n = int(rng.integers(1, 40))
        L_T = int(rng.choice([1, 2, 3, 4, 8, 50]))
        factor = float(rng.choice([1.0, 1.5, 2.0, 2.5, 3.0, 0.5]))
        dW = rng.choice(vals, n).astype(np.float32) * np.float32(rng.choice([1.0, 1e-3]))
        r = rng.choice(vals, n).astype(np.float32)
        res = r.copy()
        p = cref.pack(dW, res, L_T, factor=factor)
        cnt, words, scale, res2, _ = scalar.pack(dW, r, L_T, factor=factor)
        raw2 = scalar.to_stream(n, L_T, cnt, words, scale, factor=factor)
        assert bytes(p.raw) == raw2, (trial, n, L_T, factor)
        np.testing.assert_array_equal(res, np.array(res2, dtype=np.float32))


def test_bad_factor_is_refused():
    d = np.zeros(8, np.float32)
    for bad in (-1.0, float("inf"), float("nan")):
        with pytest.raises(RuntimeError):
            cref.pack(d, d.copy(), 4, factor=bad)
