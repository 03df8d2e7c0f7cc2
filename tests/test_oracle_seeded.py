"""The oracle on the seeded synthetic workloads: cross-check values recorded from
two independent earlier implementations, and the compression-rate statistics the
paper reports (about 5 sent per bin, ~40x at L_T = 50, towards ~200x at L_T = 500;
Section "Experiment Results").  CPU only."""
import zlib

import numpy as np
import pytest

from oracle import cref
from paper_1712_02679_b200 import synth
from tests.helpers import crc_counts_words, read_rows


def test_generator_first_values_and_sigmas():
    for step, dw0, *_ in read_rows("seeded_pins.txt", "cfg1"):
        dW = synth.make_dw(1, 0, 0, int(step), 100352, heavy=False, sigma=1e-3)
        assert dW[0] == np.float32(float(dw0))
    seen = {}
    for tensor, n, L_T, sigma, *_ in read_rows("seeded_pins.txt", "cfg2"):
        seen[int(tensor)] = (int(n), int(L_T), float(sigma))
    specs = synth.config2_tensors()
    for t, (n, L_T, sigma) in seen.items():
        assert (specs[t].n, specs[t].L_T) == (n, L_T)
        assert synth.sigma_for(2, t) == pytest.approx(sigma, rel=1e-8)


def test_config1_ten_carried_steps():
    n, L_T = 100352, 50
    residue = np.zeros(n, np.float32)
    rows = read_rows("seeded_pins.txt", "cfg1")
    assert len(rows) == 10
    for step, _dw0, n_sel, scale_bits, crc, tail in rows:
        dW = synth.make_dw(1, 0, 0, int(step), n, heavy=False, sigma=1e-3)
        p = cref.pack(dW, residue, L_T)
        assert p.n_sel == int(n_sel)
        assert p.scale_bits == int(scale_bits, 16)
        assert crc_counts_words(p.bin_cnt, p.words) == int(crc, 16)
        assert p.n_bins == 2008 and int(p.bin_cnt[-1]) == int(tail)


def test_config2_twenty_carried_steps_heavy_tailed():
    want = {}
    for tensor, n, L_T, sigma, step, n_sel, scale_bits, crc in read_rows("seeded_pins.txt", "cfg2"):
        want[(int(tensor), int(step))] = (int(n_sel), int(scale_bits, 16), int(crc, 16))
    for t, spec in enumerate(synth.config2_tensors()):
        residue = np.zeros(spec.n, np.float32)
        for step in range(20):
            dW = synth.make_dw(2, 0, t, step, spec.n, heavy=True)
            p = cref.pack(dW, residue, spec.L_T)
            if (t, step) in want:
                assert (p.n_sel, p.scale_bits, crc_counts_words(p.bin_cnt, p.words)) == want[(t, step)], (t, step)


def test_decode_sum_of_four_learners():
    spec = synth.config2_tensors()[7]
    streams = []
    for learner, n_sel, scale_bits in read_rows("seeded_pins.txt", "decode"):
        dW = synth.make_dw(2, int(learner), 7, 0, spec.n, heavy=True)
        p = cref.pack(dW, np.zeros(spec.n, np.float32), spec.L_T)
        assert (p.n_sel, p.scale_bits) == (int(n_sel), int(scale_bits, 16))
        streams.append(p.raw)
    dst = cref.unpack_sum(streams, spec.n)
    (nonzero, crc, total), = read_rows("seeded_pins.txt", "decode_dst")
    assert int(np.count_nonzero(dst)) == int(nonzero)
    assert zlib.crc32(dst.astype("<f4").tobytes()) & 0xFFFFFFFF == int(crc, 16)
    assert float(dst.astype(np.float64).sum()) == pytest.approx(float(total), rel=1e-8)


# --------------------------------------------------------------------------
# statistics the paper prints (a +-10 % band, not an equality)
# --------------------------------------------------------------------------

def _rate(p):
    return 32.0 * p.n / (8.0 * p.w * p.n_sel)


def test_rate_reaches_the_papers_40x_at_bin_length_50():
    # "typically selects only up to 5 elements within each bin" -> 32*50/(8*5) = 40x
    n = 1_000_000
    rng = np.random.default_rng(11)
    residue = np.zeros(n, np.float32)
    per_bin = []
    for step in range(24):
        p = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), residue, 50)
        per_bin.append(p.n_sel / p.n_bins)
    # first step: fraction of a Gaussian bin of 50 with 2|x| >= max|x| (scale free)
    assert per_bin[0] / 50 == pytest.approx(0.2213, rel=0.02)
    assert per_bin[0] > per_bin[5] > per_bin[9] >= per_bin[23] - 0.05   # more is sent early
    assert per_bin[23] == pytest.approx(5.0, rel=0.05)
    assert _rate(p) == pytest.approx(40.0, rel=0.10)


def test_rate_climbs_towards_the_papers_200x_at_bin_length_500():
    n = 1_000_000
    rng = np.random.default_rng(12)
    residue = np.zeros(n, np.float32)
    rates = []
    for step in range(40):
        p = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), residue, 500)
        rates.append(_rate(p))
        if step == 0:
            assert p.n_sel / n == pytest.approx(0.1104, rel=0.02)
    assert rates[0] == pytest.approx(18.0, rel=0.1)
    assert rates[5] == pytest.approx(66.0, rel=0.1)
    assert rates[19] == pytest.approx(124.0, rel=0.1)
    assert rates[39] == pytest.approx(151.0, rel=0.1)
    assert all(b > a * 0.95 for a, b in zip(rates, rates[1:]))   # climbs, up to noise
    # 16-bit words, about 5-6 per bin of 500 in the steady state is the paper's ~200x
    assert 32 * 500 / (16 * 5) == 200


def test_heavy_tailed_inputs_compress_harder():
    n = 500_000
    for L_T, lo, hi in [(50, 75, 110), (500, 380, 520)]:
        rng = np.random.default_rng(L_T)
        residue = np.zeros(n, np.float32)
        for _ in range(4):
            p = cref.pack(synth.heavy_dw(n, 1e-3, rng), residue, L_T)
        assert lo <= _rate(p) <= hi, (L_T, _rate(p))
