"""Pins of stream version 2 (bins told apart by a first-of-bin flag in the words instead of a count per bin: the
paper's rate figures, Section "Experiment Results", count the words alone).  Hand-worked bytes, the round trip
with version 1, a decoder that reads the flags directly, brute force against the scalar restatement, and the
size formula that gives the wire rate."""
import struct

import numpy as np
import pytest

from oracle import cref, scalar


def test_hand_worked_stream():
    """The worked example of the main fixture (L_T = 4, n = 14): bin 0 sends places 0 (+), 1 (-), 3 (+); bin 1
    places 0 (+), 3 (+); bin 2 nothing; bin 3 places 0 (+), 1 (+).  Version 1 words 01 07 0D | 01 0D | | 01 05
    with counts 3 2 0 2; version 2: the first word of a bin gets bit 1, the sign moves to bit 0, bin 2 becomes the
    marker (index 4, flag set) = 0x12."""
    residue = np.array([0, 0, 0, 0, 1, 0, 0, .5, .25, 0, 0, 0, 1, .25], np.float32)
    dW = np.array([.5, -.25, .125, .25, -.25, .125, -.125, .25, -.25, 0, 0, 0, -.75, .25], np.float32)
    v1 = cref.pack(dW, residue.copy(), 4).raw
    v2 = cref.to_v2(v1)
    head = struct.pack("<IHBBIIQQQQIIQ", 0x31434441, 2, 1, 0, 4, 1000, 14, 4, 1, 7, 0x3EE00000, 1, 96)
    directory = struct.pack("<2Q", 0, 8)
    words = bytes([0x02, 0x05, 0x0C, 0x02, 0x0C, 0x12, 0x02, 0x04]) + bytes(8)
    assert bytes(v2) == head + directory + words
    assert bytes(cref.from_v2(v2)) == bytes(v1)
    want = np.array([.4375, -.4375, 0, .4375, .4375, 0, 0, .4375, 0, 0, 0, 0, .4375, .4375], np.float32)
    assert np.array_equal(cref.unpack_sum_v2([v2], 14), want)


@pytest.mark.parametrize("L_T,n", [(50, 100352), (500, 147456 + 3), (63, 70000), (64, 70000), (65, 70001), (7, 30011),
                                   (1001, 50001), (5000, 123457), (16383, 16383 * 5 + 2), (50, 0), (4, 3)])
def test_round_trip_sum_and_size(L_T, n):
    rng = np.random.default_rng(L_T + n)
    raws1, raws2 = [], []
    for l in range(3):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        if n > 4000:
            dW[1000 * l:1000 * l + 2200] = 0        # a stretch of bins that send nothing: markers
        p = cref.pack(dW, np.zeros(n, np.float32), L_T)
        v2 = cref.to_v2(p.raw)
        assert np.array_equal(cref.from_v2(v2), p.raw)
        # size: header, directory, one word per sent element and one per empty bin, nothing else
        w2 = 1 if L_T <= 63 else 2
        n_empty = int(np.count_nonzero(p.bin_cnt == 0))
        r16 = lambda x: (x + 15) & ~15
        assert v2.size == r16(64 + 8 * (p.n_tiles + 1)) + r16(w2 * (p.n_sel + n_empty))
        assert struct.unpack_from("<H", v2, 4)[0] == 2 and struct.unpack_from("<I", v2, 52)[0] == n_empty
        raws1.append(p.raw)
        raws2.append(v2)
    a, b = cref.unpack_sum(raws1, n), cref.unpack_sum_v2(raws2, n)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_wire_rate_closes_on_the_papers_accounting():
    """L_T = 50, Gaussian gradient, first step: version 1 pays a count byte per bin on top of the words, version 2
    only the directory (8 bytes per 4000 elements): within 2 % of 32 bits / 8 bits per sent element."""
    rng = np.random.default_rng(9)
    n = 4000 * 500
    p = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), 50)
    paper = 32.0 * n / (8.0 * p.n_sel)
    v1_rate, v2_rate = 4.0 * n / p.bytes_used, 4.0 * n / cref.to_v2(p.raw).size
    assert v1_rate < 0.93 * paper
    assert 0.98 * paper < v2_rate < paper


@pytest.mark.parametrize("L_T", [1, 2, 3, 4, 8])
def test_brute_force_against_the_scalar_restatement(L_T):
    rng = np.random.default_rng(200 + L_T)
    values = np.array([0, 0, .125, -.125, .25, -.25, .5, -.5, 1, -1], np.float32)
    for _ in range(400):
        n = int(rng.integers(1, 13))
        dW = rng.choice(values, n)
        res = rng.choice(values, n)
        p = cref.pack(dW, res.copy(), L_T)
        bc, words, scale, _, _ = scalar.pack(dW, res, L_T)
        assert bytes(cref.to_v2(p.raw)) == scalar.to_stream_v2(n, L_T, bc, words, scale)


def test_malformed_version_2_streams_are_refused():
    rng = np.random.default_rng(4)
    n = 5000
    v2 = cref.to_v2(cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), 50).raw)
    pay = (64 + 8 * 3 + 15) & ~15                      # two tiles: three directory entries
    bad = v2.copy()
    bad[pay] &= 0xFD                                   # the very first word loses its flag: no bin is open
    with pytest.raises(RuntimeError):
        cref.unpack_sum_v2([bad], n)
    with pytest.raises(RuntimeError):
        cref.from_v2(bad)
    bad = v2.copy()
    bad[pay + 1] = (51 << 2)                           # an index past the bin (and not the marker's)
    with pytest.raises(RuntimeError):
        cref.unpack_sum_v2([bad], n)
    with pytest.raises((RuntimeError, AssertionError)):
        cref.to_v2(v2)                                 # not a version-1 stream
