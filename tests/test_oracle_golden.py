"""The oracle against hand-worked bins and the word-format examples (CPU only)."""
import numpy as np
import pytest

from oracle import cref, scalar
from tests.helpers import f32, read_sections

SEC = read_sections("worked_bins.txt")
L_T = int(SEC[""]["L_T"][0])
N = int(SEC[""]["n"][0])


def _hex(vals):
    return np.array([int(v, 16) for v in vals], dtype=np.uint8)


def test_step1_default_reading():
    s = SEC["step1"]
    residue = f32(s["residue"]).copy()
    p = cref.pack(f32(s["dW"]), residue, L_T, want_gmax=True)
    assert p.n == N and p.w == 1 and p.n_bins == 4
    np.testing.assert_array_equal(p.g_max, f32(s["g_max"]))
    assert p.scale == np.float32(float(s["scale"][0]))
    np.testing.assert_array_equal(p.bin_cnt, [int(v) for v in s["bin_cnt"]])
    np.testing.assert_array_equal(p.words, _hex(s["payload_hex"]))
    np.testing.assert_array_equal(residue, f32(s["residue_out"]))
    assert p.n_sel == 7


def test_step1_intermediate_G_and_H_match_the_fixture():
    # the fixture's G and H rows are what Algorithm 2's first two statements give
    s = SEC["step1"]
    G = f32(s["residue"]) + f32(s["dW"])
    np.testing.assert_array_equal(G, f32(s["G"]))
    np.testing.assert_array_equal(G + f32(s["dW"]), f32(s["H"]))
    s2 = SEC["step2"]
    G2 = f32(s["residue_out"]) + f32(s2["dW"])
    np.testing.assert_array_equal(G2, f32(s2["G"]))
    np.testing.assert_array_equal(G2 + f32(s2["dW"]), f32(s2["H"]))


def test_step1_literal_algorithm2():
    s = SEC["step1"]
    residue = f32(s["residue"]).copy()
    p = cref.pack(f32(s["dW"]), residue, L_T, flags=1)
    np.testing.assert_array_equal(p.bin_cnt, [int(v) for v in s["literal_bin_cnt"]])
    np.testing.assert_array_equal(p.words, _hex(s["literal_payload_hex"]))
    np.testing.assert_array_equal(residue, f32(s["literal_residue_out"]))
    assert p.scale == np.float32(float(s["scale"][0]))   # same g_max vector, same scale


def test_step2_carried_residue_and_decode_sum():
    s1, s2 = SEC["step1"], SEC["step2"]
    residue = f32(s1["residue"]).copy()
    p1 = cref.pack(f32(s1["dW"]), residue, L_T)
    p2 = cref.pack(f32(s2["dW"]), residue, L_T, want_gmax=True)
    np.testing.assert_array_equal(p2.g_max, f32(s2["g_max"]))
    assert p2.scale == np.float32(float(s2["scale"][0]))
    np.testing.assert_array_equal(p2.bin_cnt, [int(v) for v in s2["bin_cnt"]])
    np.testing.assert_array_equal(p2.words, _hex(s2["payload_hex"]))
    np.testing.assert_array_equal(residue, f32(s2["residue_out"]))
    dst = cref.unpack_sum([p1.raw, p2.raw], N)
    np.testing.assert_array_equal(dst, f32(SEC["decode_sum"]["dst"]))


def test_scalar_oracle_reproduces_the_fixture_too():
    s1, s2 = SEC["step1"], SEC["step2"]
    cnt, words, scale, res, gmax = scalar.pack(f32(s1["dW"]), f32(s1["residue"]), L_T)
    assert cnt == [int(v) for v in s1["bin_cnt"]]
    assert words == [int(v, 16) for v in s1["payload_hex"]]
    assert float(scale) == float(s1["scale"][0])
    np.testing.assert_array_equal(np.array(res, dtype=np.float32), f32(s1["residue_out"]))
    cnt2, words2, scale2, res2, _ = scalar.pack(f32(s2["dW"]), res, L_T)
    assert cnt2 == [int(v) for v in s2["bin_cnt"]]
    assert words2 == [int(v, 16) for v in s2["payload_hex"]]
    dst = scalar.unpack_sum([(cnt, words, scale), (cnt2, words2, scale2)], N, L_T)
    np.testing.assert_array_equal(np.array(dst, dtype=np.float32), f32(SEC["decode_sum"]["dst"]))


def test_stream_directory_and_header_of_the_fixture():
    s = SEC["step1"]
    residue = f32(s["residue"]).copy()
    p = cref.pack(f32(s["dW"]), residue, L_T)
    # L_T = 4 -> 4 * (1000 // 4) = 1000 bins per directory tile -> one tile
    assert p.tile_bins == 1000 and p.n_tiles == 1
    np.testing.assert_array_equal(p.tile_off, [0, 7])
    # header 64 | tile_off 2*8 = 16 | bin_cnt 4 -> 16 | payload 7 -> 16
    assert p.bytes_used == 64 + 16 + 16 + 16
    assert p.raw[64 + 16 + 16 + 7:].tolist() == [0] * 9     # zero padding to 16 bytes
    ref = scalar.to_stream(N, L_T, p.bin_cnt.tolist(), p.words.tolist(), p.scale)
    assert p.raw.tobytes() == ref


@pytest.mark.parametrize("line", open(__file__.replace("test_oracle_golden.py", "golden/word_format.txt")).read().splitlines())
def test_word_format_examples(line):
    line = line.split("#", 1)[0].split()
    if not line:
        return
    lt, idx, sign, word = int(line[0]), int(line[1]), line[2], int(line[3], 16)
    # one bin of L_T elements; only `idx` is non-zero, so it is the bin maximum and is sent
    dW = np.zeros(lt, dtype=np.float32)
    dW[idx] = 1.0 if sign == "+" else -1.0
    residue = np.zeros(lt, dtype=np.float32)
    p = cref.pack(dW, residue, lt)
    assert p.w == (1 if lt <= 64 else 2)
    assert p.n_sel == 1 and int(p.words[0]) == word
    assert p.scale == np.float32(1.0) and residue[idx] == 0.0
    if p.w == 2:   # little-endian on the wire
        at = p.bytes_used - 16
        assert p.raw[at] == (word & 0xFF) and p.raw[at + 1] == (word >> 8)
