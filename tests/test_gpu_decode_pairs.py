"""unpack()-and-sum for tensors of 256 tiles and more whose tiles have 80 bins of 8-bit words (L_T = 48, 49, 50):
the decoder takes their tiles in pairs, a lane per bin.  Every case is compared bit for bit with the oracle's
ordered sum (Algorithm 1, unpack() and the sum half of averageGradients()); the streams are the oracle's own,
so a failure here is the decoder's."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal

pytestmark = pytest.mark.gpu


def oracle_streams(L_T, n, k, rng, dense_learner=None):
    packs = []
    for l in range(k):
        r = rng.normal(0, 2e-3, n).astype(np.float32)
        dW = rng.normal(0, 1e-3 * (1 + l % 3), n).astype(np.float32)
        if l == dense_learner:
            # every element of a stretch ties for its bin's maximum: all of them are sent, so this learner's
            # words of those tiles overflow its staging region and are read from global memory
            r[:] = 0
            lo, hi = 4000 * 7, 4000 * 23
            dW[lo:hi] = np.where(rng.random(hi - lo) < 0.5, -1.0, 1.0).astype(np.float32) * np.float32(0.25)
        packs.append(cref.pack(dW, r, L_T))
    return packs


def decode(raws, n, L_T=None):
    dev = torch.device("cuda:0")
    bufs = [torch.from_numpy(r.copy()).to(dev) for r in raws]
    dst = torch.full((n,), float("nan"), dtype=torch.float32, device=dev)
    if L_T is None:
        B.adacomp_decompress_accumulate(bufs, len(bufs), dst)
    else:
        B.adacomp_decompress_accumulate_ex(bufs, len(bufs), dst, n, L_T)
    torch.cuda.synchronize()
    return dst.cpu().numpy()


@pytest.mark.parametrize("L_T,n,k", [
    (50, 4000 * 300, 3),               # an even number of whole tiles
    (50, 4000 * 301 + 1234, 4),        # the last pair is one tile and a ragged one
    (50, 4000 * 256 + 1, 1),           # the smallest tensor that goes in pairs; its last tile is one element
    (49, 3920 * 257 + 17, 5),
    (48, 3840 * 260 + 3800, 2),
    (50, 4000 * 400 + 77, 9),          # more learners than one group of four
    (50, 4000 * 270 + 50, 40),         # more learners than fit a slot: several rounds per pair
])
def test_pairs_of_tiles_match_the_oracle(L_T, n, k):
    rng = np.random.default_rng(L_T * 1000 + k)
    packs = oracle_streams(L_T, n, k, rng)
    raws = [p.raw for p in packs]
    want = cref.unpack_sum(raws, n)
    B.adacomp_device_status_reset()
    assert_f32_bits_equal(decode(raws, n, L_T), want, f"pairs, shape given: L_T={L_T} n={n} k={k}")
    assert_f32_bits_equal(decode(raws, n), want, f"pairs, shape from the headers: L_T={L_T} n={n} k={k}")
    assert B.adacomp_device_status() == 0


def test_pairs_with_a_learner_that_overflows_its_staging_region():
    L_T, n, k = 50, 4000 * 280 + 9, 4
    rng = np.random.default_rng(5)
    packs = oracle_streams(L_T, n, k, rng, dense_learner=2)
    raws = [p.raw for p in packs]
    B.adacomp_device_status_reset()
    assert_f32_bits_equal(decode(raws, n, L_T), cref.unpack_sum(raws, n), "pairs, dense learner")
    assert B.adacomp_device_status() == 0


def test_pairs_flag_malformed_words_and_counts():
    """As for single tiles: a word with the reserved code or an index past its bin is skipped and reported;
    a bin count that disagrees with the directory is reported and costs at most the pair of tiles it is in."""
    L_T, n = 50, 4000 * 300 + 77
    rng = np.random.default_rng(11)
    good, a = oracle_streams(L_T, n, 2, rng)
    pos, codes = a.positions_and_codes()
    bin_cnt_at = (64 + 8 * (a.n_tiles + 1) + 15) & ~15
    payload_at = (bin_cnt_at + a.n_bins + 15) & ~15
    alone = cref.unpack_sum([good.raw], n)
    both = cref.unpack_sum([good.raw, a.raw], n)
    for what, word_of, status in (("reserved code", lambda j: (int(a.words[j]) & 0xFC) | 0b10, B.ADACOMP_DEV_RESERVED_CODE),
                                  ("index past the bin", lambda j: (L_T << 2) | int(codes[j]), B.ADACOMP_DEV_BAD_STREAM)):
        j = a.n_sel // 2 + 3
        bad = a.raw.copy()
        bad[payload_at + j] = word_of(j)
        B.adacomp_device_status_reset()
        got = decode([good.raw, bad], n, L_T)
        assert B.adacomp_device_status() == status, what
        want = both.copy()
        want[pos[j]] = alone[pos[j]]                           # the bad word is skipped
        assert_f32_bits_equal(got, want, what)
    b = a.n_bins // 2
    bad = a.raw.copy()
    bad[bin_cnt_at + b] = int(a.bin_cnt[b]) + 1
    B.adacomp_device_status_reset()
    got = decode([good.raw, bad], n, L_T)
    assert B.adacomp_device_status() & B.ADACOMP_DEV_BAD_STREAM
    reach = 2 * 4000 + L_T
    lo, hi = max(0, b * L_T - reach), min(n, (b + 1) * L_T + reach)
    assert_f32_bits_equal(got[:lo], both[:lo], "inflated count, before")
    assert_f32_bits_equal(got[hi:], both[hi:], "inflated count, after")
    assert np.all(np.isfinite(got))
    B.adacomp_device_status_reset()
    assert B.adacomp_device_status() == 0
