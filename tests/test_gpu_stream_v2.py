"""Stream version 2 on the GPU (first-of-bin flags instead of a count per bin; Section "Experiment Results" counts
the words alone): adacomp_stream_to_v2 of a stream packed by the library must be the oracle's version-2 bytes, and
adacomp_stream_from_v2 must give back the version-1 stream, which then decodes to the oracle's sum."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import GpuLayer, assert_f32_bits_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def same_bytes(got, want, what):
    assert got.size == want.size, f"{what}: {got.size} bytes, oracle {want.size}"
    if not np.array_equal(got, want):
        at = int(np.flatnonzero(got != want)[0])
        raise AssertionError(f"{what}: first differing byte at {at} (gpu {got[at]:#x}, oracle {want[at]:#x}) of {want.size}")


@pytest.mark.parametrize("L_T,n", [(50, 100352), (50, 4000 * 300 + 1234), (500, 147456 + 3), (63, 70000), (64, 70000), (65, 70001),
                                   (7, 30011), (1, 4001), (1001, 50001), (5000, 123457), (16383, 16383 * 5 + 2), (50, 0), (4, 3),
                                   (100, 4000 * 9 + 50), (41, 3936 * 7 + 5)])
def test_conversions_match_the_oracle(L_T, n):
    rng = np.random.default_rng(L_T * 3 + n)
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    if n > 9000:
        dW[3000:3000 + 4 * L_T + 777] = 0            # bins that send nothing: markers, also across a tile boundary
        dW[n - 2 * L_T:] = 0
    want1 = cref.pack(dW, np.zeros(n, np.float32), L_T)
    layer = GpuLayer(n, L_T)
    raw1, _, _ = layer.compress(dW)
    assert np.array_equal(raw1, want1.raw)
    want2 = cref.to_v2(want1.raw)
    v2 = torch.full((B.adacomp_v2_capacity(n, L_T),), 0xAB, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_device_status_reset()
    B.adacomp_stream_to_v2(layer.packed, v2, cnt, n, L_T)
    torch.cuda.synchronize()
    words, used = (int(x) for x in cnt.cpu())
    assert used == want2.size and words == want1.n_sel + int(np.count_nonzero(want1.bin_cnt == 0))
    same_bytes(v2[:used].cpu().numpy(), want2, f"to_v2 L_T={L_T} n={n}")
    back = torch.full((B.adacomp_packed_capacity(n, L_T),), 0xCD, dtype=torch.uint8, device=DEV)
    B.adacomp_stream_from_v2(v2, back, n, L_T)
    torch.cuda.synchronize()
    same_bytes(back[:want1.bytes_used].cpu().numpy(), want1.raw, f"from_v2 L_T={L_T} n={n}")
    assert B.adacomp_device_status() == 0
    if n:
        dst = torch.empty(n, device=DEV)
        B.adacomp_decompress_accumulate_ex([back], 1, dst, n, L_T)
        torch.cuda.synchronize()
        assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum_v2([want2], n), "decode of the converted stream")


def test_wrong_shape_and_malformed_streams_are_flagged_without_faulting():
    n, L_T = 4000 * 40 + 9, 50
    rng = np.random.default_rng(1)
    want1 = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L_T)
    v1 = torch.from_numpy(want1.raw.copy()).to(DEV)
    v2 = torch.zeros(B.adacomp_v2_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_device_status_reset()
    B.adacomp_stream_to_v2(v1, torch.zeros(B.adacomp_v2_capacity(n + 50, L_T), dtype=torch.uint8, device=DEV), cnt, n + 50, L_T)
    assert B.adacomp_device_status() == B.ADACOMP_DEV_HEADER_MISMATCH and int(cnt[1]) == 0
    B.adacomp_device_status_reset()
    # a version-2 stream whose first word lost its flag, and one with an inflated directory entry
    good2 = cref.to_v2(want1.raw)
    pay = (64 + 8 * (want1.n_tiles + 1) + 15) & ~15
    for what, edit in (("no bin open", lambda b: b.__setitem__(pay, b[pay] & 0xFD)),
                       ("directory past the words", lambda b: b.__setitem__(slice(64 + 8, 64 + 16), np.frombuffer((10 ** 9).to_bytes(8, "little"), np.uint8)))):
        bad = good2.copy()
        edit(bad)
        out = torch.zeros(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
        B.adacomp_stream_from_v2(torch.from_numpy(bad).to(DEV), out, n, L_T)
        torch.cuda.synchronize()
        assert B.adacomp_device_status() & B.ADACOMP_DEV_BAD_STREAM, what
        B.adacomp_device_status_reset()
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_stream_to_v2(v1, v2[:1024], cnt, n, L_T)       # output too small
    assert e.value.code == -5
    assert B.adacomp_v2_capacity(100, 16384) == 0
