"""Parity of adacomp_compress_scaled (the selection's scale-factor, Section 2.4) with the oracle."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import GpuLayer, assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu


def _compress_scaled(layer, dW, factor):
    layer.grad[:layer.n].copy_(torch.from_numpy(np.ascontiguousarray(dW)))
    layer.packed.fill_(0xAB)
    B.adacomp_compress_scaled(layer.grad, layer.residue, layer.n, layer.L_T, layer.packed, layer.count, factor)
    torch.cuda.synchronize()
    n_sel, used = (int(v) for v in layer.count.cpu())
    return layer.packed[:used].cpu().numpy(), n_sel


@pytest.mark.parametrize("factor", [1.0, 1.5, 2.0, 3.0])
@pytest.mark.parametrize("L_T,n", [(50, 100352), (500, 147456 + 3), (50, 4000 * 30), (7, 1000), (64, 70000),
                                   (1001, 50001), (500, 77), (100, 4000 * 9 + 7), (250, 4000 * 5 + 249), (1000, 4000 * 7 + 1)])
def test_scaled_selection_matches_oracle_over_three_steps(L_T, n, factor):
    rng = np.random.default_rng(int(1000 * factor) + L_T + n)
    r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
    layer = GpuLayer(n, L_T, r_cpu)
    sent = []
    for step in range(3):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        want = cref.pack(dW, r_cpu, L_T, factor=factor)
        raw, n_sel = _compress_scaled(layer, dW, factor)
        assert_stream_equal(raw, want, f"factor {factor} L_T={L_T} n={n} step {step}")
        assert n_sel == want.n_sel
        assert_f32_bits_equal(layer.residue_host(), r_cpu, f"residue step {step}")
        sent.append(n_sel)
    assert B.adacomp_device_status() == 0


def test_more_is_sent_as_the_factor_grows_and_factor_one_sends_one_per_bin():
    rng = np.random.default_rng(9)
    n, L_T = 4000 * 50, 50
    r = rng.normal(0, 3e-3, n).astype(np.float32)
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    counts = []
    for factor in (1.0, 1.5, 2.0, 3.0):
        layer = GpuLayer(n, L_T, r)
        _, n_sel = _compress_scaled(layer, dW, factor)
        counts.append(n_sel)
    assert counts[0] == n // L_T                     # continuous data: no ties, one maximum per bin
    assert counts == sorted(counts) and counts[-1] > counts[0]


def test_streams_made_with_a_factor_decode_like_any_other():
    rng = np.random.default_rng(10)
    n, L_T = 4000 * 7 + 5, 500
    streams = []
    for l in range(3):
        r = rng.normal(0, 2e-3, n).astype(np.float32)
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        raw, _ = _compress_scaled(GpuLayer(n, L_T, r), dW, 1.5)
        streams.append(raw)
    dev = torch.device("cuda:0")
    bufs = [torch.from_numpy(s.copy()).to(dev) for s in streams]
    dst = torch.empty(n, dtype=torch.float32, device=dev)
    B.adacomp_decompress_accumulate(bufs, 3, dst)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum(streams, n), "decode of scaled streams")
    assert B.adacomp_device_status() == 0


def test_bad_factor_is_refused_on_the_host():
    layer = GpuLayer(100, 50)
    for bad in (0.0, -2.0, float("inf"), float("nan")):
        with pytest.raises(RuntimeError):
            B.adacomp_compress_scaled(layer.grad, layer.residue, 100, 50, layer.packed, layer.count, bad)
