"""Parity of adacomp_compress_bf16 (bfloat16 gradient, widened exactly on load) with the oracle."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import GpuLayer, assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu


def _bf16_bits(rng, n, sigma=1e-3):
    g = rng.normal(0, sigma, n).astype(np.float32)
    return (g.view(np.uint32) >> 16).astype(np.uint16)


def _compress(layer, bits):
    dev = layer.residue.device
    g = torch.from_numpy(bits.view(np.int16).copy()).to(dev).view(torch.bfloat16)
    if g.numel() < 8:                                    # keep the allocation 16-byte sized
        g = torch.cat([g, torch.zeros(8 - g.numel(), dtype=torch.bfloat16, device=dev)])
    layer.packed.fill_(0xAB)
    B.adacomp_compress_bf16(g, layer.residue, layer.n, layer.L_T, layer.packed, layer.count)
    torch.cuda.synchronize()
    n_sel, used = (int(v) for v in layer.count.cpu())
    return layer.packed[:used].cpu().numpy(), n_sel


@pytest.mark.parametrize("L_T,n", [(50, 100352), (50, 4000 * 33), (50, 4000 * 3 + 1999), (500, 147456 + 3), (500, 4000 * 21),
                                   (7, 1000), (64, 70000), (65, 70001), (1001, 50001), (500, 5), (50, 0),
                                   (100, 4000 * 17 + 50), (125, 4000 * 8 + 124), (200, 4000 * 11), (250, 4000 * 6 + 1),
                                   (1000, 4000 * 9 + 999)])
def test_bf16_gradient_matches_oracle_over_three_steps(L_T, n):
    rng = np.random.default_rng(7000 + L_T + n)
    r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
    layer = GpuLayer(n, L_T, r_cpu)
    for step in range(3):
        bits = _bf16_bits(rng, n)
        want = cref.pack_bf16(bits, r_cpu, L_T)
        raw, n_sel = _compress(layer, bits)
        assert_stream_equal(raw, want, f"bf16 L_T={L_T} n={n} step {step}")
        assert n_sel == want.n_sel
        if n:
            assert_f32_bits_equal(layer.residue_host(), r_cpu, f"residue step {step}")
    assert B.adacomp_device_status() == 0


def test_special_values_widen_exactly():
    """Signed zeros, subnormal bfloat16 values and the largest finite ones go through unchanged."""
    n, L_T = 4000 * 2, 50
    bits = np.zeros(n, np.uint16)
    bits[0::7] = 0x8000          # -0.0
    bits[1::7] = 0x0001          # smallest subnormal
    bits[2::7] = 0x807f          # largest negative subnormal
    bits[3::7] = 0x3f80          # 1.0
    bits[4::7] = 0xbf80          # -1.0
    bits[5::50] = 0x7f7f         # largest finite
    r_cpu = np.zeros(n, np.float32)
    layer = GpuLayer(n, L_T, r_cpu)
    want = cref.pack_bf16(bits, r_cpu, L_T)
    raw, _ = _compress(layer, bits)
    assert_stream_equal(raw, want, "special values")
    assert_f32_bits_equal(layer.residue_host(), r_cpu, "residue")
    B.adacomp_device_status_reset()
