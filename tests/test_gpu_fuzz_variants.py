"""Seeded fuzz over the entry points beside compress / decompress-accumulate: bfloat16 gradients, the
selection's scale-factor, and the fused optimizer steps, on random shapes against the oracle."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import GpuLayer, assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _shape(rng):
    L_T = int(rng.choice([int(rng.integers(1, 130)), int(rng.integers(130, 1100)), int(rng.integers(1100, 16385)),
                          50, 500, 50, 500]))
    n = int(rng.integers(1, 80000))
    return n, L_T


def test_fuzz_bf16_and_scaled_pack():
    rng = np.random.default_rng(777)
    for case in range(30):
        n, L_T = _shape(rng)
        sigma = 10.0 ** rng.uniform(-4, 0)
        r_cpu = rng.normal(0, sigma, n).astype(np.float32)
        layer = GpuLayer(n, L_T, r_cpu)
        for step in range(2):
            g = rng.normal(0, sigma, n).astype(np.float32)
            layer.packed.fill_(0xAB)
            if case % 2 == 0:
                bits = (g.view(np.uint32) >> 16).astype(np.uint16)
                want = cref.pack_bf16(bits, r_cpu, L_T)
                gb = torch.from_numpy(np.concatenate([bits, np.zeros(8, np.uint16)]).view(np.int16).copy()).to(DEV).view(torch.bfloat16)
                B.adacomp_compress_bf16(gb, layer.residue, n, L_T, layer.packed, layer.count)
            else:
                factor = float(rng.choice([1.0, 1.25, 1.5, 2.0, 2.5, 3.0]))
                want = cref.pack(g, r_cpu, L_T, factor=factor)
                layer.grad[:n].copy_(torch.from_numpy(g))
                B.adacomp_compress_scaled(layer.grad, layer.residue, n, L_T, layer.packed, layer.count, factor)
            torch.cuda.synchronize()
            used = int(layer.count[1])
            assert_stream_equal(layer.packed[:used].cpu().numpy(), want, f"case {case} step {step} n={n} L_T={L_T}")
            assert_f32_bits_equal(layer.residue_host(), r_cpu, f"residue case {case} step {step}")
    assert B.adacomp_device_status() == 0


def test_fuzz_fused_optimizer_steps():
    rng = np.random.default_rng(778)
    for case in range(24):
        n, L_T = _shape(rng)
        k = int(rng.integers(1, 9))
        streams = []
        for l in range(k):
            r = rng.normal(0, 2e-3, n).astype(np.float32)
            dW = rng.normal(0, 10.0 ** rng.uniform(-4, -2), n).astype(np.float32)
            streams.append(cref.pack(dW, r, L_T).raw)
        bufs = [torch.from_numpy(s.copy()).to(DEV) for s in streams]
        w = rng.normal(0, 1, n).astype(np.float32)
        m = rng.normal(0, 1e-3, n).astype(np.float32)
        v = (rng.normal(0, 1e-3, n).astype(np.float32)) ** 2
        pad = lambda a: torch.from_numpy(np.concatenate([a, np.zeros(8, np.float32)])).to(DEV)
        wd, md, vd = pad(w), pad(m), pad(v)
        if case % 2 == 0:
            lr, mu = float(10.0 ** rng.uniform(-3, 0)), float(rng.choice([0.0, 0.5, 0.9, 0.99]))
            want_w, want_m = cref.average_sgd(streams, n, w, m, lr, mu)
            B.adacomp_decompress_average_sgd(bufs, k, wd, md, n, L_T, lr, mu)
            want_v = v
        else:
            hy = dict(step_size=float(10.0 ** rng.uniform(-4, -1)), beta1=float(rng.choice([0.0, 0.9])),
                      beta2=float(rng.choice([0.5, 0.999])), eps=float(rng.choice([1e-8, 1e-3])))
            want_w, want_m, want_v = cref.average_adam(streams, n, w, m, v, **hy)
            B.adacomp_decompress_average_adam(bufs, k, wd, md, vd, n, L_T, hy["step_size"], hy["beta1"], hy["beta2"], hy["eps"])
        torch.cuda.synchronize()
        what = f"case {case} n={n} L_T={L_T} k={k}"
        assert_f32_bits_equal(md.cpu().numpy()[:n], want_m, "m " + what)
        assert_f32_bits_equal(vd.cpu().numpy()[:n], want_v, "v " + what)
        assert_f32_bits_equal(wd.cpu().numpy()[:n], want_w, "w " + what)
    assert B.adacomp_device_status() == 0


def test_fuzz_lazy_scale_pack():
    """Lazy-scale pack() on random shapes over the bin lengths it takes (41..1000 and the multiples of 4 up to
    4000): three carried steps equal the oracle's streams, a flush gives the oracle's residue, and the eager
    entry point carries on from there."""
    rng = np.random.default_rng(4242)
    for case in range(24):
        L_T = int(rng.integers(41, 1001)) if case % 3 else 4 * int(rng.integers(251, 1001))
        n = int(rng.integers(1, 120000))
        sigma = 10.0 ** rng.uniform(-4, 0)
        r_cpu = rng.normal(0, sigma, n).astype(np.float32)
        layer = GpuLayer(n, L_T, r_cpu)
        state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
        assert state.numel() > 0
        B.adacomp_lazy_state_init(state, n, L_T)
        for step in range(3):
            g = rng.normal(0, sigma, n).astype(np.float32)
            want = cref.pack(g, r_cpu, L_T)
            layer.grad[:n].copy_(torch.from_numpy(g))
            layer.packed.fill_(0xAB)
            B.adacomp_compress_lazy(layer.grad, layer.residue, state, n, L_T, layer.packed, layer.count)
            torch.cuda.synchronize()
            assert_stream_equal(layer.packed[:int(layer.count[1])].cpu().numpy(), want, f"case {case} step {step} n={n} L_T={L_T}")
        B.adacomp_residue_flush(layer.residue, state, n, L_T)
        assert_f32_bits_equal(layer.residue_host(), r_cpu, f"flushed residue case {case} n={n} L_T={L_T}")
        g = rng.normal(0, sigma, n).astype(np.float32)
        want = cref.pack(g, r_cpu, L_T)
        layer.grad[:n].copy_(torch.from_numpy(g))
        B.adacomp_compress(layer.grad, layer.residue, n, L_T, layer.packed, layer.count)
        torch.cuda.synchronize()
        assert_stream_equal(layer.packed[:int(layer.count[1])].cpu().numpy(), want, f"eager after flush, case {case}")
        assert_f32_bits_equal(layer.residue_host(), r_cpu, f"eager residue case {case}")
    assert B.adacomp_device_status() == 0
