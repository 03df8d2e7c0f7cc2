"""The second quantiser (scale = mean |G| of the sent elements; Section 2.5 leaves the quantisation function
open) on the GPU against the oracle, bit for bit: streams, scales and residues over carried steps, in eager and
lazy-scale mode, with 16-bit gradients and a factor, for every tile-pass form; the streams decode like any other."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal
from tests.test_gpu_formats import make_grad

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
Q = B.ADACOMP_QUANT_SENT_MEAN if hasattr(B, "ADACOMP_QUANT_SENT_MEAN") else 1


def run(L_T, n, grad_type=0, factor=0.0, lazy=False, flags=0, steps=3):
    rng = np.random.default_rng(L_T * 13 + n)
    r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
    res = torch.zeros(max(n, 4), device=DEV)
    res[:n] = torch.from_numpy(r_cpu)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    state = None
    if lazy:
        state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
        B.adacomp_lazy_state_init(state, n, L_T)
    raws = []
    for step in range(steps):
        g_dev, g_cpu = make_grad(rng, n, grad_type)
        want = cref.pack(g_cpu, r_cpu, L_T, flags=flags & 1, factor=factor, quantiser=1)
        B.adacomp_compress_opt(g_dev, res, n, L_T, packed, cnt, flags=flags, grad_type=grad_type, factor=factor,
                               lazy_state=state, quantiser=Q)
        torch.cuda.synchronize()
        what = f"L_T={L_T} n={n} step={step} lazy={lazy}"
        raw = packed[:int(cnt[1])].cpu().numpy()
        assert_stream_equal(raw, want, what)
        if not lazy:
            assert_f32_bits_equal(res[:n].cpu().numpy(), r_cpu, what + " residue")
        raws.append(raw)
    if lazy:
        B.adacomp_residue_flush(res, state, n, L_T)
        torch.cuda.synchronize()
        assert_f32_bits_equal(res[:n].cpu().numpy(), r_cpu, "residue after the flush")
    assert B.adacomp_device_status() == 0
    return raws


@pytest.mark.parametrize("L_T,n", [(50, 4000 * 9 + 1999), (500, 4000 * 7 + 3), (100, 4000 * 5 + 50), (250, 4000 * 3 + 1),
                                   (64, 3840 * 6 + 5), (41, 3936 * 5 + 40), (400, 3200 * 6 + 2), (3000, 3000 * 9 + 2),
                                   (7, 3001), (1001, 50001), (5000, 5000 * 7 + 11), (16384, 16384 * 3 + 5), (50, 0), (50, 7)])
def test_sent_mean_quantiser_eager(L_T, n):
    run(L_T, n)


@pytest.mark.parametrize("L_T,n", [(50, 4000 * 9 + 1999), (500, 4000 * 7 + 3), (64, 3840 * 6 + 5), (400, 3200 * 6 + 2)])
def test_sent_mean_quantiser_lazy_scale(L_T, n):
    run(L_T, n, lazy=True)


def test_sent_mean_quantiser_with_other_options_and_decode():
    run(50, 4000 * 11 + 7, grad_type=B.ADACOMP_GRAD_F16, factor=1.5, lazy=True, steps=4)
    run(500, 4000 * 5 + 499, grad_type=B.ADACOMP_GRAD_BF16, factor=3.0)
    run(50, 20011, flags=B.ADACOMP_FLAG_LITERAL)            # the literal flag takes the any-L_T kernel
    n, L_T = 4000 * 13 + 5, 50
    a = run(L_T, n, steps=1)[0]
    b = run(L_T, n + 0, factor=1.5, steps=1)[0]
    dev_bufs = [torch.from_numpy(r.copy()).to(DEV) for r in (a, b)]
    dst = torch.empty(n, device=DEV)
    B.adacomp_decompress_accumulate_ex(dev_bufs, 2, dst, n, L_T)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum([a, b], n), "decode of streams of the second quantiser")


def test_list_with_a_layer_of_the_second_quantiser():
    rng = np.random.default_rng(3)
    layers = []
    for L_T, n, q in [(50, 4000 * 6 + 1, 0), (500, 4000 * 4 + 9, 1), (50, 4000 * 3, 1), (100, 4000 * 2 + 50, 0)]:
        r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
        layers.append(dict(n=n, L_T=L_T, quantiser=q, r_cpu=r_cpu, residue=torch.from_numpy(r_cpu.copy()).to(DEV),
                           packed_out=torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV),
                           count_out=torch.zeros(2, dtype=torch.int64, device=DEV)))
    for step in range(2):
        wants = []
        for d in layers:
            d["grad"], g_cpu = make_grad(rng, d["n"], 0)
            wants.append(cref.pack(g_cpu, d["r_cpu"], d["L_T"], quantiser=d["quantiser"]))
        B.adacomp_compress_multi_opt(layers, len(layers))
        torch.cuda.synchronize()
        for i, (d, want) in enumerate(zip(layers, wants)):
            assert_stream_equal(d["packed_out"][:int(d["count_out"][1])].cpu().numpy(), want, f"layer {i} step {step}")
            assert_f32_bits_equal(d["residue"].cpu().numpy(), d["r_cpu"], f"layer {i} residue")
    assert B.adacomp_device_status() == 0
