"""pack() options in combination: 16-bit gradients (bfloat16, binary16), the selection's factor and lazy-scale
mode together, on the bin lengths of every tile-pass form (the seven specialised ones, the any-bin form, one-bin
tiles, the any-L_T kernel).  Every stream and every residue is compared bit for bit with the oracle, which
packs the exactly widened gradient (Algorithm 2; Section 2.4 for the factor)."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_grad(rng, n, grad_type, sigma=1e-3):
    """(device tensor for the library, float32 numpy array the oracle packs)."""
    g = rng.normal(0, sigma, n).astype(np.float32)
    pad = max(n, 8)
    if grad_type == B.ADACOMP_GRAD_F32:
        t = torch.zeros(pad, dtype=torch.float32, device=DEV)
        t[:n] = torch.from_numpy(g)
        return t, g
    if grad_type == B.ADACOMP_GRAD_BF16:
        bits = (g.view(np.uint32) >> 16).astype(np.uint16)
        wide = cref.bf16_to_f32(bits)
        t = torch.zeros(pad, dtype=torch.bfloat16, device=DEV)
        t[:n] = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
        return t, wide
    bits = g.astype(np.float16).view(np.uint16)
    wide = cref.f16_to_f32(bits)
    t = torch.zeros(pad, dtype=torch.float16, device=DEV)
    t[:n] = torch.from_numpy(bits.view(np.int16).copy()).view(torch.float16)
    return t, wide


def run(L_T, n, grad_type, factor, lazy, steps=3, seed=0):
    rng = np.random.default_rng(seed + L_T * 7 + n)
    r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
    res = torch.zeros(max(n, 4), device=DEV)
    res[:n] = torch.from_numpy(r_cpu)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    state = None
    if lazy:
        state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
        B.adacomp_lazy_state_init(state, n, L_T)
    for step in range(steps):
        g_dev, g_cpu = make_grad(rng, n, grad_type)
        want = cref.pack(g_cpu, r_cpu, L_T, factor=factor)
        packed.fill_(0xAB)
        B.adacomp_compress_opt(g_dev, res, n, L_T, packed, cnt, grad_type=grad_type, factor=factor, lazy_state=state)
        torch.cuda.synchronize()
        what = f"L_T={L_T} n={n} grad_type={grad_type} factor={factor} lazy={lazy} step={step}"
        assert int(cnt[0]) == want.n_sel, what
        assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), want, what)
        if not lazy:
            assert_f32_bits_equal(res[:n].cpu().numpy(), r_cpu, what + " residue")
    if lazy:
        B.adacomp_residue_flush(res, state, n, L_T)
        torch.cuda.synchronize()
        assert_f32_bits_equal(res[:n].cpu().numpy(), r_cpu, "residue after the flush")
    assert B.adacomp_device_status() == 0


SHAPES = [(50, 4000 * 9 + 1999), (500, 4000 * 7 + 3), (100, 4000 * 5 + 50), (125, 4000 * 4 + 124), (200, 4000 * 6),
          (250, 4000 * 3 + 1), (1000, 4000 * 5 + 999),            # the seven specialised bin lengths
          (64, 3840 * 6 + 5), (41, 3936 * 5 + 40), (400, 3200 * 6 + 2), (96, 3840 * 4 + 95),     # any-bin form, tiles of a multiple of 8 elements
          (3000, 3000 * 9 + 2)]                                     # one-bin tiles


@pytest.mark.parametrize("grad_type", [B.ADACOMP_GRAD_BF16, B.ADACOMP_GRAD_F16])
@pytest.mark.parametrize("L_T,n", SHAPES + [(7, 3001), (43, 3956 * 4 + 9), (1001, 50001), (5000, 5000 * 7 + 11), (50, 0), (50, 5)])
def test_sixteen_bit_gradients_eager(L_T, n, grad_type):
    run(L_T, n, grad_type, 0.0, False)


@pytest.mark.parametrize("grad_type", [B.ADACOMP_GRAD_BF16, B.ADACOMP_GRAD_F16])
@pytest.mark.parametrize("L_T,n", SHAPES)
def test_sixteen_bit_gradients_lazy_scale(L_T, n, grad_type):
    run(L_T, n, grad_type, 0.0, True)


@pytest.mark.parametrize("factor", [1.0, 1.5, 3.0])
@pytest.mark.parametrize("L_T,n", [(50, 4000 * 9 + 1999), (500, 4000 * 7 + 3), (64, 3840 * 6 + 5), (400, 3200 * 6 + 2)])
def test_factor_with_lazy_scale(L_T, n, factor):
    run(L_T, n, B.ADACOMP_GRAD_F32, factor, True)


def test_everything_at_once():
    run(50, 4000 * 21 + 7, B.ADACOMP_GRAD_F16, 1.5, True, steps=4)
    run(500, 4000 * 11 + 499, B.ADACOMP_GRAD_BF16, 3.0, True, steps=4)
    run(64, 3840 * 8 + 63, B.ADACOMP_GRAD_F16, 1.5, False)


def test_binary16_special_values_widen_exactly():
    """Signed zeros, subnormals, the largest finite value and values that binary32 holds exactly but
    bfloat16 would round."""
    n, L_T = 4000 * 2, 50
    bits = np.zeros(n, np.uint16)
    bits[0::7] = 0x8000          # -0.0
    bits[1::7] = 0x0001          # smallest subnormal, 2^-24
    bits[2::7] = 0x83ff          # largest negative subnormal
    bits[3::7] = 0x3c01          # 1 + 2^-10
    bits[4::7] = 0xbc00          # -1.0
    bits[5::50] = 0x7bff         # 65504
    r_cpu = np.zeros(n, np.float32)
    res = torch.zeros(n, device=DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    g = torch.from_numpy(bits.view(np.int16).copy()).to(DEV).view(torch.float16)
    want = cref.pack_f16(bits, r_cpu, L_T)
    B.adacomp_compress_f16(g, res, n, L_T, packed, cnt)
    torch.cuda.synchronize()
    assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), want, "special values")
    assert_f32_bits_equal(res.cpu().numpy(), r_cpu, "residue")
    B.adacomp_device_status_reset()


def test_unsupported_combinations_are_refused_on_the_host():
    n, L_T = 3956 * 4, 43            # tiles of 3956 elements: 16-bit tiles are not multiples of 16 bytes
    g = torch.zeros(n, dtype=torch.bfloat16, device=DEV)
    res = torch.zeros(n, device=DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
    B.adacomp_lazy_state_init(state, n, L_T)
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_compress_opt(g, res, n, L_T, packed, cnt, grad_type=B.ADACOMP_GRAD_BF16, lazy_state=state)
    assert e.value.code == -9
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_compress_opt(res, res, n, L_T, packed, cnt, grad_type=7)
    assert e.value.code == -6


def _list_case(rng, lazy):
    """A parameter list whose layers differ in bin length, gradient format and factor."""
    shapes = [(50, 4000 * 13 + 17, B.ADACOMP_GRAD_F32, 0.0), (500, 4000 * 6 + 499, B.ADACOMP_GRAD_BF16, 0.0),
              (50, 4000 * 3, B.ADACOMP_GRAD_F16, 1.5), (100, 4000 * 4 + 1, B.ADACOMP_GRAD_F32, 3.0),
              (64, 3840 * 5 + 9, B.ADACOMP_GRAD_F16, 0.0), (400, 3200 * 3 + 77, B.ADACOMP_GRAD_BF16, 1.5),
              (500, 864, B.ADACOMP_GRAD_F32, 0.0), (50, 10, B.ADACOMP_GRAD_F16, 0.0), (200, 4000 * 2 + 150, B.ADACOMP_GRAD_F16, 0.0)]
    if not lazy:
        shapes.append((43, 3956 * 3 + 5, B.ADACOMP_GRAD_BF16, 0.0))      # 16-bit tiles off the 16-byte boundaries: plain loads
    layers = []
    for L_T, n, gt, factor in shapes:
        r_cpu = rng.normal(0, 2e-3, n).astype(np.float32)
        res = torch.zeros(max(n, 4), device=DEV)
        res[:n] = torch.from_numpy(r_cpu)
        d = dict(n=n, L_T=L_T, grad_type=gt, factor=factor, residue=res, r_cpu=r_cpu,
                 packed_out=torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV),
                 count_out=torch.zeros(2, dtype=torch.int64, device=DEV))
        if lazy:
            d["lazy_state"] = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
            B.adacomp_lazy_state_init(d["lazy_state"], n, L_T)
        layers.append(d)
    return layers


@pytest.mark.parametrize("lazy", [False, True])
def test_parameter_list_with_per_layer_options(lazy):
    rng = np.random.default_rng(4242 + lazy)
    layers = _list_case(rng, lazy)
    for step in range(3):
        wants = []
        for d in layers:
            d["grad"], g_cpu = make_grad(rng, d["n"], d["grad_type"])
            wants.append(cref.pack(g_cpu, d["r_cpu"], d["L_T"], factor=d["factor"]))
            d["packed_out"].fill_(0xAB)
        B.adacomp_compress_multi_opt(layers, len(layers))
        torch.cuda.synchronize()
        for i, (d, want) in enumerate(zip(layers, wants)):
            what = f"layer {i} L_T={d['L_T']} n={d['n']} step {step} lazy={lazy}"
            assert int(d["count_out"][0]) == want.n_sel, what
            assert_stream_equal(d["packed_out"][:int(d["count_out"][1])].cpu().numpy(), want, what)
            if not lazy:
                assert_f32_bits_equal(d["residue"][:d["n"]].cpu().numpy(), d["r_cpu"], what + " residue")
    if lazy:
        for d in layers:
            B.adacomp_residue_flush(d["residue"], d["lazy_state"], d["n"], d["L_T"])
        torch.cuda.synchronize()
        for i, d in enumerate(layers):
            assert_f32_bits_equal(d["residue"][:d["n"]].cpu().numpy(), d["r_cpu"], f"layer {i} residue after the flush")
    assert B.adacomp_device_status() == 0


def test_parameter_list_where_only_some_layers_are_lazy():
    rng = np.random.default_rng(77)
    layers = _list_case(rng, True)
    for d in layers[::2]:
        del d["lazy_state"]
    for step in range(2):
        wants = []
        for d in layers:
            d["grad"], g_cpu = make_grad(rng, d["n"], d["grad_type"])
            wants.append(cref.pack(g_cpu, d["r_cpu"], d["L_T"], factor=d["factor"]))
        B.adacomp_compress_multi_opt(layers, len(layers))
        torch.cuda.synchronize()
        for i, (d, want) in enumerate(zip(layers, wants)):
            assert_stream_equal(d["packed_out"][:int(d["count_out"][1])].cpu().numpy(), want, f"layer {i} step {step}")
    assert B.adacomp_device_status() == 0
