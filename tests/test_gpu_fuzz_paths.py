"""Seeded fuzz over the forms pack() can take for one input: the one-kernel form against the streaming kernels, a
parameter list against its layers packed one by one, lazy-scale against eager mode; streams, counts and residues
must agree bit for bit, and the smaller cases are also compared with the oracle."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FAST = [50, 100, 125, 200, 250, 500, 1000]


def pack_one(g, res, n, L_T, flags=0, factor=0.0, grad_type=0, lazy_state=None):
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_compress_opt(g, res, n, L_T, packed, cnt, flags=flags, factor=factor, grad_type=grad_type, lazy_state=lazy_state)
    torch.cuda.synchronize()
    return packed[:int(cnt[1])].clone(), cnt.clone()


@pytest.mark.parametrize("seed", [11, 12])
def test_one_kernel_form_against_streaming_kernels(seed):
    rng = np.random.default_rng(seed)
    for _ in range(60):
        L_T = int(rng.choice(FAST))
        n = int(rng.integers(1, 5_000_000)) if rng.random() < 0.3 else int(rng.integers(1, 60_000))
        factor = float(rng.choice([0.0, 0.0, 1.0, 1.5, 3.0]))
        g = torch.randn(n, device=DEV) * 1e-3
        if rng.random() < 0.3:
            g[::7] = 0
        r0 = torch.randn(n, device=DEV) * 2e-3
        ra, rb = r0.clone(), r0.clone()
        a, ca = pack_one(g, ra, n, L_T, 0, factor)
        b, cb = pack_one(g, rb, n, L_T, B.ADACOMP_FLAG_STREAMING, factor)
        assert torch.equal(ca, cb) and torch.equal(a, b), (L_T, n, factor)
        assert torch.equal(ra.view(torch.int32), rb.view(torch.int32)), (L_T, n, factor)
        if n < 200_000:
            rc = r0.cpu().numpy().copy()
            w = cref.pack(g.cpu().numpy(), rc, L_T, factor=factor)
            assert np.array_equal(a.cpu().numpy(), w.raw), (L_T, n, factor)
            assert np.array_equal(ra.cpu().numpy().view(np.uint32), rc.view(np.uint32)), (L_T, n, factor)
    assert B.adacomp_device_status() == 0


@pytest.mark.parametrize("seed", [21, 22])
def test_lists_against_their_layers_one_by_one(seed):
    rng = np.random.default_rng(seed)
    for _ in range(25):
        k = int(rng.integers(2, 40))
        big = rng.random() < 0.3
        layers, singles = [], []
        for t in range(k):
            L_T = int(rng.choice([50, 500] if rng.random() < 0.8 else [100, 64, 400]))
            n = int(rng.integers(1, 400_000 if big else 30_000))
            g = torch.randn(n, device=DEV) * 1e-3
            r0 = torch.randn(n, device=DEV) * 2e-3
            rl = torch.zeros(max(n, 4), device=DEV)
            rl[:n] = r0
            gl = torch.zeros(max(n, 4), device=DEV)
            gl[:n] = g
            layers.append(dict(grad=gl, residue=rl, n=n, L_T=L_T,
                               packed_out=torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV),
                               count_out=torch.zeros(2, dtype=torch.int64, device=DEV)))
            rs = r0.clone()
            singles.append((pack_one(g, rs, n, L_T, B.ADACOMP_FLAG_STREAMING), rs))
        B.adacomp_compress_multi(layers, k)
        torch.cuda.synchronize()
        for t in range(k):
            (s, c), rs = singles[t]
            L = layers[t]
            assert torch.equal(L["count_out"], c), (t, L["n"], L["L_T"], k)
            assert torch.equal(L["packed_out"][:int(c[1])], s), (t, L["n"], L["L_T"], k)
            assert torch.equal(L["residue"][:L["n"]].view(torch.int32), rs.view(torch.int32)), (t, L["n"], L["L_T"], k)
    assert B.adacomp_device_status() == 0


def test_lazy_scale_against_eager_mode_with_every_gradient_format():
    rng = np.random.default_rng(31)
    for _ in range(20):
        L_T = int(rng.choice(FAST + [64, 400]))
        n = int(rng.integers(1, 2_000_000))
        gt = int(rng.choice([0, 1, 2]))
        state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
        B.adacomp_lazy_state_init(state, n, L_T)
        re, rl = torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
        for step in range(3):
            g32 = torch.randn(n, device=DEV) * 1e-3
            g = g32 if gt == 0 else g32.to(torch.bfloat16 if gt == 1 else torch.float16)
            a, ca = pack_one(g, re, n, L_T, 0, 0.0, gt)
            b, cb = pack_one(g, rl, n, L_T, 0, 0.0, gt, state)
            assert torch.equal(ca, cb) and torch.equal(a, b), (L_T, n, gt, step)
        B.adacomp_residue_flush(rl, state, n, L_T)
        torch.cuda.synchronize()
        assert torch.equal(re.view(torch.int32), rl.view(torch.int32)), (L_T, n, gt)
    assert B.adacomp_device_status() == 0
