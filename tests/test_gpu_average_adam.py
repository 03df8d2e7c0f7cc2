"""Parity of adacomp_decompress_average_adam (unpack + averageGradients + Adam step in one pass) with the
oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal
from tests.test_gpu_average_sgd import _streams

pytestmark = pytest.mark.gpu
HYPER = dict(step_size=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)


def _state(rng, n):
    w = rng.normal(0, 1, n).astype(np.float32)
    m = rng.normal(0, 1e-3, n).astype(np.float32)
    v = (rng.normal(0, 1e-3, n).astype(np.float32)) ** 2
    m[::11] = 0                                   # first steps of training: zero moments in places
    v[::13] = 0
    return w, m, v


def _dev(a, fill):
    return torch.from_numpy(np.concatenate([a, np.full(8, fill, np.float32)])).to("cuda:0")


@pytest.mark.parametrize("L_T,n,k", [(50, 100352, 1), (50, 4000 * 37 + 11, 4), (500, 147456, 8), (500, 4000 * 20 + 3, 3),
                                     (50, 4000 * 6 + 1, 16), (3, 9001, 3), (64, 70000, 2), (1001, 50001, 2), (500, 12, 2),
                                     (58, 68 * 58 * 5 + 3, 3), (300, 12 * 300 * 9 + 7, 4), (3000, 3000 * 21 + 2, 3),
                                     (16384, 16384 * 4 + 5000, 2)])
def test_fused_adam_matches_oracle_over_two_steps(L_T, n, k):
    rng = np.random.default_rng(2000 * L_T + n + k)
    w, m, v = _state(rng, n)
    wd, md, vd = _dev(w, 7.0), _dev(m, -7.0), _dev(v, 3.0)
    for step in range(2):
        streams = _streams(rng, n, L_T, k)
        w, m, v = cref.average_adam(streams, n, w, m, v, **HYPER)
        bufs = [torch.from_numpy(s.copy()).to("cuda:0") for s in streams]
        B.adacomp_decompress_average_adam(bufs, k, wd, md, vd, n, L_T, HYPER["step_size"], HYPER["beta1"],
                                          HYPER["beta2"], HYPER["eps"])
        torch.cuda.synchronize()
        gw, gm, gv = wd.cpu().numpy(), md.cpu().numpy(), vd.cpu().numpy()
        assert np.all(gw[n:] == 7.0) and np.all(gm[n:] == -7.0) and np.all(gv[n:] == 3.0), "wrote past the layer"
        assert_f32_bits_equal(gm[:n], m, f"m step {step} L_T={L_T} n={n} k={k}")
        assert_f32_bits_equal(gv[:n], v, f"v step {step}")
        assert_f32_bits_equal(gw[:n], w, f"w step {step}")
    assert B.adacomp_device_status() == 0


def test_layer_list_in_one_call():
    rng = np.random.default_rng(8)
    shapes = [(864, 500), (5120, 50), (4000 * 1100 + 7, 50), (147456, 500), (67, 500), (100, 7), (3996 * 3 + 5, 333),
              (3840 * 2 + 7, 64)]
    k = 3
    streams_cpu, bufs, st, dv = [], [], [], []
    for n, L_T in shapes:
        ls = _streams(rng, n, L_T, k)
        streams_cpu.append(ls)
        bufs += [torch.from_numpy(s.copy()).to("cuda:0") for s in ls]
        w, m, v = _state(rng, n)
        st.append((w, m, v))
        dv.append((_dev(w, 7.0), _dev(m, -7.0), _dev(v, 3.0)))
    B.adacomp_decompress_average_adam_multi(bufs, k, [d[0] for d in dv], [d[1] for d in dv], [d[2] for d in dv],
                                            [n for n, _ in shapes], [L for _, L in shapes], len(shapes),
                                            HYPER["step_size"], HYPER["beta1"], HYPER["beta2"], HYPER["eps"])
    torch.cuda.synchronize()
    for t, (n, L_T) in enumerate(shapes):
        w, m, v = cref.average_adam(streams_cpu[t], n, *st[t], **HYPER)
        gw, gm, gv = (d.cpu().numpy() for d in dv[t])
        assert np.all(gw[n:] == 7.0) and np.all(gm[n:] == -7.0) and np.all(gv[n:] == 3.0), f"layer {t}"
        assert_f32_bits_equal(gm[:n], m, f"m layer {t}")
        assert_f32_bits_equal(gv[:n], v, f"v layer {t}")
        assert_f32_bits_equal(gw[:n], w, f"w layer {t}")
    assert B.adacomp_device_status() == 0
