"""Parity of adacomp_decompress_average_sgd (unpack + averageGradients + updateWeights in one pass)
against the oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import GpuLayer, assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu


def _streams(rng, n, L_T, k, dense_learner=None):
    out = []
    for l in range(k):
        r = rng.normal(0, 2e-3, n).astype(np.float32)
        dW = rng.normal(0, 1e-3 * (1 + l % 3), n).astype(np.float32)
        if dense_learner == l:
            dW = np.where(rng.random(n) < 0.5, -1.0, 1.0).astype(np.float32) * np.float32(0.5)
            r = np.zeros(n, np.float32)
        want = cref.pack(dW, r.copy(), L_T)
        raw, _, _ = GpuLayer(n, L_T, r).compress(dW)
        assert_stream_equal(raw, want)
        out.append(raw)
    return out


def _gpu_step(streams, n, L_T, w, v, lr, mu):
    dev = torch.device("cuda:0")
    bufs = [torch.from_numpy(s.copy()).to(dev) for s in streams]
    wd = torch.from_numpy(np.concatenate([w, np.full(8, 7.0, np.float32)])).to(dev)      # guard elements behind the layer
    vd = torch.from_numpy(np.concatenate([v, np.full(8, -7.0, np.float32)])).to(dev)
    B.adacomp_decompress_average_sgd(bufs, len(bufs), wd, vd, n, L_T, lr, mu)
    torch.cuda.synchronize()
    wh, vh = wd.cpu().numpy(), vd.cpu().numpy()
    assert np.all(wh[w.size:] == 7.0) and np.all(vh[v.size:] == -7.0), "wrote past the layer"
    return wh[:w.size], vh[:v.size]


@pytest.mark.parametrize("L_T,n,k", [(50, 100352, 1), (50, 4000 * 37 + 11, 4), (500, 147456, 8), (500, 4000 * 20 + 3, 3),
                                     (50, 4000 * 6 + 1, 16), (3, 9001, 3), (64, 70000, 2), (62, 31 * 3968 + 5, 3),
                                     (100, 50007, 5), (1001, 50001, 2), (16384, 100001, 3), (500, 12, 2),
                                     # bin-count runs that are no multiple of 16 bytes; 5 and 15 bins per warp
                                     (52, 76 * 52 * 5 + 9, 3), (63, 60 * 63 * 6 + 2, 4), (200, 20 * 200 * 7 + 3, 3),
                                     # one bin per tile: items of 4096 elements over 1 to 6 bins
                                     (1003, 4096 * 9 + 700, 4), (2000, 2000 * 30 + 1, 3), (5000, 5000 * 17 + 4097, 5)])
def test_fused_update_matches_oracle(L_T, n, k):
    rng = np.random.default_rng(1000 * L_T + n + k)
    streams = _streams(rng, n, L_T, k)
    w = rng.normal(0, 1, n).astype(np.float32)
    v = rng.normal(0, 1e-2, n).astype(np.float32)
    lr, mu = 0.1, 0.9
    want_w, want_v = cref.average_sgd(streams, n, w, v, lr, mu)
    got_w, got_v = _gpu_step(streams, n, L_T, w, v, lr, mu)
    assert_f32_bits_equal(got_v, want_v, f"momentum L_T={L_T} n={n} k={k}")
    assert_f32_bits_equal(got_w, want_w, f"weights L_T={L_T} n={n} k={k}")
    assert B.adacomp_device_status() == 0


def test_dense_learner_and_two_steps_in_a_row():
    """A learner that sends every element overflows its staging region (read from global memory instead);
    two calls in a row carry weights and momentum on."""
    rng = np.random.default_rng(3)
    for L_T, n, k in [(50, 4000 * 9 + 123, 5), (500, 4000 * 5 + 77, 4)]:
        w = rng.normal(0, 1, n).astype(np.float32)
        v = np.zeros(n, np.float32)
        gw, gv = w.copy(), v.copy()
        for step in range(2):
            streams = _streams(rng, n, L_T, k, dense_learner=2)
            w, v = cref.average_sgd(streams, n, w, v, 0.05, 0.9)
            gw, gv = _gpu_step(streams, n, L_T, gw, gv, 0.05, 0.9)
            assert_f32_bits_equal(gv, v, f"momentum step {step} L_T={L_T}")
            assert_f32_bits_equal(gw, w, f"weights step {step} L_T={L_T}")
    assert B.adacomp_device_status() == 0


def test_wrong_shape_leaves_the_arrays_alone_and_sets_a_status_bit():
    rng = np.random.default_rng(4)
    n, L_T = 20000, 50
    streams = _streams(rng, n, L_T, 2)
    w = rng.normal(0, 1, n).astype(np.float32)
    v = rng.normal(0, 1, n).astype(np.float32)
    B.adacomp_device_status_reset()
    got_w, got_v = _gpu_step(streams, n - 50, L_T, w, v, 0.1, 0.9)       # the streams say n, the caller n - 50
    assert B.adacomp_device_status() & B.ADACOMP_DEV_HEADER_MISMATCH
    np.testing.assert_array_equal(got_w, w)
    np.testing.assert_array_equal(got_v, v)
    B.adacomp_device_status_reset()


def test_layer_list_in_one_call_matches_per_layer_oracle():
    """Small layers share a batched launch, the large ones take the single-layer kernels; bin lengths mixed."""
    rng = np.random.default_rng(6)
    shapes = [(864, 500), (9216, 500), (5120, 50), (4000 * 1100 + 7, 50), (147456, 500), (67, 500), (2048, 50),
              (4000 * 1060, 500), (100, 7), (3996 * 3 + 5, 333), (3840 * 2 + 7, 64), (4000 * 2 + 999, 1000)]
    k = 3
    dev = torch.device("cuda:0")
    streams_cpu, bufs, ws, vs, w_dev, v_dev = [], [], [], [], [], []
    for n, L_T in shapes:
        layer_streams = _streams(rng, n, L_T, k)
        streams_cpu.append(layer_streams)
        bufs += [torch.from_numpy(s.copy()).to(dev) for s in layer_streams]
        w = rng.normal(0, 1, n).astype(np.float32)
        v = rng.normal(0, 1e-2, n).astype(np.float32)
        ws.append(w)
        vs.append(v)
        w_dev.append(torch.from_numpy(np.concatenate([w, np.full(4, 7.0, np.float32)])).to(dev))
        v_dev.append(torch.from_numpy(np.concatenate([v, np.full(4, -7.0, np.float32)])).to(dev))
    B.adacomp_decompress_average_sgd_multi(bufs, k, w_dev, v_dev, [n for n, _ in shapes], [L for _, L in shapes],
                                           len(shapes), 0.1, 0.9)
    torch.cuda.synchronize()
    for t, (n, L_T) in enumerate(shapes):
        want_w, want_v = cref.average_sgd(streams_cpu[t], n, ws[t], vs[t], 0.1, 0.9)
        got_w, got_v = w_dev[t].cpu().numpy(), v_dev[t].cpu().numpy()
        assert np.all(got_w[n:] == 7.0) and np.all(got_v[n:] == -7.0), f"layer {t}: wrote past the layer"
        assert_f32_bits_equal(got_v[:n], want_v, f"momentum layer {t} n={n} L_T={L_T}")
        assert_f32_bits_equal(got_w[:n], want_w, f"weights layer {t} n={n} L_T={L_T}")
    assert B.adacomp_device_status() == 0
