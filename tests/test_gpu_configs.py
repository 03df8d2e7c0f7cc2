"""Parity of the CUDA path with the oracle on the workload shapes of the benchmark configs:
the ResNet-50 parameter list with 8 learners, the speech DNN with 16 learners, the flat
bandwidth sweep (eager and lazy pack), and one full-size (2^30) case."""
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from paper_1712_02679_b200 import synth
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _oracle_many(jobs, threads=8):
    """jobs: (dW, residue, L_T) -> list of Packed; residues updated in place.  The C oracle
    releases the GIL, so independent layers run on separate host threads."""
    with ThreadPoolExecutor(threads) as ex:
        return list(ex.map(lambda j: cref.pack(j[0], j[1], j[2]), jobs))


def _multi_tensor_case(cfg, specs, learners, heavy_sigma=None):
    dev = torch.device(DEV)
    n_t = len(specs)
    # one flat allocation per learner and kind, carved into 16-byte aligned per-tensor views
    def carve(total_fn, dtype):
        sizes = [(total_fn(s) + 127) // 128 * 128 for s in specs]
        flat = torch.zeros(sum(sizes), dtype=dtype, device=dev)
        views, at = [], 0
        for s, size in zip(specs, sizes):
            views.append(flat[at:at + total_fn(s)])
            at += size
        return flat, views
    streams_cpu = [[None] * learners for _ in range(n_t)]
    packed_views = []
    for l in range(learners):
        dws = [synth.make_dw(cfg, l, t, 0, s.n, heavy=True, sigma=heavy_sigma) for t, s in enumerate(specs)]
        r_cpu = [np.zeros(s.n, np.float32) for s in specs]
        want = _oracle_many([(dws[t], r_cpu[t], specs[t].L_T) for t in range(n_t)])
        _, grad = carve(lambda s: max(s.n, 4), torch.float32)
        _, res = carve(lambda s: max(s.n, 4), torch.float32)
        _, packed = carve(lambda s: B.adacomp_packed_capacity(s.n, s.L_T), torch.uint8)
        counts = torch.zeros(n_t, 2, dtype=torch.int64, device=dev)
        for t in range(n_t):
            grad[t][:specs[t].n].copy_(torch.from_numpy(dws[t]))
        descs = [dict(grad=grad[t], residue=res[t], n=specs[t].n, L_T=specs[t].L_T, packed_out=packed[t],
                      count_out=counts[t]) for t in range(n_t)]
        B.adacomp_compress_multi(descs, n_t)
        torch.cuda.synchronize()
        host_counts = counts.cpu().numpy()
        for t in range(n_t):
            used = int(host_counts[t, 1])
            assert int(host_counts[t, 0]) == want[t].n_sel, (l, t)
            assert_stream_equal(packed[t][:used].cpu().numpy(), want[t], f"learner {l} tensor {t} {specs[t].name}")
            streams_cpu[t][l] = want[t].raw
        got_res = [res[t][:specs[t].n].cpu().numpy() for t in range(n_t)]
        for t in range(n_t):
            assert_f32_bits_equal(got_res[t], r_cpu[t], f"residue learner {l} tensor {t}")
        packed_views.append(packed)
    # one decode-sum of the `learners` streams of every tensor
    _, dsts = carve(lambda s: max(s.n, 4), torch.float32)
    flat_packed = [packed_views[l][t] for t in range(n_t) for l in range(learners)]
    B.adacomp_decompress_accumulate_multi_ex(flat_packed, learners, dsts, [s.n for s in specs],
                                             [s.L_T for s in specs], n_t)
    torch.cuda.synchronize()
    with ThreadPoolExecutor(8) as ex:
        refs = list(ex.map(lambda t: cref.unpack_sum(streams_cpu[t], specs[t].n), range(n_t)))
    for t in range(n_t):
        assert_f32_bits_equal(dsts[t][:specs[t].n].cpu().numpy(), refs[t], f"dense sum tensor {t}")
    assert B.adacomp_device_status() == 0


def test_config3_resnet50_parameter_list_eight_learners():
    specs = synth.resnet50_tensors()
    assert len(specs) == 161 and sum(s.n for s in specs) == 25_557_032
    _multi_tensor_case(3, specs, learners=8)


def test_config4_speech_dnn_sixteen_learners():
    # the 1024-wide variant keeps 16 learners' oracle runs within seconds
    specs = synth.config4_tensors(hidden=1024)
    assert sum(s.n for s in specs) == 15_216_640
    _multi_tensor_case(4, specs, learners=16, heavy_sigma=1e-3)


def test_lstm_parameter_list_eight_learners():
    specs = synth.lstm_tensors()
    assert len(specs) == 10 and sum(s.n for s in specs) == 2048 * (67 + 512 + 512 + 512) + 4 * 2048 + 67 * 512 + 67
    _multi_tensor_case(6, specs, learners=8)


def test_mixed_list_whose_layers_of_bin_length_50_get_batches_of_their_own():
    # 3000 tiles and more of bin length 50 beside other bin lengths: the 50s are packed by the batch form with
    # the tile's shape compiled in, the others by the any-bin form; the order of the layers in the list stays free
    T = synth.TensorSpec
    specs = [T("fc_a", 4000 * 1100 + 37, 50, "fc"), T("conv_a", 4000 * 40 + 499, 500, "conv"), T("fc_b", 4000 * 1000, 50, "fc"),
             T("bn", 256, 500, "bn"), T("other", 4000 * 30 + 50, 100, "conv"), T("fc_c", 4000 * 950 + 1, 50, "fc"),
             T("fc_bias", 1000, 50, "fc"), T("conv_b", 4000 * 25, 500, "conv")]
    _multi_tensor_case(7, specs, learners=2, heavy_sigma=1e-3)


@pytest.mark.parametrize("L_T", [50, 500])
@pytest.mark.parametrize("log2n", [20, 22, 24])
def test_config5_sweep_point_prewarmed_eager_and_lazy(L_T, log2n):
    n, k = 1 << log2n, 4
    dev = torch.device(DEV)
    rng = np.random.default_rng([5, L_T, log2n])
    draw = lambda: rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)
    r_cpu = [np.zeros(n, np.float32) for _ in range(k)]
    res_e = [torch.zeros(n, device=dev) for _ in range(k)]
    res_l = [torch.zeros(n, device=dev) for _ in range(k)]
    cap = B.adacomp_packed_capacity(n, L_T)
    packed = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(k)]
    packed_l = torch.empty(cap, dtype=torch.uint8, device=dev)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    state = [torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=dev) for _ in range(k)]
    for s in state:
        B.adacomp_lazy_state_init(s, n, L_T)
    want_last = [None] * k
    for step in range(6):                      # 5 pre-warm steps, then the measured one
        dws = [draw() for _ in range(k)]
        want = _oracle_many([(dws[l], r_cpu[l], L_T) for l in range(k)], threads=4)
        for l in range(k):
            g = torch.from_numpy(dws[l]).to(dev)
            B.adacomp_compress(g, res_e[l], n, L_T, packed[l], cnt)
            torch.cuda.synchronize()
            assert_stream_equal(packed[l][:int(cnt[1])].cpu().numpy(), want[l], f"eager step {step} learner {l}")
            B.adacomp_compress_lazy(g, res_l[l], state[l], n, L_T, packed_l, cnt)
            torch.cuda.synchronize()
            assert_stream_equal(packed_l[:int(cnt[1])].cpu().numpy(), want[l], f"lazy step {step} learner {l}")
        want_last = want
    for l in range(k):
        assert_f32_bits_equal(res_e[l].cpu().numpy(), r_cpu[l], f"eager residue learner {l}")
        B.adacomp_residue_flush(res_l[l], state[l], n, L_T)
        assert_f32_bits_equal(res_l[l].cpu().numpy(), r_cpu[l], f"flushed lazy residue learner {l}")
    dst = torch.empty(n, device=dev)
    B.adacomp_decompress_accumulate(packed, k, dst)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum([w.raw for w in want_last], n), "dense sum")
    # the rate is where the paper puts it for Gaussian inputs at step 6 (about 35x / 66x)
    rate = 32.0 * n / (8.0 * want_last[0].w * want_last[0].n_sel)
    assert rate == pytest.approx(35.0 if L_T == 50 else 66.0, rel=0.1)
    assert B.adacomp_device_status() == 0


def test_full_size_2_to_30_two_learners():
    """The benchmark's largest tensor, in the launch configuration bench.py times: two learners'
    first step from a zero residue, a carried second step for learner 0, and the dense sum."""
    n, L_T = 1 << 30, 50
    dev = torch.device(DEV)
    gen = torch.Generator(device=dev)
    cap = B.adacomp_packed_capacity(n, L_T)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    g = torch.empty(n, device=dev)
    packed, raws = [], []
    res0 = None
    r_cpu0 = None
    for l in range(2):
        gen.manual_seed(900 + l)
        g.normal_(0.0, 1e-3, generator=gen)            # seeded torch generator, copied to the host
        dW = g.cpu().numpy()
        r_cpu = np.zeros(n, np.float32)
        want = cref.pack(dW, r_cpu, L_T)
        res = torch.zeros(n, device=dev)
        pk = torch.empty(cap, dtype=torch.uint8, device=dev)
        B.adacomp_compress(g, res, n, L_T, pk, cnt)
        torch.cuda.synchronize()
        used = int(cnt[1])
        assert int(cnt[0]) == want.n_sel
        assert_stream_equal(pk[:used].cpu().numpy(), want, f"2^30 learner {l} step 0")
        assert_f32_bits_equal(res.cpu().numpy(), r_cpu, f"2^30 residue learner {l}")
        assert want.n_sel / n == pytest.approx(0.2213, rel=0.01)   # first-step fraction, scale free
        packed.append(pk)
        raws.append(want.raw)
        if l == 0:
            res0, r_cpu0 = res, r_cpu
        del dW
    dst = torch.empty(n, device=dev)
    B.adacomp_decompress_accumulate(packed, 2, dst)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum(raws, n), "2^30 dense sum")
    del dst, raws
    # carried step for learner 0
    gen.manual_seed(950)
    g.normal_(0.0, 1e-3, generator=gen)
    dW = g.cpu().numpy()
    want = cref.pack(dW, r_cpu0, L_T)
    B.adacomp_compress(g, res0, n, L_T, packed[0], cnt)
    torch.cuda.synchronize()
    assert_stream_equal(packed[0][:int(cnt[1])].cpu().numpy(), want, "2^30 learner 0 step 1")
    assert_f32_bits_equal(res0.cpu().numpy(), r_cpu0, "2^30 residue learner 0 step 1")
    assert B.adacomp_device_status() == 0


@pytest.mark.parametrize("L_T", [50, 500])
@pytest.mark.parametrize("log2n,learners", [(26, 4), (28, 1)])
def test_config5_upper_sweep_points_prewarmed(L_T, log2n, learners):
    """The sweep's points above 2^24: six carried steps (five pre-warm steps and the measured one), eager
    and lazy-scale pack() compared with the oracle byte for byte at every step, then the dense sum; all four
    learners at 2^26, learner 0 alone at 2^28.  The gradients come from a seeded torch CUDA generator and are
    copied to the host for the oracle."""
    n, k = 1 << log2n, learners
    dev = torch.device(DEV)
    gen = torch.Generator(device=dev)
    gen.manual_seed(7000 + log2n + L_T)
    g = torch.empty(n, device=dev)
    r_cpu = [np.zeros(n, np.float32) for _ in range(k)]
    res_e = [torch.zeros(n, device=dev) for _ in range(k)]
    res_l = [torch.zeros(n, device=dev) for _ in range(k)]
    cap = B.adacomp_packed_capacity(n, L_T)
    packed = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(k)]
    packed_l = torch.empty(cap, dtype=torch.uint8, device=dev)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    state = [torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=dev) for _ in range(k)]
    for s in state:
        B.adacomp_lazy_state_init(s, n, L_T)
    last = [None] * k
    for step in range(6):
        for l in range(k):
            g.normal_(0.0, 1e-3, generator=gen)
            want = cref.pack(g.cpu().numpy(), r_cpu[l], L_T)
            B.adacomp_compress(g, res_e[l], n, L_T, packed[l], cnt)
            torch.cuda.synchronize()
            assert_stream_equal(packed[l][:int(cnt[1])].cpu().numpy(), want, f"eager step {step} learner {l}")
            B.adacomp_compress_lazy(g, res_l[l], state[l], n, L_T, packed_l, cnt)
            torch.cuda.synchronize()
            assert_stream_equal(packed_l[:int(cnt[1])].cpu().numpy(), want, f"lazy step {step} learner {l}")
            last[l] = want.raw
    for l in range(k):
        assert_f32_bits_equal(res_e[l].cpu().numpy(), r_cpu[l], f"eager residue learner {l}")
        B.adacomp_residue_flush(res_l[l], state[l], n, L_T)
        assert_f32_bits_equal(res_l[l].cpu().numpy(), r_cpu[l], f"flushed lazy residue learner {l}")
    del res_e, res_l, state, g
    dst = torch.empty(n, device=dev)
    B.adacomp_decompress_accumulate_ex(packed, k, dst, n, L_T)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum(last, n), "dense sum")
    assert B.adacomp_device_status() == 0


def test_full_size_2_to_30_lazy_scale_two_carried_steps_and_flush():
    """The entry point that meets the bandwidth target at 2^30, adacomp_compress_lazy, against the oracle:
    two carried steps (the second applies the first one's pending subtraction while it loads), every stream
    byte for byte, then the flush that turns the buffer into the paper's residue."""
    n, L_T = 1 << 30, 50
    dev = torch.device(DEV)
    gen = torch.Generator(device=dev)
    g = torch.empty(n, device=dev)
    res = torch.zeros(n, device=dev)
    r_cpu = np.zeros(n, np.float32)
    pk = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=dev)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=dev)
    B.adacomp_lazy_state_init(state, n, L_T)
    for step in range(2):
        gen.manual_seed(1200 + step)
        g.normal_(0.0, 1e-3, generator=gen)
        want = cref.pack(g.cpu().numpy(), r_cpu, L_T)
        B.adacomp_compress_lazy(g, res, state, n, L_T, pk, cnt)
        torch.cuda.synchronize()
        assert int(cnt[0]) == want.n_sel
        assert_stream_equal(pk[:int(cnt[1])].cpu().numpy(), want, f"2^30 lazy step {step}")
        del want
    B.adacomp_residue_flush(res, state, n, L_T)
    torch.cuda.synchronize()
    assert_f32_bits_equal(res.cpu().numpy(), r_cpu, "2^30 lazy residue after the flush")
    assert B.adacomp_device_status() == 0


def test_full_size_2_to_30_bins_of_500_and_the_fused_update():
    """2^30 elements at L_T = 500 (16-bit words): two learners' eager pack() and the dense sum against the
    oracle; then, at L_T = 50, the fused unpack + average + SGD step of the same size, compared in slices with
    the oracle's averageGradients() / updateWeights() so that the host never holds more than a few full-size
    arrays."""
    n = 1 << 30
    dev = torch.device(DEV)
    gen = torch.Generator(device=dev)
    g = torch.empty(n, device=dev)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    for L_T in (500, 50):
        cap = B.adacomp_packed_capacity(n, L_T)
        packed, raws = [], []
        for l in range(2):
            gen.manual_seed(1300 + l + L_T)
            g.normal_(0.0, 1e-3, generator=gen)
            r_cpu = np.zeros(n, np.float32)
            want = cref.pack(g.cpu().numpy(), r_cpu, L_T)
            res = torch.zeros(n, device=dev)
            pk = torch.empty(cap, dtype=torch.uint8, device=dev)
            B.adacomp_compress(g, res, n, L_T, pk, cnt)
            torch.cuda.synchronize()
            assert_stream_equal(pk[:int(cnt[1])].cpu().numpy(), want, f"2^30 L_T={L_T} learner {l}")
            assert_f32_bits_equal(res.cpu().numpy(), r_cpu, f"2^30 L_T={L_T} residue learner {l}")
            packed.append(pk)
            raws.append(want.raw)
            del res, r_cpu, want
        want_sum = cref.unpack_sum(raws, n)
        if L_T == 500:
            dst = torch.empty(n, device=dev)
            B.adacomp_decompress_accumulate_ex(packed, 2, dst, n, L_T)
            torch.cuda.synchronize()
            assert_f32_bits_equal(dst.cpu().numpy(), want_sum, "2^30 L_T=500 dense sum")
            del dst
        else:
            # weights and momentum that are cheap to make on both sides and exact in binary32
            idx = torch.arange(n, device=dev, dtype=torch.int32)
            w = ((idx % 1021).to(torch.float32) - 510.0) * (1.0 / 1024.0)
            v = ((idx % 509).to(torch.float32) - 254.0) * (1.0 / 4096.0)
            del idx
            B.adacomp_decompress_average_sgd(packed, 2, w, v, n, L_T, 0.1, 0.9)
            torch.cuda.synchronize()
            w_gpu, v_gpu = w.cpu().numpy(), v.cpu().numpy()
            del w, v
            f = np.float32
            step = 1 << 26
            for lo in range(0, n, step):
                i = np.arange(lo, lo + step, dtype=np.int64)
                w0 = ((i % 1021).astype(np.float32) - f(510.0)) * f(1.0 / 1024.0)
                v0 = ((i % 509).astype(np.float32) - f(254.0)) * f(1.0 / 4096.0)
                w1, v1 = cref.sgd_step(want_sum[lo:lo + step], 2, w0, v0, 0.1, 0.9)
                assert_f32_bits_equal(v_gpu[lo:lo + step], v1, f"2^30 fused update, momentum from {lo}")
                assert_f32_bits_equal(w_gpu[lo:lo + step], w1, f"2^30 fused update, weights from {lo}")
        del packed, raws, want_sum
    assert B.adacomp_device_status() == 0

