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
