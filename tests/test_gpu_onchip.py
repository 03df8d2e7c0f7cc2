"""pack() in one kernel (a layer whose tiles all stay in shared memory until the scale of Section 2.5 is known)
against the oracle, bit for bit, and against the streaming kernels that ADACOMP_FLAG_STREAMING selects: streams,
counts and residues over carried steps, for every bin length the form takes, whole and ragged last tiles, one
tile, more tiles than CTAs, the largest layer the form takes and the first it does not, with a factor, under a
CUDA graph, and through the entry point that brings its own scratch."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
STREAMING = B.ADACOMP_FLAG_STREAMING


def carried(L_T, n, steps=3, factor=0.0, flags=0, seed=0, sigma=1e-3):
    rng = np.random.default_rng(seed + L_T * 7 + n)
    r_cpu = rng.normal(0, 2 * sigma, n).astype(np.float32)
    res = torch.zeros(max(n, 4), device=DEV)
    res[:n] = torch.from_numpy(r_cpu)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    out = []
    for step in range(steps):
        g_cpu = rng.normal(0, sigma, n).astype(np.float32)
        if step == 1 and n > 100:
            g_cpu[::97] = 0.0
            g_cpu[5:n:1013] *= 40.0
        g_dev = torch.from_numpy(g_cpu).to(DEV)
        want = cref.pack(g_cpu, r_cpu, L_T, factor=factor)          # (advances r_cpu)
        B.adacomp_compress_opt(g_dev, res, n, L_T, packed, cnt, flags=flags, factor=factor)
        torch.cuda.synchronize()
        what = f"L_T={L_T} n={n} step={step} flags={flags}"
        raw = packed[:int(cnt[1])].cpu().numpy()
        assert_stream_equal(raw, want, what)
        assert_f32_bits_equal(res[:n].cpu().numpy(), r_cpu, what + " residue")
        out.append(raw)
    assert B.adacomp_device_status() == 0
    return out


SHAPES = [(50, 4000), (50, 3999), (50, 1), (50, 49), (50, 4000 * 9 + 1999), (50, 4000 * 300 + 50), (50, 4000 * 613),
          (500, 4000 * 7 + 3), (500, 4000 * 297 + 499), (100, 4000 * 5 + 50), (125, 4000 * 11 + 124), (200, 4000 * 3 + 1),
          (250, 4000 * 2), (1000, 4000 * 6 + 999), (1000, 1000)]


@pytest.mark.parametrize("L_T,n", SHAPES)
def test_one_kernel_pack_matches_the_oracle(L_T, n):
    carried(L_T, n)


@pytest.mark.parametrize("L_T,n", SHAPES)
def test_streaming_kernels_on_the_same_layers(L_T, n):
    carried(L_T, n, flags=STREAMING)


def test_with_a_factor_and_all_zero_input():
    carried(50, 4000 * 21 + 7, factor=1.5)
    carried(500, 4000 * 21 + 7, factor=3.0)
    n, L_T = 4000 * 5 + 3, 50
    res = torch.zeros(n, device=DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_compress(torch.zeros(n, device=DEV), res, n, L_T, packed, cnt)
    torch.cuda.synchronize()
    z = np.zeros(n, np.float32)
    assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), cref.pack(z, z.copy(), L_T), "all zero")
    assert int(cnt[0]) == 0 and not res.any()


def test_the_largest_layer_of_the_form_and_the_first_beyond_it():
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    cap_tiles = sms * 2 * 4
    for L_T in (50, 500):
        for n in (4000 * cap_tiles, 4000 * cap_tiles - 1, 4000 * cap_tiles + 1, 4000 * (cap_tiles - sms) + 17):
            carried(L_T, n, steps=2)


def test_non_finite_values_are_reported_like_the_streaming_kernels_report_them():
    n, L_T = 4000 * 4, 50
    g = torch.randn(n, device=DEV) * 1e-3
    g[1234] = float("inf")
    res = torch.zeros(n, device=DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_device_status_reset()
    B.adacomp_compress(g, res, n, L_T, packed, cnt)
    torch.cuda.synchronize()
    assert B.adacomp_device_status() & B.ADACOMP_DEV_NONFINITE
    B.adacomp_device_status_reset()
    torch.cuda.synchronize()
    assert B.adacomp_device_status() == 0


def test_under_a_cuda_graph():
    n, L_T = 4000 * 40 + 11, 50
    rng = np.random.default_rng(5)
    r_cpu = np.zeros(n, np.float32)
    g_dev = torch.zeros(n, device=DEV)
    res = torch.zeros(n, device=DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    B.adacomp_compress(g_dev, res, n, L_T, packed, cnt)        # (first call outside the capture)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            B.adacomp_compress(g_dev, res, n, L_T, packed, cnt, stream=s.cuda_stream)
    for step in range(3):
        g_cpu = rng.normal(0, 1e-3, n).astype(np.float32)
        g_dev.copy_(torch.from_numpy(g_cpu))
        want = cref.pack(g_cpu, r_cpu, L_T)
        graph.replay()
        torch.cuda.synchronize()
        assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), want, f"replay {step}")
        assert_f32_bits_equal(res.cpu().numpy(), r_cpu, f"replay {step} residue")


def test_through_the_entry_point_with_its_own_scratch():
    n, L_T = 4000 * 50 + 3, 500
    rng = np.random.default_rng(9)
    r_cpu = rng.normal(0, 1e-3, n).astype(np.float32)
    res = torch.from_numpy(r_cpu).to(DEV)
    g_cpu = rng.normal(0, 1e-3, n).astype(np.float32)
    g_dev = torch.from_numpy(g_cpu).to(DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    want = cref.pack(g_cpu, r_cpu, L_T)
    B.adacomp_compress_static(g_dev, res, n, L_T, packed, cnt)
    torch.cuda.synchronize()
    assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), want, "own scratch")
    assert_f32_bits_equal(res.cpu().numpy(), r_cpu, "own scratch residue")


# ---- a whole parameter list in one kernel ----

def run_list(shapes, steps=2, factors=None, seed=3):
    """shapes: (L_T, n) per layer; every step and layer against the oracle."""
    rng = np.random.default_rng(seed)
    layers, r_cpu = [], []
    for t, (L_T, n) in enumerate(shapes):
        r = rng.normal(0, 2e-3, n).astype(np.float32)
        res = torch.zeros(max(n, 4), device=DEV)
        res[:n] = torch.from_numpy(r)
        r_cpu.append(r)
        layers.append(dict(grad=torch.zeros(max(n, 4), device=DEV), residue=res, n=n, L_T=L_T,
                           packed_out=torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV),
                           count_out=torch.zeros(2, dtype=torch.int64, device=DEV),
                           factor=0.0 if factors is None else factors[t]))
    for step in range(steps):
        want = []
        for t, (L_T, n) in enumerate(shapes):
            g = rng.normal(0, 1e-3, n).astype(np.float32)
            layers[t]["grad"][:n].copy_(torch.from_numpy(g))
            want.append(cref.pack(g, r_cpu[t], L_T, factor=layers[t]["factor"]))
        if factors is None:
            B.adacomp_compress_multi(layers, len(layers))
        else:
            B.adacomp_compress_multi_opt(layers, len(layers))
        torch.cuda.synchronize()
        for t, (L_T, n) in enumerate(shapes):
            what = f"step {step} layer {t} L_T={L_T} n={n}"
            used = int(layers[t]["count_out"][1])
            assert_stream_equal(layers[t]["packed_out"][:used].cpu().numpy(), want[t], what)
            assert_f32_bits_equal(layers[t]["residue"][:n].cpu().numpy(), r_cpu[t], what + " residue")
    assert B.adacomp_device_status() == 0


def test_list_in_one_kernel_mixed_bin_lengths_ragged_and_tiny_layers():
    run_list([(500, 4000 * 7 + 3), (50, 4000 * 5 + 49), (500, 64), (50, 1), (500, 4000 * 2), (50, 4000), (500, 3999),
              (50, 4000 * 30 + 1999), (500, 4000 * 41 + 1)], steps=3)


def test_list_in_one_kernel_with_factors():
    run_list([(500, 4000 * 6 + 7), (50, 4000 * 9 + 11), (500, 4000 * 3)], factors=[1.5, 0.0, 3.0])


def test_list_at_the_capacity_of_the_one_kernel_form_and_beyond():
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    cap_tiles = sms * 2 * 2                         # (lists: two tiles per CTA)
    half = cap_tiles // 2
    run_list([(50, 4000 * half), (500, 4000 * (cap_tiles - half) - 17)], steps=2)           # exactly the capacity
    run_list([(50, 4000 * half), (500, 4000 * (cap_tiles - half) + 1)], steps=2)            # one tile more: the batch kernels


def test_list_with_another_bin_length_takes_the_batch_kernels():
    run_list([(500, 4000 * 6 + 7), (100, 4000 * 4 + 50), (50, 4000 * 3 + 1)], steps=2)


def test_list_in_one_kernel_under_a_cuda_graph():
    shapes = [(500, 4000 * 11 + 5), (50, 4000 * 6 + 3), (500, 1000)]
    rng = np.random.default_rng(21)
    layers, r_cpu = [], []
    for L_T, n in shapes:
        r_cpu.append(np.zeros(n, np.float32))
        layers.append(dict(grad=torch.zeros(n, device=DEV), residue=torch.zeros(n, device=DEV), n=n, L_T=L_T,
                           packed_out=torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV),
                           count_out=torch.zeros(2, dtype=torch.int64, device=DEV)))
    descs = B.make_layer_descs(layers)
    B.adacomp_compress_multi(descs, len(layers))            # (first call outside the capture)
    torch.cuda.synchronize()
    s = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            B.adacomp_compress_multi(descs, len(layers), stream=s.cuda_stream)
    for step in range(3):
        want = []
        for t, (L_T, n) in enumerate(shapes):
            g = rng.normal(0, 1e-3, n).astype(np.float32)
            layers[t]["grad"].copy_(torch.from_numpy(g))
            want.append(cref.pack(g, r_cpu[t], L_T))
        graph.replay()
        torch.cuda.synchronize()
        for t, (L_T, n) in enumerate(shapes):
            used = int(layers[t]["count_out"][1])
            assert_stream_equal(layers[t]["packed_out"][:used].cpu().numpy(), want[t], f"replay {step} layer {t}")
            assert_f32_bits_equal(layers[t]["residue"].cpu().numpy(), r_cpu[t], f"replay {step} layer {t} residue")


def test_list_in_one_kernel_with_more_layers_than_the_small_table():
    rng = np.random.default_rng(77)
    shapes = [(500 if t % 3 else 50, int(rng.integers(1, 3 * 4000))) for t in range(60)]
    run_list(shapes, steps=2, seed=78)
    shapes = [(50 if t % 2 else 500, int(rng.integers(1, 2 * 4000))) for t in range(200)]      # two batches
    run_list(shapes, steps=1, seed=79)
