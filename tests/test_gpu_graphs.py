"""The entry points are stream-ordered and allocate nothing, so a whole step can be captured into a CUDA graph
and replayed: same bytes as the direct calls, with new gradients written into the captured buffers."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal

pytestmark = pytest.mark.gpu


def test_captured_step_replays_bit_exactly():
    dev = torch.device("cuda:0")
    n, L_T, k = 100352, 50, 2
    rng = np.random.default_rng(12)
    grads = [torch.zeros(n, device=dev) for _ in range(k)]
    residues = [torch.zeros(n, device=dev) for _ in range(k)]
    packed = [torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=dev) for _ in range(k)]
    counts = [torch.zeros(2, dtype=torch.int64, device=dev) for _ in range(k)]
    dst = torch.empty(n, device=dev)
    w = torch.from_numpy(np.linspace(-1, 1, n, dtype=np.float32)).to(dev)
    v = torch.zeros(n, device=dev)

    def step():
        for l in range(k):
            B.adacomp_compress(grads[l], residues[l], n, L_T, packed[l], counts[l])
        B.adacomp_decompress_accumulate_ex(packed, k, dst, n, L_T)
        B.adacomp_decompress_average_sgd(packed, k, w, v, n, L_T, 0.1, 0.9)

    step()                                   # first use: one-time attribute set-up happens outside the capture
    for r in residues:
        r.zero_()
    w.copy_(torch.from_numpy(np.linspace(-1, 1, n, dtype=np.float32)))
    v.zero_()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for r in residues:                       # capture does not run anything: start from a known state
        r.zero_()
    r_cpu = [np.zeros(n, np.float32) for _ in range(k)]
    w_cpu, v_cpu = np.linspace(-1, 1, n, dtype=np.float32), np.zeros(n, np.float32)
    for it in range(3):
        dws = [rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(k)]
        for l in range(k):
            grads[l].copy_(torch.from_numpy(dws[l]))
        graph.replay()
        torch.cuda.synchronize()
        want = [cref.pack(dws[l], r_cpu[l], L_T) for l in range(k)]
        for l in range(k):
            used = int(counts[l][1])
            assert used == want[l].bytes_used
            assert np.array_equal(packed[l][:used].cpu().numpy(), want[l].raw), f"replay {it} learner {l}"
            assert_f32_bits_equal(residues[l].cpu().numpy(), r_cpu[l], f"residue replay {it} learner {l}")
        streams = [x.raw for x in want]
        assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum(streams, n), f"dense sum replay {it}")
        w_cpu, v_cpu = cref.average_sgd(streams, n, w_cpu, v_cpu, 0.1, 0.9)
        assert_f32_bits_equal(w.cpu().numpy(), w_cpu, f"weights replay {it}")
    assert B.adacomp_device_status() == 0
