"""Lazy-scale pack(): every stream must equal the oracle's (and so the eager path's) bit for bit
over carried steps; after a flush the residue must be the oracle's residue bit for bit."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from paper_1712_02679_b200 import synth
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu


class LazyLayer:
    def __init__(self, n, L_T, residue0=None):
        dev = torch.device("cuda:0")
        self.n, self.L_T = n, L_T
        self.residue = torch.zeros(n, dtype=torch.float32, device=dev)
        if residue0 is not None:
            self.residue.copy_(torch.from_numpy(residue0))
        self.grad = torch.empty(n, dtype=torch.float32, device=dev)
        self.packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=dev)
        self.count = torch.zeros(2, dtype=torch.int64, device=dev)
        self.state = torch.full((B.adacomp_lazy_state_bytes(n, L_T),), 0x5A, dtype=torch.uint8, device=dev)
        B.adacomp_lazy_state_init(self.state, n, L_T)

    def step(self, dW):
        self.grad.copy_(torch.from_numpy(dW))
        self.packed.fill_(0xAB)
        B.adacomp_compress_lazy(self.grad, self.residue, self.state, self.n, self.L_T, self.packed, self.count)
        torch.cuda.synchronize()
        used = int(self.count[1])
        return self.packed[:used].cpu().numpy()

    def flushed_residue(self):
        B.adacomp_residue_flush(self.residue, self.state, self.n, self.L_T)
        torch.cuda.synchronize()
        return self.residue.cpu().numpy()


@pytest.mark.parametrize("L_T,n,heavy", [(50, 100352, False), (500, 147456, True), (50, 4000 * 37 + 1234, True),
                                         (500, 4000 * 300 - 7, False), (50, 3999, False), (500, 17, False),
                                         (50, 4000 * 296, False), (100, 4000 * 31 + 99, True), (125, 4000 * 12 + 1, False),
                                         (200, 4000 * 40, False), (250, 4000 * 9 + 3999, True), (1000, 4000 * 25 + 500, False),
                                         # bins that do not line up with the 25-element segments (tiles of 3936, 3840, 3600, 3996 elements)
                                         (41, 3936 * 21 + 40, True), (64, 3840 * 30, False), (300, 3600 * 17 + 1801, True),
                                         (999, 3996 * 12 + 5, False), (65, 3900 * 3 - 1, False),
                                         # a tile is one bin
                                         (1004, 1004 * 41 + 3, False), (2000, 2000 * 33 + 1999, True), (4000, 4000 * 9 + 1, False)])
def test_lazy_steps_match_oracle_and_flush_restores_the_residue(L_T, n, heavy):
    rng = np.random.default_rng(n + L_T)
    res0 = rng.normal(0, 2e-3, n).astype(np.float32)
    r_cpu = res0.copy()
    layer = LazyLayer(n, L_T, res0)
    for step in range(6):
        dW = synth.heavy_dw(n, 1e-3, rng) if heavy else rng.normal(0, 1e-3, n).astype(np.float32)
        want = cref.pack(dW, r_cpu, L_T)
        raw = layer.step(dW)
        assert_stream_equal(raw, want, f"lazy L_T={L_T} n={n} step={step}")
        if step in (2, 5):       # flush mid-run and at the end: residue is the oracle's, bit for bit
            assert_f32_bits_equal(layer.flushed_residue(), r_cpu, f"flush after step {step}")
            # a second flush is a no-op
            assert_f32_bits_equal(layer.flushed_residue(), r_cpu, "second flush")
    assert B.adacomp_device_status() == 0


def test_unflushed_residue_holds_G_and_eager_continues_after_a_flush():
    n, L_T = 4000 * 20 + 77, 50
    rng = np.random.default_rng(5)
    r_cpu = np.zeros(n, np.float32)
    layer = LazyLayer(n, L_T)
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    G = r_cpu + dW
    want = cref.pack(dW, r_cpu, L_T)
    assert_stream_equal(layer.step(dW), want)
    assert_f32_bits_equal(layer.residue.cpu().numpy(), G, "before the flush the buffer holds G")
    assert_f32_bits_equal(layer.flushed_residue(), r_cpu)
    # now the plain entry point can take over
    dW2 = rng.normal(0, 1e-3, n).astype(np.float32)
    want2 = cref.pack(dW2, r_cpu, L_T)
    layer.grad.copy_(torch.from_numpy(dW2))
    B.adacomp_compress(layer.grad, layer.residue, n, L_T, layer.packed, layer.count)
    torch.cuda.synchronize()
    assert_stream_equal(layer.packed[:int(layer.count[1])].cpu().numpy(), want2)
    assert_f32_bits_equal(layer.residue.cpu().numpy(), r_cpu)


def test_lazy_rejects_other_bin_lengths_and_foreign_state():
    dev = torch.device("cuda:0")
    assert B.adacomp_lazy_state_bytes(1000, 40) == 0
    assert B.adacomp_lazy_state_bytes(100000, 1001) == 0
    assert B.adacomp_lazy_state_bytes(100352, 50) == 64 + 26 * 640
    n = 8000
    t = torch.zeros(n, device=dev)
    packed = torch.empty(B.adacomp_packed_capacity(n, 40), dtype=torch.uint8, device=dev)
    cnt = torch.zeros(2, dtype=torch.int64, device=dev)
    state = torch.zeros(4096, dtype=torch.uint8, device=dev)
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_compress_lazy(t, t.clone(), state, n, 40, packed, cnt)
    assert e.value.code == -9
    # a state initialised for another tensor: status bit, nothing written
    layer = LazyLayer(n, 50)
    other = torch.zeros(B.adacomp_lazy_state_bytes(2 * n, 50), dtype=torch.uint8, device=dev)
    B.adacomp_lazy_state_init(other, 2 * n, 50)
    B.adacomp_device_status_reset()
    layer.residue.fill_(1.0)
    layer.grad.fill_(0.5)
    layer.count.fill_(-1)
    B.adacomp_compress_lazy(layer.grad, layer.residue, other, n, 50, layer.packed, layer.count)
    assert B.adacomp_device_status() & B.ADACOMP_DEV_HEADER_MISMATCH
    assert torch.all(layer.residue == 1.0)
    B.adacomp_device_status_reset()


def test_lazy_multi_matches_oracle_over_steps_and_flags_a_foreign_state():
    """adacomp_compress_multi_lazy on a parameter list (layers and bin lengths change from tile to tile inside
    one batch; one layer beyond the batch's size limit, one with one-bin tiles): every stream equals the
    oracle's at every step, and after a flush every residue does.  Then one layer is given another layer's
    state: flagged, left untouched, its stream empty, the others unaffected."""
    specs = synth.resnet50_tensors()[:12] + [
        synth.TensorSpec("lt64", 3840 * 5 + 77, 64, "conv"), synth.TensorSpec("lt333", 3996 * 3 + 5, 333, "fc"),
        synth.TensorSpec("mid", (1 << 22) + 99, 500, "fc"), synth.TensorSpec("tiny", 17, 50, "conv"),
        synth.TensorSpec("lt1000", 4000 * 6 + 999, 1000, "fc"), synth.TensorSpec("one_bin", 3000 * 9 + 1, 3000, "fc"),
        synth.TensorSpec("alone", (1 << 25) + 3, 50, "conv")]
    layers = [LazyLayer(s.n, s.L_T) for s in specs]
    r_cpu = [np.zeros(s.n, np.float32) for s in specs]
    descs = [dict(grad=L.grad, residue=L.residue, n=L.n, L_T=L.L_T, packed_out=L.packed, count_out=L.count)
             for L in layers]
    states = [L.state for L in layers]
    for step in range(3):
        wants = []
        for t, s in enumerate(specs):
            dW = synth.make_dw(3, step, t, 1, s.n, heavy=(t % 2 == 0))
            layers[t].grad.copy_(torch.from_numpy(dW))
            wants.append(cref.pack(dW, r_cpu[t], s.L_T))
        B.adacomp_compress_multi_lazy(descs, states, len(descs))
        torch.cuda.synchronize()
        for t, L in enumerate(layers):
            assert_stream_equal(L.packed[:int(L.count[1])].cpu().numpy(), wants[t], f"step {step} tensor {t} ({specs[t].name})")
    for t, L in enumerate(layers):
        assert_f32_bits_equal(L.flushed_residue(), r_cpu[t], f"flushed residue of tensor {t}")
    assert B.adacomp_device_status() == 0

    # layer 3 gets layer 4's state
    before = [L.residue.clone() for L in layers]
    swapped = list(states)
    swapped[3] = states[4]
    wants = []
    for t, s in enumerate(specs):
        dW = synth.make_dw(3, 7, t, 1, s.n, heavy=False)
        layers[t].grad.copy_(torch.from_numpy(dW))
        wants.append(None if t == 3 else cref.pack(dW, r_cpu[t], s.L_T))
    B.adacomp_compress_multi_lazy(descs, swapped, len(descs))
    torch.cuda.synchronize()
    assert B.adacomp_device_status() & B.ADACOMP_DEV_HEADER_MISMATCH
    B.adacomp_device_status_reset()
    assert torch.equal(layers[3].residue, before[3])
    assert int(layers[3].count[0]) == 0
    for t, L in enumerate(layers):
        if t != 3:
            assert_stream_equal(L.packed[:int(L.count[1])].cpu().numpy(), wants[t], f"after the swap, tensor {t}")
    assert B.adacomp_device_status() == 0


def test_lazy_multi_with_a_single_layer_is_the_single_tensor_call():
    n, L_T = 4000 * 9 + 41, 50
    rng = np.random.default_rng(31)
    r_cpu = np.zeros(n, np.float32)
    layer = LazyLayer(n, L_T)
    desc = [dict(grad=layer.grad, residue=layer.residue, n=n, L_T=L_T, packed_out=layer.packed, count_out=layer.count)]
    for step in range(3):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        want = cref.pack(dW, r_cpu, L_T)
        layer.grad.copy_(torch.from_numpy(dW))
        B.adacomp_compress_multi_lazy(desc, [layer.state], 1)
        torch.cuda.synchronize()
        assert_stream_equal(layer.packed[:int(layer.count[1])].cpu().numpy(), want, f"step {step}")
    assert_f32_bits_equal(layer.flushed_residue(), r_cpu)
    # a bin length the lazy mode does not take: refused on the host, nothing launched
    other = LazyLayer(n, 50)
    bad = [dict(grad=other.grad, residue=other.residue, n=n, L_T=40, packed_out=other.packed, count_out=other.count)]
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_compress_multi_lazy(bad, [other.state], 1)
    assert e.value.code == -9
    assert B.adacomp_device_status() == 0
