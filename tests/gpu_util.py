"""Helpers for the GPU parity tests: run the C-ABI path on numpy inputs."""
import numpy as np
import torch

from paper_1712_02679_b200 import binding as B


class GpuLayer:
    """One learner's state for one layer: residue on the device plus a packed buffer."""

    def __init__(self, n, L_T, residue=None):
        self.n, self.L_T = n, L_T
        dev = torch.device("cuda:0")
        self.residue = torch.zeros(max(n, 4), dtype=torch.float32, device=dev)
        if residue is not None and n:
            self.residue[:n].copy_(torch.from_numpy(residue))
        self.cap = B.adacomp_packed_capacity(n, L_T)
        self.packed = torch.empty(self.cap, dtype=torch.uint8, device=dev)
        self.count = torch.zeros(2, dtype=torch.int64, device=dev)
        self.grad = torch.zeros(max(n, 4), dtype=torch.float32, device=dev)

    def compress(self, dW, flags=0, poison=True):
        if self.n:
            self.grad[:self.n].copy_(torch.from_numpy(np.ascontiguousarray(dW)))
        if poison:
            self.packed.fill_(0xAB)          # stale bytes must never leak into the stream
        if flags:
            B.adacomp_compress_ex(self.grad, self.residue, self.n, self.L_T, self.packed,
                                  self.count, None, flags)
        else:
            B.adacomp_compress(self.grad, self.residue, self.n, self.L_T, self.packed, self.count)
        torch.cuda.synchronize()
        n_sel, used = (int(v) for v in self.count.cpu())
        raw = self.packed[:used].cpu().numpy()
        return raw, n_sel, used

    def residue_host(self):
        return self.residue[:self.n].cpu().numpy()


def assert_stream_equal(raw, oracle_packed, what=""):
    """Bit-exact: header (scale, counts), directory, bin counts, words, padding."""
    want = oracle_packed.raw
    assert raw.size == want.size, f"{what}: bytes_used {raw.size} != {want.size}"
    if not np.array_equal(raw, want):
        at = int(np.flatnonzero(raw != want)[0])
        raise AssertionError(f"{what}: first differing byte at {at} "
                             f"(gpu {raw[at]:#x}, oracle {want[at]:#x}) of {want.size}")


def assert_f32_bits_equal(a, b, what=""):
    a = np.ascontiguousarray(a, np.float32).view(np.uint32)
    b = np.ascontiguousarray(b, np.float32).view(np.uint32)
    if not np.array_equal(a, b):
        at = int(np.flatnonzero(a != b)[0])
        raise AssertionError(f"{what}: {np.count_nonzero(a != b)} words differ, first at {at}: "
                             f"{a[at]:#x} vs {b[at]:#x}")
