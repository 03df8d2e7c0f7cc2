"""The C-ABI library loads without a GPU, exports what include/adacomp.h declares,
and rejects bad arguments on the host before touching CUDA.  CPU only."""
import ctypes as C
import os
import re

import pytest

from oracle import cref
from paper_1712_02679_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "adacomp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(adacomp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"adacomp_compress", "adacomp_decompress_accumulate", "adacomp_packed_capacity",
            "adacomp_device_status"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_has_the_same_names():
    for name in declared_functions():
        assert callable(getattr(binding, name)), name


def test_version_and_error_text(lib):
    assert binding.adacomp_version() == 1
    assert binding.adacomp_strerror(0) == "ok"
    texts = {binding.adacomp_strerror(c) for c in range(-7, 0)}
    assert len(texts) == 7 and "unknown error code" not in texts
    assert binding.adacomp_strerror(-99) == "unknown error code"


@pytest.mark.parametrize("n,L_T", [(0, 50), (1, 1), (100352, 50), (864, 500), (10 ** 6, 64),
                                   (10 ** 6, 65), (12345, 1001), (99999, 16384), (1 << 30, 50)])
def test_capacity_covers_the_worst_case_stream(n, L_T):
    cap = binding.adacomp_packed_capacity(n, L_T)
    assert cap % 16 == 0
    # every element sent: the stream itself must fit with room for the scratch behind it
    assert cap >= cref.stream_bytes(n, L_T, n)
    w = 1 if L_T <= 64 else 2
    assert cap <= 64 + 3 * n * w + n // 100 + 70000   # not wildly oversized either


def test_capacity_of_invalid_bin_length_is_zero():
    assert binding.adacomp_packed_capacity(100, 0) == 0
    assert binding.adacomp_packed_capacity(100, 16385) == 0


def test_host_side_argument_checks_need_no_gpu(lib):
    A = 0x1000          # fake, 16-byte aligned, never dereferenced: the checks come first
    f = lib.adacomp_compress
    assert f(None, A, 10, 50, A, A, None) == -1
    assert f(A, A, 10, 50, None, A, None) == -1
    assert f(A, A, 10, 50, A, None, None) == -1
    assert f(A, A, 10, 0, A, A, None) == -2
    assert f(A, A, 10, 16385, A, A, None) == -2
    assert f(A + 4, A, 10, 50, A, A, None) == -3
    assert f(A, A + 8, 10, 50, A, A, None) == -3
    assert f(A, A, 10, 50, A + 1, A, None) == -3
    assert f(A, A, 1 << 40, 1, A, A, None) == -5
    assert lib.adacomp_compress_ex(A, A, 10, 50, A, A, None, 2) == -6
    g = lib.adacomp_decompress_accumulate
    ptrs = (C.c_void_p * 2)(A, A)
    assert g(None, 1, A, None) == -1
    assert g(ptrs, 2, None, None) == -1
    assert g(ptrs, 0, A, None) == -4
    assert g(ptrs, 65, A, None) == -4
    bad = (C.c_void_p * 2)(A, None)
    assert g(bad, 2, A, None) == -1
    odd = (C.c_void_p * 1)(A + 2)
    assert g(odd, 1, A, None) == -3
    assert g(ptrs, 2, A + 4, None) == -3
    um = lib.adacomp_decompress_average_sgd_multi
    lr, mu = C.c_float(0.1), C.c_float(0.9)
    one64, one32 = (C.c_uint64 * 1)(10), (C.c_uint32 * 1)(50)
    wl, bad_w = (C.c_void_p * 1)(A), (C.c_void_p * 1)(A + 4)
    assert um(ptrs, 2, wl, None, one64, one32, 1, lr, mu, None) == -1
    assert um(ptrs, 2, bad_w, wl, one64, one32, 1, lr, mu, None) == -3
    assert um(ptrs, 2, wl, wl, one64, (C.c_uint32 * 1)(0), 1, lr, mu, None) == -2
    assert um(None, 2, None, None, None, None, 0, lr, mu, None) == 0
    ad = lib.adacomp_decompress_average_adam
    hy = (C.c_float(1e-3), C.c_float(0.9), C.c_float(0.999), C.c_float(1e-8))
    assert ad(ptrs, 2, A, A, None, 10, 50, *hy, None) == -1
    assert ad(ptrs, 2, A, A, A + 4, 10, 50, *hy, None) == -3
    assert ad(ptrs, 2, A, A, A, 10, 0, *hy, None) == -2
    assert ad(ptrs, 65, A, A, A, 10, 50, *hy, None) == -4
    assert lib.adacomp_decompress_average_adam_multi(ptrs, 2, wl, wl, None, one64, one32, 1, *hy, None) == -1
    hb = lib.adacomp_compress_bf16
    assert hb(None, A, 10, 50, A, A, None) == -1
    assert hb(A, A, 10, 0, A, A, None) == -2
    assert hb(A + 2, A, 10, 50, A, A, None) == -3
    sc = lib.adacomp_compress_scaled
    assert sc(A, A, 10, 50, A, A, None, C.c_float(0.0)) == -6
    assert sc(A, A, 10, 50, A, A, None, C.c_float(-1.5)) == -6
    assert sc(A, A, 10, 50, A, A, None, C.c_float(float("nan"))) == -6
    assert sc(None, A, 10, 50, A, A, None, C.c_float(1.5)) == -1
    assert sc(A, A, 10, 0, A, A, None, C.c_float(1.5)) == -2
    assert sc(A + 4, A, 10, 50, A, A, None, C.c_float(1.5)) == -3
    u = lib.adacomp_decompress_average_sgd
    lr, mu = C.c_float(0.1), C.c_float(0.9)
    assert u(ptrs, 2, None, A, 10, 50, lr, mu, None) == -1
    assert u(ptrs, 2, A, None, 10, 50, lr, mu, None) == -1
    assert u(None, 2, A, A, 10, 50, lr, mu, None) == -1
    assert u(ptrs, 2, A, A, 10, 0, lr, mu, None) == -2
    assert u(ptrs, 2, A, A, 10, 16385, lr, mu, None) == -2
    assert u(ptrs, 2, A + 4, A, 10, 50, lr, mu, None) == -3
    assert u(ptrs, 2, A, A + 8, 10, 50, lr, mu, None) == -3
    assert u(ptrs, 0, A, A, 10, 50, lr, mu, None) == -4
    assert lib.adacomp_device_status(None, None) == -1
    descs = (binding.adacomp_layer_desc * 1)()
    descs[0].grad, descs[0].residue, descs[0].n, descs[0].L_T = A, A, 5, 0
    descs[0].packed_out, descs[0].count_out = A, A
    assert lib.adacomp_compress_multi(descs, 1, None) == -2
    assert lib.adacomp_compress_multi(None, 1, None) == -1
    assert lib.adacomp_compress_multi(None, 0, None) == 0
    assert lib.adacomp_compress_multi_lazy(descs, None, 1, None) == -1
    assert lib.adacomp_compress_multi_lazy(None, None, 0, None) == 0
    # a list is checked as a whole before anything is enqueued: a misaligned count_out or an oversized layer
    # anywhere in it is refused on the host
    two = (binding.adacomp_layer_desc * 2)()
    for d in two:
        d.grad, d.residue, d.n, d.L_T, d.packed_out, d.count_out = A, A, 5000, 50, A, A
    two[1].count_out = A + 4
    assert lib.adacomp_compress_multi(two, 2, None) == -3
    two[1].count_out = A
    two[1].n, two[1].L_T = 1 << 40, 1
    assert lib.adacomp_compress_multi(two, 2, None) == -5
    # the host-buffer form validates before its first copy
    ch = lib.adacomp_compress_host
    assert ch(A, A, A, 10, 0, A, A, A, 100, A, None) == -2
    assert ch(A, A + 4, A, 10, 50, A, A, A, 100, A, None) == -3
    assert ch(A, A, A, 10, 50, A, A + 4, A, 100, A, None) == -3
    assert ch(A, A, A, 10, 50, None, A, A, 100, A, None) == -1
    assert ch(A, A, A, 1 << 40, 1, A, A, A, 100, A, None) == -5


def test_binding_refuses_cpu_tensors():
    import torch
    t = torch.zeros(16)
    with pytest.raises(ValueError, match="CUDA"):
        binding.adacomp_compress(t, t, 16, 50, torch.zeros(4096, dtype=torch.uint8),
                                 torch.zeros(2, dtype=torch.int64))


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libadacomp.so"))
    with pytest.raises(ImportError, match="no CPU fallback"):
        binding.lib()
