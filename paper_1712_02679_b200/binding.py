"""Thin ctypes binding of libadacomp.so: same names as the C ABI, argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  There is no CPU
fallback: if the shared library has not been built, or a tensor is not on a
CUDA device, the call raises.  PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libadacomp.so")

ADACOMP_FLAG_LITERAL = 1
ADACOMP_FLAG_GENERIC_PATH = 256
ADACOMP_FLAG_STREAMING = 512
ADACOMP_MAX_STREAMS = 64

ADACOMP_DEV_NONFINITE = 1
ADACOMP_DEV_HEADER_MISMATCH = 2
ADACOMP_DEV_RESERVED_CODE = 4
ADACOMP_DEV_TIMEOUT = 8
ADACOMP_DEV_BAD_STREAM = 16


class AdaCompError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what} failed: {code} ({adacomp_strerror(code)})")
        self.code = code


class adacomp_layer_desc(C.Structure):
    _fields_ = [("grad", C.c_void_p), ("residue", C.c_void_p), ("n", C.c_uint64),
                ("L_T", C.c_uint32), ("flags", C.c_uint32), ("packed_out", C.c_void_p),
                ("count_out", C.c_void_p)]


class adacomp_options(C.Structure):
    _fields_ = [("flags", C.c_uint32), ("grad_type", C.c_uint32), ("factor", C.c_float), ("quantiser", C.c_uint32),
                ("lazy_state", C.c_void_p)]


ADACOMP_GRAD_F32, ADACOMP_GRAD_BF16, ADACOMP_GRAD_F16 = 0, 1, 2
ADACOMP_QUANT_BIN_MAX_MEAN, ADACOMP_QUANT_SENT_MEAN = 0, 1
_GRAD_DTYPES = {ADACOMP_GRAD_F32: torch.float32, ADACOMP_GRAD_BF16: torch.bfloat16, ADACOMP_GRAD_F16: torch.float16}

_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1712_02679_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.adacomp_version.restype = C.c_int
        L.adacomp_strerror.restype = C.c_char_p
        L.adacomp_strerror.argtypes = [C.c_int]
        L.adacomp_packed_capacity.restype = C.c_size_t
        L.adacomp_packed_capacity.argtypes = [C.c_uint64, C.c_uint32]
        L.adacomp_compress.restype = C.c_int
        L.adacomp_compress.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p,
                                       C.c_void_p, C.c_void_p]
        L.adacomp_compress_static.restype = C.c_int
        L.adacomp_compress_static.argtypes = L.adacomp_compress.argtypes
        L.adacomp_compress_ex.restype = C.c_int
        L.adacomp_compress_ex.argtypes = L.adacomp_compress.argtypes + [C.c_uint32]
        L.adacomp_decompress_accumulate.restype = C.c_int
        L.adacomp_decompress_accumulate.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.adacomp_decompress_accumulate_ex.restype = C.c_int
        L.adacomp_decompress_accumulate_ex.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint64,
                                                       C.c_uint32, C.c_void_p]
        L.adacomp_decompress_average_sgd_multi.restype = C.c_int
        L.adacomp_decompress_average_sgd_multi.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                                           C.c_void_p, C.c_uint32, C.c_float, C.c_float, C.c_void_p]
        L.adacomp_decompress_average_adam.restype = C.c_int
        L.adacomp_decompress_average_adam.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                                      C.c_uint32, C.c_float, C.c_float, C.c_float, C.c_float, C.c_void_p]
        L.adacomp_decompress_average_adam_multi.restype = C.c_int
        L.adacomp_decompress_average_adam_multi.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p,
                                                            C.c_void_p, C.c_void_p, C.c_uint32, C.c_float, C.c_float,
                                                            C.c_float, C.c_float, C.c_void_p]
        L.adacomp_compress_f16.restype = C.c_int
        L.adacomp_compress_f16.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p,
                                           C.c_void_p]
        L.adacomp_compress_multi_opt.restype = C.c_int
        L.adacomp_compress_multi_opt.argtypes = [C.POINTER(adacomp_layer_desc), C.POINTER(adacomp_options), C.c_uint32,
                                                 C.c_void_p]
        L.adacomp_compress_opt.restype = C.c_int
        L.adacomp_compress_opt.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p,
                                           C.POINTER(adacomp_options), C.c_void_p]
        L.adacomp_compress_bf16.restype = C.c_int
        L.adacomp_compress_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p,
                                            C.c_void_p]
        L.adacomp_compress_scaled.restype = C.c_int
        L.adacomp_compress_scaled.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p,
                                              C.c_void_p, C.c_float]
        L.adacomp_decompress_average_sgd.restype = C.c_int
        L.adacomp_decompress_average_sgd.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_uint64,
                                                     C.c_uint32, C.c_float, C.c_float, C.c_void_p]
        L.adacomp_decompress_accumulate_multi_ex.restype = C.c_int
        L.adacomp_decompress_accumulate_multi_ex.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                                             C.c_void_p, C.c_uint32, C.c_void_p]
        L.adacomp_compress_profile.restype = C.c_int
        L.adacomp_compress_profile.argtypes = L.adacomp_compress_ex.argtypes + [C.c_void_p, C.c_void_p]
        L.adacomp_lazy_state_bytes.restype = C.c_size_t
        L.adacomp_lazy_state_bytes.argtypes = [C.c_uint64, C.c_uint32]
        L.adacomp_lazy_state_init.restype = C.c_int
        L.adacomp_lazy_state_init.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p]
        L.adacomp_compress_lazy.restype = C.c_int
        L.adacomp_compress_lazy.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32,
                                            C.c_void_p, C.c_void_p, C.c_void_p]
        L.adacomp_residue_flush.restype = C.c_int
        L.adacomp_residue_flush.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p]
        L.adacomp_compress_host.restype = C.c_int
        L.adacomp_compress_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32,
                                            C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                            C.c_void_p, C.c_void_p]
        L.adacomp_decompress_accumulate_host.restype = C.c_int
        L.adacomp_decompress_accumulate_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p,
                                                         C.c_uint32, C.c_void_p, C.c_void_p,
                                                         C.c_uint64, C.c_void_p]
        L.adacomp_compress_multi.restype = C.c_int
        L.adacomp_compress_multi.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p]
        L.adacomp_compress_multi_lazy.restype = C.c_int
        L.adacomp_compress_multi_lazy.argtypes = [C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p]
        L.adacomp_decompress_accumulate_multi.restype = C.c_int
        L.adacomp_decompress_accumulate_multi.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p,
                                                          C.c_uint32, C.c_void_p]
        L.adacomp_set_device.restype = C.c_int
        L.adacomp_set_device.argtypes = [C.c_int]
        L.adacomp_device_status.restype = C.c_int
        L.adacomp_device_status.argtypes = [C.c_void_p, C.c_void_p]
        L.adacomp_device_status_reset.restype = C.c_int
        L.adacomp_device_status_reset.argtypes = [C.c_void_p]
        _lib = L
    return _lib


def _dev_ptr(t: Optional[torch.Tensor], what: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{what} must be a CUDA tensor (no CPU path exists)")
    if not t.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{what} must have dtype {dtype}")
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise AdaCompError(rc, what)


def adacomp_version() -> int:
    return int(lib().adacomp_version())


def adacomp_strerror(code: int) -> str:
    return lib().adacomp_strerror(int(code)).decode()


def adacomp_packed_capacity(n: int, L_T: int) -> int:
    return int(lib().adacomp_packed_capacity(int(n), int(L_T)))


def adacomp_compress(grad, residue, n: int, L_T: int, packed_out, count_out, stream=None) -> None:
    """pack(): see include/adacomp.h.  count_out is an int64[2] CUDA tensor."""
    _check(lib().adacomp_compress(_dev_ptr(grad, "grad", torch.float32),
                                  _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                  _dev_ptr(packed_out, "packed_out", torch.uint8),
                                  _dev_ptr(count_out, "count_out", torch.int64), _stream(stream)),
           "adacomp_compress")


def adacomp_compress_static(grad, residue, n: int, L_T: int, packed_out, count_out,
                            stream=None) -> None:
    """pack() for callers that may not allocate device memory: same results as
    adacomp_compress, but the compressor's scratch is an 8 MiB array built into the library,
    so packed_out only has to hold the stream.  Tensors that need more scratch raise
    AdaCompError(-8).  Calls that overlap on the GPU share (and would corrupt) that array."""
    _check(lib().adacomp_compress_static(_dev_ptr(grad, "grad", torch.float32),
                                         _dev_ptr(residue, "residue", torch.float32), int(n),
                                         int(L_T), _dev_ptr(packed_out, "packed_out", torch.uint8),
                                         _dev_ptr(count_out, "count_out", torch.int64),
                                         _stream(stream)),
           "adacomp_compress_static")


def adacomp_compress_ex(grad, residue, n: int, L_T: int, packed_out, count_out, stream=None,
                        flags: int = 0) -> None:
    _check(lib().adacomp_compress_ex(_dev_ptr(grad, "grad", torch.float32),
                                     _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                     _dev_ptr(packed_out, "packed_out", torch.uint8),
                                     _dev_ptr(count_out, "count_out", torch.int64), _stream(stream),
                                     int(flags)),
           "adacomp_compress_ex")


def adacomp_compress_bf16(grad_bf16, residue, n: int, L_T: int, packed_out, count_out, stream=None) -> None:
    """pack() of a bfloat16 gradient (widened exactly on load); residue and stream as for a binary32 gradient."""
    _check(lib().adacomp_compress_bf16(_dev_ptr(grad_bf16, "grad_bf16", torch.bfloat16),
                                       _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                       _dev_ptr(packed_out, "packed_out", torch.uint8),
                                       _dev_ptr(count_out, "count_out", torch.int64), _stream(stream)),
           "adacomp_compress_bf16")


def adacomp_compress_f16(grad_f16, residue, n: int, L_T: int, packed_out, count_out, stream=None) -> None:
    """pack() of a binary16 gradient (widened exactly on load); residue and stream as for a binary32 gradient."""
    _check(lib().adacomp_compress_f16(_dev_ptr(grad_f16, "grad_f16", torch.float16),
                                      _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                      _dev_ptr(packed_out, "packed_out", torch.uint8),
                                      _dev_ptr(count_out, "count_out", torch.int64), _stream(stream)),
           "adacomp_compress_f16")


def adacomp_compress_opt(grad, residue, n: int, L_T: int, packed_out, count_out, flags: int = 0,
                         grad_type: int = ADACOMP_GRAD_F32, factor: float = 0.0, lazy_state=None, quantiser: int = 0,
                         stream=None) -> None:
    """pack() with every option at once (flags, gradient format, the selection's factor, quantiser, lazy-scale state)."""
    opt = adacomp_options(int(flags), int(grad_type), float(factor), int(quantiser),
                          _dev_ptr(lazy_state, "lazy_state", torch.uint8) if lazy_state is not None else None)
    _check(lib().adacomp_compress_opt(_dev_ptr(grad, "grad", _GRAD_DTYPES.get(int(grad_type))),
                                      _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                      _dev_ptr(packed_out, "packed_out", torch.uint8),
                                      _dev_ptr(count_out, "count_out", torch.int64), C.byref(opt), _stream(stream)),
           "adacomp_compress_opt")


def adacomp_compress_scaled(grad, residue, n: int, L_T: int, packed_out, count_out, factor: float, stream=None) -> None:
    """pack() with the selection's scale-factor: H = residue + factor * dW (factor 1: bin maxima only)."""
    _check(lib().adacomp_compress_scaled(_dev_ptr(grad, "grad", torch.float32), _dev_ptr(residue, "residue", torch.float32),
                                         int(n), int(L_T), _dev_ptr(packed_out, "packed_out", torch.uint8),
                                         _dev_ptr(count_out, "count_out", torch.int64), _stream(stream), C.c_float(factor)),
           "adacomp_compress_scaled")


def adacomp_decompress_accumulate(packed: Sequence[torch.Tensor], k_streams: int, dst,
                                  stream=None) -> None:
    """unpack()-and-sum of k streams into dst (fully overwritten)."""
    ptrs = (C.c_void_p * max(int(k_streams), 1))(
        *[_dev_ptr(p, "packed[l]", torch.uint8) for p in packed[:k_streams]])
    _check(lib().adacomp_decompress_accumulate(ptrs, int(k_streams),
                                               _dev_ptr(dst, "dst", torch.float32), _stream(stream)),
           "adacomp_decompress_accumulate")


def adacomp_decompress_accumulate_ex(packed: Sequence[torch.Tensor], k_streams: int, dst, n: int,
                                     L_T: int, stream=None) -> None:
    """unpack()-and-sum when the caller knows (n, L_T): the grid is sized to the tensor."""
    ptrs = (C.c_void_p * max(int(k_streams), 1))(
        *[_dev_ptr(p, "packed[l]", torch.uint8) for p in packed[:k_streams]])
    _check(lib().adacomp_decompress_accumulate_ex(ptrs, int(k_streams), _dev_ptr(dst, "dst", torch.float32),
                                                  int(n), int(L_T), _stream(stream)),
           "adacomp_decompress_accumulate_ex")


def adacomp_decompress_average_sgd(packed: Sequence[torch.Tensor], k_streams: int, weights, momentum, n: int,
                                   L_T: int, lr: float, mu: float, stream=None) -> None:
    """unpack(), averageGradients() and updateWeights() (SGD with momentum) in one pass; weights and
    momentum are updated in place."""
    ptrs = (C.c_void_p * max(int(k_streams), 1))(
        *[_dev_ptr(p, "packed[l]", torch.uint8) for p in packed[:k_streams]])
    _check(lib().adacomp_decompress_average_sgd(ptrs, int(k_streams), _dev_ptr(weights, "weights", torch.float32),
                                                _dev_ptr(momentum, "momentum", torch.float32), int(n), int(L_T),
                                                C.c_float(lr), C.c_float(mu), _stream(stream)),
           "adacomp_decompress_average_sgd")


def adacomp_decompress_average_adam(packed: Sequence[torch.Tensor], k_streams: int, weights, m, v, n: int, L_T: int,
                                    step_size: float, beta1: float, beta2: float, eps: float, stream=None) -> None:
    """unpack(), averageGradients() and an Adam step in one pass; weights, m and v are updated in place."""
    ptrs = (C.c_void_p * max(int(k_streams), 1))(
        *[_dev_ptr(p, "packed[l]", torch.uint8) for p in packed[:k_streams]])
    _check(lib().adacomp_decompress_average_adam(ptrs, int(k_streams), _dev_ptr(weights, "weights", torch.float32),
                                                 _dev_ptr(m, "m", torch.float32), _dev_ptr(v, "v", torch.float32),
                                                 int(n), int(L_T), C.c_float(step_size), C.c_float(beta1),
                                                 C.c_float(beta2), C.c_float(eps), _stream(stream)),
           "adacomp_decompress_average_adam")


def adacomp_decompress_average_adam_multi(packed, k_streams: int, weights, m, v, n: Sequence[int], L_T: Sequence[int],
                                          n_layers: int, step_size: float, beta1: float, beta2: float, eps: float,
                                          stream=None) -> None:
    """adacomp_decompress_average_adam for a list of layers."""
    if not isinstance(packed, C.Array):
        packed = make_pointer_array(packed, torch.uint8)
    arrs = [a if isinstance(a, C.Array) else make_pointer_array(a, torch.float32) for a in (weights, m, v)]
    ns = (C.c_uint64 * max(int(n_layers), 1))(*[int(x) for x in n[:n_layers]])
    lts = (C.c_uint32 * max(int(n_layers), 1))(*[int(x) for x in L_T[:n_layers]])
    _check(lib().adacomp_decompress_average_adam_multi(packed, int(k_streams), arrs[0], arrs[1], arrs[2], ns, lts,
                                                       int(n_layers), C.c_float(step_size), C.c_float(beta1),
                                                       C.c_float(beta2), C.c_float(eps), _stream(stream)),
           "adacomp_decompress_average_adam_multi")


def adacomp_decompress_average_sgd_multi(packed, k_streams: int, weights, momentum, n: Sequence[int],
                                         L_T: Sequence[int], n_layers: int, lr: float, mu: float, stream=None) -> None:
    """adacomp_decompress_average_sgd for a list of layers; weights[t] and momentum[t] are updated in place."""
    if not isinstance(packed, C.Array):
        packed = make_pointer_array(packed, torch.uint8)
    if not isinstance(weights, C.Array):
        weights = make_pointer_array(weights, torch.float32)
    if not isinstance(momentum, C.Array):
        momentum = make_pointer_array(momentum, torch.float32)
    ns = (C.c_uint64 * max(int(n_layers), 1))(*[int(v) for v in n[:n_layers]])
    lts = (C.c_uint32 * max(int(n_layers), 1))(*[int(v) for v in L_T[:n_layers]])
    _check(lib().adacomp_decompress_average_sgd_multi(packed, int(k_streams), weights, momentum, ns, lts, int(n_layers),
                                                      C.c_float(lr), C.c_float(mu), _stream(stream)),
           "adacomp_decompress_average_sgd_multi")


def adacomp_decompress_accumulate_multi_ex(packed, k_streams: int, dst, n: Sequence[int],
                                           L_T: Sequence[int], n_layers: int, stream=None) -> None:
    """adacomp_decompress_accumulate_multi with the layers' shapes known on the host."""
    if not isinstance(packed, C.Array):
        packed = make_pointer_array(packed, torch.uint8)
    if not isinstance(dst, C.Array):
        dst = make_pointer_array(dst, torch.float32)
    ns = (C.c_uint64 * max(int(n_layers), 1))(*[int(v) for v in n[:n_layers]])
    lts = (C.c_uint32 * max(int(n_layers), 1))(*[int(v) for v in L_T[:n_layers]])
    _check(lib().adacomp_decompress_accumulate_multi_ex(packed, int(k_streams), dst, ns, lts, int(n_layers),
                                                        _stream(stream)),
           "adacomp_decompress_accumulate_multi_ex")


def adacomp_lazy_state_bytes(n: int, L_T: int) -> int:
    return int(lib().adacomp_lazy_state_bytes(int(n), int(L_T)))


def adacomp_lazy_state_init(state, n: int, L_T: int, stream=None) -> None:
    _check(lib().adacomp_lazy_state_init(_dev_ptr(state, "state", torch.uint8), int(n), int(L_T),
                                         _stream(stream)), "adacomp_lazy_state_init")


def adacomp_compress_lazy(grad, residue, state, n: int, L_T: int, packed_out, count_out,
                          stream=None) -> None:
    """Lazy-scale pack(): same stream as adacomp_compress; `residue` keeps G until the next
    call or adacomp_residue_flush (see include/adacomp.h)."""
    _check(lib().adacomp_compress_lazy(_dev_ptr(grad, "grad", torch.float32),
                                       _dev_ptr(residue, "residue", torch.float32),
                                       _dev_ptr(state, "state", torch.uint8), int(n), int(L_T),
                                       _dev_ptr(packed_out, "packed_out", torch.uint8),
                                       _dev_ptr(count_out, "count_out", torch.int64), _stream(stream)),
           "adacomp_compress_lazy")


def adacomp_residue_flush(residue, state, n: int, L_T: int, stream=None) -> None:
    _check(lib().adacomp_residue_flush(_dev_ptr(residue, "residue", torch.float32),
                                       _dev_ptr(state, "state", torch.uint8), int(n), int(L_T),
                                       _stream(stream)), "adacomp_residue_flush")


def adacomp_compress_profile(grad, residue, n: int, L_T: int, packed_out, count_out, stream=None,
                             flags: int = 0, events: Sequence[torch.cuda.Event] = (),
                             lazy_state=None) -> None:
    """adacomp_compress_ex (or, with lazy_state, adacomp_compress_lazy) with four torch CUDA
    events (already recorded once, so that their handles exist) recorded around the three kernels."""
    assert len(events) == 4
    handles = (C.c_void_p * 4)(*[int(e.cuda_event) for e in events])
    _check(lib().adacomp_compress_profile(_dev_ptr(grad, "grad", torch.float32),
                                          _dev_ptr(residue, "residue", torch.float32), int(n),
                                          int(L_T), _dev_ptr(packed_out, "packed_out", torch.uint8),
                                          _dev_ptr(count_out, "count_out", torch.int64),
                                          _stream(stream), int(flags), handles,
                                          _dev_ptr(lazy_state, "lazy_state", torch.uint8)),
           "adacomp_compress_profile")


def _host_ptr(t: torch.Tensor, what: str, dtype) -> int:
    if t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
        raise ValueError(f"{what} must be a contiguous host tensor of dtype {dtype}")
    return t.data_ptr()


def adacomp_compress_host(grad_host, grad_stage, residue, n: int, L_T: int, packed_dev, count_dev,
                          packed_host, count_host, stream=None) -> None:
    """pack() of a host-resident gradient; synchronises.  count_host: int64[2] host tensor."""
    _check(lib().adacomp_compress_host(_host_ptr(grad_host, "grad_host", torch.float32),
                                       _dev_ptr(grad_stage, "grad_stage", torch.float32),
                                       _dev_ptr(residue, "residue", torch.float32), int(n), int(L_T),
                                       _dev_ptr(packed_dev, "packed_dev", torch.uint8),
                                       _dev_ptr(count_dev, "count_dev", torch.int64),
                                       _host_ptr(packed_host, "packed_host", torch.uint8),
                                       packed_host.numel(),
                                       _host_ptr(count_host, "count_host", torch.int64),
                                       _stream(stream)),
           "adacomp_compress_host")


def adacomp_decompress_accumulate_host(packed_host: Sequence[torch.Tensor],
                                       packed_bytes: Sequence[int],
                                       packed_stage: Sequence[torch.Tensor], k_streams: int,
                                       dst_dev, dst_host, n: int, stream=None) -> None:
    """unpack()-and-sum of host-resident streams into dst_host; synchronises."""
    k = int(k_streams)
    hp = (C.c_void_p * max(k, 1))(*[_host_ptr(p, "packed_host[l]", torch.uint8) for p in packed_host[:k]])
    nb = (C.c_uint64 * max(k, 1))(*[int(b) for b in packed_bytes[:k]])
    sp = (C.c_void_p * max(k, 1))(*[_dev_ptr(p, "packed_stage[l]", torch.uint8) for p in packed_stage[:k]])
    _check(lib().adacomp_decompress_accumulate_host(hp, nb, sp, k, _dev_ptr(dst_dev, "dst_dev", torch.float32),
                                                    _host_ptr(dst_host, "dst_host", torch.float32),
                                                    int(n), _stream(stream)),
           "adacomp_decompress_accumulate_host")


def make_layer_descs(layers: Sequence[dict]):
    """HOST array of adacomp_layer_desc from dicts with the struct's field names."""
    arr = (adacomp_layer_desc * max(len(layers), 1))()
    for i, d in enumerate(layers):
        arr[i].grad = _dev_ptr(d["grad"], "grad", _GRAD_DTYPES.get(int(d.get("grad_type", 0))))
        arr[i].residue = _dev_ptr(d["residue"], "residue", torch.float32)
        arr[i].n = int(d["n"])
        arr[i].L_T = int(d["L_T"])
        arr[i].flags = int(d.get("flags", 0))
        arr[i].packed_out = _dev_ptr(d["packed_out"], "packed_out", torch.uint8)
        arr[i].count_out = _dev_ptr(d["count_out"], "count_out", torch.int64)
    return arr


def adacomp_compress_multi(layers, n_layers: int, stream=None) -> None:
    """layers: a ctypes array from make_layer_descs (or a list of dicts)."""
    if not isinstance(layers, C.Array):
        layers = make_layer_descs(layers)
    _check(lib().adacomp_compress_multi(layers, int(n_layers), _stream(stream)),
           "adacomp_compress_multi")


def adacomp_compress_multi_lazy(layers, states, n_layers: int, stream=None) -> None:
    """adacomp_compress_multi in lazy-scale mode; states[t]: layer t's lazy state (uint8 CUDA tensors)."""
    if not isinstance(layers, C.Array):
        layers = make_layer_descs(layers)
    if not isinstance(states, C.Array):
        states = make_pointer_array(states, torch.uint8)
    _check(lib().adacomp_compress_multi_lazy(layers, states, int(n_layers), _stream(stream)),
           "adacomp_compress_multi_lazy")


def adacomp_compress_multi_opt(layers: Sequence[dict], n_layers: int, stream=None) -> None:
    """layers: dicts with the descriptor's fields and, optionally, grad_type, factor and lazy_state."""
    descs = make_layer_descs(layers)
    opts = (adacomp_options * max(len(layers), 1))()
    for i, d in enumerate(layers):
        st = d.get("lazy_state")
        opts[i] = adacomp_options(0, int(d.get("grad_type", 0)), float(d.get("factor", 0.0)), int(d.get("quantiser", 0)),
                                  _dev_ptr(st, "lazy_state", torch.uint8) if st is not None else None)
    _check(lib().adacomp_compress_multi_opt(descs, opts, int(n_layers), _stream(stream)), "adacomp_compress_multi_opt")


def make_pointer_array(tensors: Sequence[torch.Tensor], dtype):
    return (C.c_void_p * max(len(tensors), 1))(*[_dev_ptr(t, "tensor", dtype) for t in tensors])


def adacomp_decompress_accumulate_multi(packed, k_streams: int, dst, n_layers: int,
                                        stream=None) -> None:
    """packed[t * k_streams + l]: learner l's stream of layer t; dst[t]: its output."""
    if not isinstance(packed, C.Array):
        packed = make_pointer_array(packed, torch.uint8)
    if not isinstance(dst, C.Array):
        dst = make_pointer_array(dst, torch.float32)
    _check(lib().adacomp_decompress_accumulate_multi(packed, int(k_streams), dst, int(n_layers),
                                                     _stream(stream)),
           "adacomp_decompress_accumulate_multi")


def adacomp_set_device(device: int) -> None:
    """Select the calling thread's CUDA device inside the library (see include/adacomp.h)."""
    _check(lib().adacomp_set_device(int(device)), "adacomp_set_device")


def adacomp_device_status(stream=None) -> int:
    out = C.c_uint32(0)
    _check(lib().adacomp_device_status(C.byref(out), _stream(stream)), "adacomp_device_status")
    return int(out.value)


def adacomp_v2_capacity(n: int, L_T: int) -> int:
    f = lib().adacomp_v2_capacity
    f.restype, f.argtypes = C.c_size_t, [C.c_uint64, C.c_uint32]
    return int(f(int(n), int(L_T)))


def adacomp_stream_to_v2(packed, out_v2, count_out, n: int, L_T: int, stream=None) -> None:
    """A version-1 stream re-encoded as version 2 (first-of-bin flags, no counts): the form for the wire."""
    f = lib().adacomp_stream_to_v2
    f.restype = C.c_int
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p]
    _check(f(_dev_ptr(packed, "packed", torch.uint8), _dev_ptr(out_v2, "out_v2", torch.uint8), int(out_v2.numel()),
             _dev_ptr(count_out, "count_out", torch.int64) if count_out is not None else None, int(n), int(L_T),
             _stream(stream)), "adacomp_stream_to_v2")


def adacomp_stream_from_v2(in_v2, packed_out, n: int, L_T: int, stream=None) -> None:
    """A version-2 stream re-encoded as version 1, which the decoders read."""
    f = lib().adacomp_stream_from_v2
    f.restype = C.c_int
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint32, C.c_void_p]
    _check(f(_dev_ptr(in_v2, "in_v2", torch.uint8), _dev_ptr(packed_out, "packed_out", torch.uint8),
             int(packed_out.numel()), int(n), int(L_T), _stream(stream)), "adacomp_stream_from_v2")


def adacomp_debug_waits(wait_cycles: int = 0, withhold_pack_tile: int = 0, withhold_decode_item: int = 0) -> None:
    """Testing aid: the limit of the device-side waits and one withheld copy (see include/adacomp.h)."""
    f = lib().adacomp_debug_waits
    f.restype, f.argtypes = C.c_int, [C.c_uint64, C.c_uint32, C.c_uint32]
    _check(f(int(wait_cycles), int(withhold_pack_tile), int(withhold_decode_item)), "adacomp_debug_waits")


def adacomp_device_status_reset(stream=None) -> None:
    _check(lib().adacomp_device_status_reset(_stream(stream)), "adacomp_device_status_reset")
