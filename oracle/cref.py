"""ctypes front end of the C oracle, plus a reader for the stream it emits.

TEST INFRASTRUCTURE ONLY: see the package docstring.
"""
from __future__ import annotations

import ctypes as C
import struct
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.adacomp_oracle_stream_bytes.restype = C.c_uint64
        _lib.adacomp_oracle_stream_bytes.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        _lib.adacomp_oracle_exact_sum.restype = C.c_double
        _lib.adacomp_oracle_exact_sum.argtypes = [C.c_void_p, C.c_uint64]
        _lib.adacomp_oracle_pack.restype = C.c_int
        _lib.adacomp_oracle_pack.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32,
                                             C.c_uint32, C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.adacomp_oracle_pack_scaled.restype = C.c_int
        _lib.adacomp_oracle_pack_scaled.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32,
                                                    C.c_float, C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.adacomp_oracle_set_threads.restype = None
        _lib.adacomp_oracle_set_threads.argtypes = [C.c_int]
        _lib.adacomp_oracle_get_threads.restype = C.c_int
        _lib.adacomp_oracle_get_threads.argtypes = []
        _lib.adacomp_oracle_pack_general.restype = C.c_int
        _lib.adacomp_oracle_pack_general.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32,
                                                     C.c_float, C.c_uint32, C.c_void_p, C.c_uint64, C.c_void_p]
        _lib.adacomp_oracle_v2_bytes.restype = C.c_uint64
        _lib.adacomp_oracle_v2_bytes.argtypes = [C.c_uint64, C.c_uint32, C.c_uint64]
        for name in ("adacomp_oracle_to_v2", "adacomp_oracle_from_v2"):
            getattr(_lib, name).restype = C.c_int
            getattr(_lib, name).argtypes = [C.c_void_p, C.c_void_p, C.c_uint64]
        _lib.adacomp_oracle_unpack_sum_v2.restype = C.c_int
        _lib.adacomp_oracle_unpack_sum_v2.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint64]
        _lib.adacomp_oracle_unpack_sum.restype = C.c_int
        _lib.adacomp_oracle_unpack_sum.argtypes = [C.c_void_p, C.c_uint32, C.c_void_p, C.c_uint64]
    return _lib


def set_threads(threads: int) -> None:
    """Threads pack() may spread its per-element and per-bin loops over (1 unless asked: the pinned checker).
    The result does not depend on it: bins are independent and the scale's sum is exact."""
    lib().adacomp_oracle_set_threads(int(threads))


def get_threads() -> int:
    return int(lib().adacomp_oracle_get_threads())


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def stream_bytes(n: int, L_T: int, n_sel: int) -> int:
    return int(lib().adacomp_oracle_stream_bytes(n, L_T, n_sel))


def exact_sum(values: np.ndarray) -> float:
    """Correctly rounded (to double) exact sum of non-negative float32 values."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    return float(lib().adacomp_oracle_exact_sum(_ptr(v), v.size))


@dataclass
class Packed:
    """A parsed stream (Section 'Experiment Results': sparse-indexed words)."""

    raw: np.ndarray          # uint8, exactly bytes_used long
    n: int
    L_T: int
    w: int
    flags: int
    tile_bins: int
    n_bins: int
    n_tiles: int
    n_sel: int
    scale: np.float32
    scale_bits: int
    bytes_used: int
    tile_off: np.ndarray     # uint64[n_tiles+1]
    bin_cnt: np.ndarray      # uint8/uint16[n_bins]
    words: np.ndarray        # uint8/uint16[n_sel]
    g_max: Optional[np.ndarray] = None

    def positions_and_codes(self):
        """Flat element index and ternary code of every word, in stream order."""
        bins = np.repeat(np.arange(self.n_bins, dtype=np.int64), self.bin_cnt.astype(np.int64))
        idx = (self.words.astype(np.int64) >> 2)
        return bins * self.L_T + idx, (self.words.astype(np.int64) & 3)


def parse(raw: np.ndarray) -> Packed:
    raw = np.ascontiguousarray(raw, dtype=np.uint8)
    (magic, version, w, flags, L_T, tile_bins, n, n_bins, n_tiles, n_sel, scale_bits, _rsv,
     bytes_used) = struct.unpack_from("<IHBBIIQQQQIIQ", raw.tobytes()[:64])
    assert magic == 0x31434441 and version == 1, (hex(magic), version)
    tile_off_at = 64
    bin_cnt_at = (tile_off_at + 8 * (n_tiles + 1) + 15) & ~15
    payload_at = (bin_cnt_at + n_bins * w + 15) & ~15
    dt = np.uint8 if w == 1 else np.dtype("<u2")
    tile_off = np.frombuffer(raw, dtype="<u8", count=n_tiles + 1, offset=tile_off_at).copy()
    bin_cnt = np.frombuffer(raw, dtype=dt, count=n_bins, offset=bin_cnt_at).copy()
    words = np.frombuffer(raw, dtype=dt, count=n_sel, offset=payload_at).copy()
    scale = np.frombuffer(struct.pack("<I", scale_bits), dtype=np.float32)[0]
    return Packed(raw[:bytes_used].copy(), n, L_T, w, flags, tile_bins, n_bins, n_tiles, n_sel,
                  scale, scale_bits, bytes_used, tile_off, bin_cnt, words)


def pack(dW: np.ndarray, residue: np.ndarray, L_T: int, flags: int = 0,
         want_gmax: bool = False, factor: float = 0.0, quantiser: int = 0) -> Packed:
    """Run Algorithm 2 on one layer.  `residue` (float32, contiguous) is updated in place.
    `factor` (0: the paper's H = G + dW) selects H = residue + factor * dW, `quantiser` (0: the paper's mean of
    the bin maxima) the layer's reconstruction value, see the C source."""
    assert dW.dtype == np.float32 and residue.dtype == np.float32
    assert dW.flags.c_contiguous and residue.flags.c_contiguous and dW.shape == residue.shape
    n = dW.size
    cap = stream_bytes(n, L_T, n)           # worst case: every element sent
    out = np.empty(cap, dtype=np.uint8)
    n_bins = (n + L_T - 1) // L_T
    gmax = np.empty(max(n_bins, 1), dtype=np.float32) if want_gmax else None
    rc = lib().adacomp_oracle_pack_general(_ptr(dW) if n else None, _ptr(residue) if n else None, n, L_T,
                                           flags, C.c_float(factor), int(quantiser), _ptr(out), cap,
                                           _ptr(gmax) if want_gmax else None)
    if rc != 0:
        raise RuntimeError(f"adacomp_oracle_pack failed: {rc}")
    p = parse(out)
    if want_gmax:
        p.g_max = gmax[:n_bins]
    return p


def unpack_sum(streams: Sequence[np.ndarray], n: int) -> np.ndarray:
    """Sum k packed streams, in order, into a dense float32 vector."""
    keep: List[np.ndarray] = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * len(keep))(*[_ptr(s) for s in keep])
    dst = np.empty(n, dtype=np.float32)
    rc = lib().adacomp_oracle_unpack_sum(ptrs, len(keep), _ptr(dst) if n else None, n)
    if rc != 0:
        raise RuntimeError(f"adacomp_oracle_unpack_sum failed: {rc}")
    return dst


def to_v2(raw_v1: np.ndarray) -> np.ndarray:
    """A version-1 stream re-encoded as version 2 (the bins told apart by a flag in the words; no count section)."""
    v1 = np.ascontiguousarray(raw_v1, dtype=np.uint8)
    p = parse(v1)
    n_empty = int(np.count_nonzero(p.bin_cnt == 0))
    cap = int(lib().adacomp_oracle_v2_bytes(p.n, p.L_T, p.n_sel + n_empty))
    out = np.empty(cap, dtype=np.uint8)
    rc = lib().adacomp_oracle_to_v2(_ptr(v1), _ptr(out), cap)
    if rc != 0:
        raise RuntimeError(f"adacomp_oracle_to_v2 failed: {rc}")
    return out


def from_v2(raw_v2: np.ndarray) -> np.ndarray:
    """The version-1 form of a version-2 stream."""
    v2 = np.ascontiguousarray(raw_v2, dtype=np.uint8)
    L_T, n, n_sel = struct.unpack_from("<I", v2, 8)[0], struct.unpack_from("<Q", v2, 16)[0], struct.unpack_from("<Q", v2, 40)[0]
    cap = stream_bytes(n, L_T, n_sel)
    out = np.empty(cap, dtype=np.uint8)
    rc = lib().adacomp_oracle_from_v2(_ptr(v2), _ptr(out), cap)
    if rc != 0:
        raise RuntimeError(f"adacomp_oracle_from_v2 failed: {rc}")
    return out


def unpack_sum_v2(streams: Sequence[np.ndarray], n: int) -> np.ndarray:
    """Sum k version-2 streams, in order, into a dense float32 vector (decoded from the flags alone)."""
    keep: List[np.ndarray] = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * len(keep))(*[_ptr(s) for s in keep])
    dst = np.empty(n, dtype=np.float32)
    rc = lib().adacomp_oracle_unpack_sum_v2(ptrs, len(keep), _ptr(dst) if n else None, n)
    if rc != 0:
        raise RuntimeError(f"adacomp_oracle_unpack_sum_v2 failed: {rc}")
    return dst


def average_sgd(streams: Sequence[np.ndarray], n: int, weights: np.ndarray, momentum: np.ndarray,
                lr: float, mu: float):
    """unpack(), averageGradients() and updateWeights() of Algorithm 1 ("Computation Steps") for one layer.

    The paper trains with "the conventional SGD with momentum" (momentum 0.9, Section "Discussions") and
    gives no formula; the reading taken here is the plain heavy-ball step with no dampening, Nesterov
    term or weight decay, every operation rounded to binary32 on its own (no fused multiply-add):

        s    = sum of the k decoded streams, in learner order, from +0.0f     (unpack, as unpack_sum)
        mean = s / k                                                          (averageGradients: one division)
        v'   = (mu * v) + mean                                                (updateWeights)
        w'   = w - (lr * v')

    Returns (w', v') as new float32 arrays; the inputs are not modified.
    """
    return sgd_step(unpack_sum(streams, n), len(streams), weights, momentum, lr, mu)


def sgd_step(s: np.ndarray, k: int, weights: np.ndarray, momentum: np.ndarray, lr: float, mu: float):
    """averageGradients() and updateWeights() of average_sgd on a decoded sum `s` of k streams (or on a slice
    of one, with the matching slices of the weights and the momentum): the three lines of its docstring."""
    n = s.size
    assert s.dtype == np.float32
    w = np.ascontiguousarray(weights, dtype=np.float32)
    v = np.ascontiguousarray(momentum, dtype=np.float32)
    mean = s / np.float32(k)
    v_new = np.float32(mu) * v[:n] + mean
    w_new = w[:n] - np.float32(lr) * v_new
    assert mean.dtype == v_new.dtype == w_new.dtype == np.float32
    return w_new, v_new


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) as float32 values: a bfloat16 is the upper half of a binary32, so the
    conversion appends sixteen zero bits and is exact (NaNs keep their payload)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def pack_bf16(dW_bits: np.ndarray, residue: np.ndarray, L_T: int, flags: int = 0, want_gmax: bool = False) -> Packed:
    """pack() for a gradient that arrives in bfloat16 (the paper's motivation is reduced-precision
    accelerators, Section 1; the residue, and all of Algorithm 2's arithmetic, stay binary32): the
    gradient is widened exactly and Algorithm 2 runs as for any binary32 gradient."""
    return pack(bf16_to_f32(dW_bits), residue, L_T, flags=flags, want_gmax=want_gmax)


def f16_to_f32(bits: np.ndarray) -> np.ndarray:
    """IEEE binary16 bit patterns (uint16) as float32 values.  Every binary16 value (subnormals, infinities
    and NaNs included) is a binary32 value, so the conversion is exact; numpy's cast is that conversion."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return b.view(np.float16).astype(np.float32)


def pack_f16(dW_bits: np.ndarray, residue: np.ndarray, L_T: int, flags: int = 0, want_gmax: bool = False,
             factor: float = 0.0) -> Packed:
    """pack() for a gradient that arrives in binary16: widened exactly, then Algorithm 2 as for any binary32 gradient."""
    return pack(f16_to_f32(dW_bits), residue, L_T, flags=flags, want_gmax=want_gmax, factor=factor)


def average_adam(streams: Sequence[np.ndarray], n: int, weights: np.ndarray, m: np.ndarray, v: np.ndarray,
                 step_size: float, beta1: float, beta2: float, eps: float):
    """unpack(), averageGradients() and an Adam step for one layer (the paper reports AdaComp with Adam too,
    Section "Experiments"; it prints no formula).  The step is Kingma and Ba's Algorithm 1 in the order
    its Section 2 suggests for efficiency, every operation rounded to binary32 on its own:

        mean = s / k
        m'   = (beta1 * m) + ((1 - beta1) * mean)
        v'   = (beta2 * v) + ((1 - beta2) * (mean * mean))
        w'   = w - ((step_size * m') / (sqrt(v') + eps))

    with 1 - beta computed in binary32 and step_size = alpha * sqrt(1 - beta2^t) / (1 - beta1^t) supplied by the
    caller (the bias correction belongs to the training loop, which knows t).  Returns (w', m', v')."""
    k = len(streams)
    f = np.float32
    w = np.ascontiguousarray(weights, dtype=np.float32)[:n]
    m0 = np.ascontiguousarray(m, dtype=np.float32)[:n]
    v0 = np.ascontiguousarray(v, dtype=np.float32)[:n]
    s = unpack_sum(streams, n)
    mean = s / f(k)
    c1 = f(1) - f(beta1)
    c2 = f(1) - f(beta2)
    m_new = f(beta1) * m0 + c1 * mean
    v_new = f(beta2) * v0 + c2 * (mean * mean)
    den = np.sqrt(v_new) + f(eps)
    w_new = w - (f(step_size) * m_new) / den
    assert m_new.dtype == v_new.dtype == w_new.dtype == den.dtype == np.float32
    return w_new, m_new, v_new
