"""Second, independent restatement of pack() / unpack-sum in scalar Python.

TEST INFRASTRUCTURE ONLY.  Pure loops over numpy float32 scalars and a
`fractions.Fraction` sum for the layer scale; used on tiny inputs to brute-force
the C oracle (the two are written separately and must agree byte for byte).
Follows Algorithm 2 of the paper with the readings listed in the C oracle's header.
"""
from __future__ import annotations

import struct
from fractions import Fraction
from typing import List, Sequence, Tuple

import numpy as np

f32 = np.float32


def _tile_bins(L_T: int) -> int:
    return 4 * (1000 // L_T) if L_T <= 1000 else 1


def pack(dW: Sequence[float], residue: Sequence[float], L_T: int, literal: bool = False, factor: float = 0.0,
         quantiser: int = 0):
    """Returns (bin_cnt, words, scale, new_residue, g_max).  `factor` other than 0 replaces the paper's
    H = G + dW by H = residue + factor * dW (the scale-factor of Section 2.4; 1 = local selection only).
    `quantiser` 1 replaces the mean of the bin maxima by the mean |G| of the sent elements (Section 2.5 leaves
    the quantisation function open)."""
    n = len(dW)
    dW = [f32(x) for x in dW]
    residue = [f32(x) for x in residue]
    G = [f32(residue[i] + dW[i]) for i in range(n)]          # this step's accumulated gradient
    if factor == 0.0:
        H = [f32(G[i] + dW[i]) for i in range(n)]            # the latest gradient counted twice (the selection's look-ahead)
    else:
        H = [f32(residue[i] + f32(f32(factor) * dW[i])) for i in range(n)]
    n_bins = -(-n // L_T)
    g_max = []
    for i in range(n_bins):                                  # first sweep: each bin's largest |G|
        members = G[i * L_T:(i + 1) * L_T]
        g_max.append(max((abs(x) for x in members), default=f32(0)))
    if n_bins:
        total = sum((Fraction(float(m)) for m in g_max), Fraction(0))
        S = float(total)                                     # int/int division: correctly rounded
        scale = f32(S / float(n_bins))
    else:
        scale = f32(0)
    def is_sent(index, i):
        g, h, m = G[index], H[index], g_max[i]
        return bool(m > 0 and g != 0 and (abs(h) >= m or (not literal and abs(g) == m)))

    if quantiser == 1:
        sent = [abs(G[i * L_T + j]) for i in range(n_bins) for j in range(L_T) if i * L_T + j < n and is_sent(i * L_T + j, i)]
        if sent:
            total = sum((Fraction(float(x)) for x in sent), Fraction(0))
            scale = f32(float(total) / float(len(sent)))
        else:
            scale = f32(0)
    bin_cnt: List[int] = []
    words: List[int] = []
    new_residue = list(G)
    for i in range(n_bins):                                  # second sweep: bin by bin,
        count = 0
        for j in range(L_T):                                 # place by place
            index = i * L_T + j
            if index >= n:
                break
            g, h, m = G[index], H[index], g_max[i]
            send = m > 0 and g != 0 and (abs(h) >= m or (not literal and abs(g) == m))
            if send:
                negative = bool(np.signbit(g))
                Gq = -scale if negative else scale
                words.append((j << 2) | (3 if negative else 1))
                new_residue[index] = f32(g - Gq)
                count += 1
        bin_cnt.append(count)
    return bin_cnt, words, scale, new_residue, g_max


def to_stream(n: int, L_T: int, bin_cnt: Sequence[int], words: Sequence[int], scale,
              literal: bool = False, factor: float = 0.0, quantiser: int = 0) -> bytes:
    """Serialise to the wire layout: header, tile directory, bin counts, words."""
    w = 1 if L_T <= 64 else 2
    tb = _tile_bins(L_T)
    n_bins = len(bin_cnt)
    n_tiles = -(-n_bins // tb)
    tile_off = [sum(bin_cnt[:t * tb]) for t in range(n_tiles)] + [len(words)]
    fmt = "B" if w == 1 else "H"
    pad16 = lambda b: b + bytes((-len(b)) % 16)
    body = pad16(struct.pack(f"<{n_tiles + 1}Q", *tile_off))
    body += pad16(struct.pack(f"<{n_bins}{fmt}", *bin_cnt))
    body += pad16(struct.pack(f"<{len(words)}{fmt}", *words))
    bytes_used = 64 + len(body)
    scale_bits = struct.unpack("<I", struct.pack("<f", float(scale)))[0]
    head = struct.pack("<IHBBIIQQQQIIQ", 0x31434441, 1, w, (1 if literal else 0) | (2 if factor != 0.0 else 0) | (4 if quantiser == 1 else 0), L_T, tb, n, n_bins,
                       n_tiles, len(words), scale_bits, 0, bytes_used)
    return head + body


def unpack_sum(streams: Sequence[Tuple[Sequence[int], Sequence[int], float]], n: int, L_T: int):
    """streams: (bin_cnt, words, scale) per learner.  Ordered sum from +0.0."""
    dst = [f32(0)] * n
    for bin_cnt, words, scale in streams:
        at = 0
        for b, count in enumerate(bin_cnt):
            for _ in range(count):
                word = words[at]
                at += 1
                index = b * L_T + (word >> 2)
                code = word & 3
                if code == 1:
                    dst[index] = f32(dst[index] + f32(scale))
                elif code == 3:
                    dst[index] = f32(dst[index] - f32(scale))
                elif code == 2:
                    raise ValueError("reserved ternary code")
    return dst


def to_stream_v2(n: int, L_T: int, bin_cnt: Sequence[int], words: Sequence[int], scale,
                 literal: bool = False, factor: float = 0.0, quantiser: int = 0) -> bytes:
    """Serialise to stream version 2: no counts; the first word of every bin carries a flag, a bin that sends
    nothing is one marker word (flag set, index L_T).  word = (index << 2) | (first << 1) | negative."""
    w = 1 if L_T <= 63 else 2
    tb = _tile_bins(L_T)
    n_bins = len(bin_cnt)
    n_tiles = -(-n_bins // tb)
    out_words: List[int] = []
    tile_off: List[int] = []
    at = 0
    for b, count in enumerate(bin_cnt):
        if b % tb == 0:
            tile_off.append(len(out_words))
        if count == 0:
            out_words.append((L_T << 2) | 2)
        for j in range(count):
            word = words[at]
            at += 1
            out_words.append((word & ~3) | (2 if j == 0 else 0) | (1 if (word & 3) == 3 else 0))
    tile_off.append(len(out_words))
    fmt = "B" if w == 1 else "H"
    pad16 = lambda b: b + bytes((-len(b)) % 16)
    dir_bytes = struct.pack(f"<{n_tiles + 1}Q", *tile_off)
    body = bytes((-(64 + len(dir_bytes))) % 16)
    body = dir_bytes + body + pad16(struct.pack(f"<{len(out_words)}{fmt}", *out_words))
    bytes_used = 64 + len(body)
    scale_bits = struct.unpack("<I", struct.pack("<f", float(scale)))[0]
    flags = (1 if literal else 0) | (2 if factor != 0.0 else 0) | (4 if quantiser == 1 else 0)
    head = struct.pack("<IHBBIIQQQQIIQ", 0x31434441, 2, w, flags, L_T, tb, n, n_bins, n_tiles, len(words), scale_bits,
                       sum(1 for c in bin_cnt if c == 0), bytes_used)
    return head + body

