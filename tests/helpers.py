"""Small readers for the text fixtures under tests/golden/."""
import os
import zlib

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_sections(name):
    """'key = v v v' lines grouped under [section] headers; '#' starts a comment."""
    out, cur = {"": {}}, ""
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            if line.startswith("["):
                cur = line.strip("[]")
                out[cur] = {}
                continue
            k, v = [s.strip() for s in line.split("=", 1)]
            out[cur][k] = v.split()
    return out


def read_rows(name, tag):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].split()
            if line and line[0] == tag:
                rows.append(line[1:])
    return rows


def f32(vals):
    return np.array([float(v) for v in vals], dtype=np.float32)


def crc_counts_words(bin_cnt, words):
    """zlib CRC-32 of the bin-count bytes followed by the payload bytes (little-endian)."""
    a = np.ascontiguousarray(bin_cnt).astype(bin_cnt.dtype.newbyteorder("<")).tobytes()
    b = np.ascontiguousarray(words).astype(words.dtype.newbyteorder("<")).tobytes()
    return zlib.crc32(a + b) & 0xFFFFFFFF
