"""Pins of the oracle's bfloat16-gradient front end: the widening is the library's (torch) cast and the
IEEE definition, and Algorithm 2 then sees an ordinary binary32 gradient."""
import struct

import numpy as np
import torch

from oracle import cref


def test_widening_is_exact_and_is_torchs_cast():
    rng = np.random.default_rng(31)
    bits = rng.integers(0, 1 << 16, 20000, dtype=np.uint16)
    bits = bits[(bits & 0x7f80) != 0x7f80]                   # finite values (NaN payloads compare unequal)
    got = cref.bf16_to_f32(bits)
    want = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    # the definition, on a few hand-picked patterns: 1.0, -2.0, 0.15625, smallest subnormal, -0.0
    for b, v in ((0x3f80, 1.0), (0xc000, -2.0), (0x3e20, 0.15625), (0x0001, 2.0 ** -133), (0x8000, -0.0)):
        f = cref.bf16_to_f32(np.array([b], np.uint16))[0]
        assert struct.pack("<f", f) == struct.pack("<f", v), hex(b)


def test_pack_of_a_bf16_gradient_is_pack_of_its_widened_values():
    rng = np.random.default_rng(32)
    n, L_T = 10007, 50
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    bits = (g.view(np.uint32) >> 16).astype(np.uint16)       # truncation is good enough to make test data
    r1 = rng.normal(0, 2e-3, n).astype(np.float32)
    r2 = r1.copy()
    a = cref.pack_bf16(bits, r1, L_T)
    b = cref.pack(cref.bf16_to_f32(bits), r2, L_T)
    assert bytes(a.raw) == bytes(b.raw)
    np.testing.assert_array_equal(r1, r2)
    # and it is a different stream from the unrounded gradient's: the widened values are what counts
    c = cref.pack(g, rng.normal(0, 2e-3, n).astype(np.float32), L_T)
    assert bytes(a.raw) != bytes(c.raw)
