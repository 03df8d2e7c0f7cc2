"""Pins of the oracle's binary16-gradient front end: the widening is exact, agrees with the definition of the
format on hand-picked patterns and with torch's cast on every finite pattern, and Algorithm 2 then sees an
ordinary binary32 gradient."""
import struct

import numpy as np
import torch

from oracle import cref


def test_widening_is_exact_on_every_finite_pattern_and_is_torchs_cast():
    bits = np.arange(1 << 16, dtype=np.uint16)
    bits = bits[(bits & 0x7c00) != 0x7c00]                   # finite values (NaN payloads compare unequal)
    got = cref.f16_to_f32(bits)
    want = torch.from_numpy(bits.view(np.int16).copy()).view(torch.float16).to(torch.float32).numpy()
    np.testing.assert_array_equal(got.view(np.uint32), want.view(np.uint32))
    # the definition (-1)^s 2^(e-15) (1 + m / 1024), subnormals m / 1024 * 2^-14, worked out in exact integers
    for b in (0x0001, 0x03ff, 0x0400, 0x3c00, 0xbc01, 0x7bff, 0x8000, 0x1234, 0xfbff, 0x3555):
        s, e, m = b >> 15, (b >> 10) & 31, b & 1023
        value = (m / 1024.0) * 2.0 ** -14 if e == 0 else (1.0 + m / 1024.0) * 2.0 ** (e - 15)
        value = -value if s else value
        f = cref.f16_to_f32(np.array([b], np.uint16))[0]
        assert struct.pack("<f", f) == struct.pack("<f", value), hex(b)
    inf = cref.f16_to_f32(np.array([0x7c00, 0xfc00], np.uint16))
    assert inf[0] == np.inf and inf[1] == -np.inf


def test_pack_of_a_binary16_gradient_is_pack_of_its_widened_values():
    rng = np.random.default_rng(33)
    n, L_T = 10007, 50
    g = rng.normal(0, 1e-3, n).astype(np.float32)
    bits = g.astype(np.float16).view(np.uint16)
    r1 = rng.normal(0, 2e-3, n).astype(np.float32)
    r2 = r1.copy()
    a = cref.pack_f16(bits, r1, L_T)
    b = cref.pack(cref.f16_to_f32(bits), r2, L_T)
    assert bytes(a.raw) == bytes(b.raw)
    np.testing.assert_array_equal(r1, r2)
    c = cref.pack(g, rng.normal(0, 2e-3, n).astype(np.float32), L_T)
    assert bytes(a.raw) != bytes(c.raw)
