"""Property tests (hypothesis): the C oracle against the independent scalar restatement on
arbitrary small inputs, including signed zeros, denormals, huge values and ties.  CPU only."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import cref, scalar

SPECIAL = [0.0, -0.0, 1e-45, -1e-45, 1.17549435e-38, 1e38, -1e38, 1.0, -1.0, 0.5, -0.5, 2.0 ** -126, 1e-3, -1e-3]
f32s = st.one_of(st.sampled_from(SPECIAL),
                 st.floats(width=32, allow_nan=False, allow_infinity=False, min_value=-float(np.float32(1e37)), max_value=float(np.float32(1e37))))


@st.composite
def layer(draw):
    n = draw(st.integers(1, 40))
    L_T = draw(st.sampled_from([1, 2, 3, 5, 8, 50, 64, 65, 500]))
    dW = draw(st.lists(f32s, min_size=n, max_size=n))
    res = draw(st.lists(f32s, min_size=n, max_size=n))
    return L_T, np.array(dW, np.float32), np.array(res, np.float32)


@settings(max_examples=400, deadline=None)
@given(layer(), st.booleans())
def test_c_oracle_equals_scalar_restatement(case, literal):
    L_T, dW, res = case
    rc = res.copy()
    p = cref.pack(dW, rc, L_T, flags=int(literal))
    cnt, words, scale, new_res, gmax = scalar.pack(dW, res, L_T, literal)
    assert p.raw.tobytes() == scalar.to_stream(len(dW), L_T, cnt, words, scale, literal)
    assert rc.tobytes() == np.array(new_res, np.float32).tobytes()
    # invariants that hold for any input
    pos, code = p.positions_and_codes()
    G = (res + dW).astype(np.float32)
    assert np.all(np.diff(pos) > 0) and set(np.unique(code)) <= {1, 3}
    unsent = np.ones(len(dW), bool)
    unsent[pos] = False
    assert rc[unsent].tobytes() == G[unsent].tobytes()
    if not literal and np.all(np.isfinite(G)):
        B = -(-len(dW) // L_T)
        gm = np.array([np.abs(G[b * L_T:(b + 1) * L_T]).max() for b in range(B)], np.float32)
        assert np.array_equal(p.bin_cnt > 0, gm > 0)


@settings(max_examples=150, deadline=None)
@given(st.lists(layer(), min_size=1, max_size=4))
def test_unpack_sum_equals_scalar_restatement(cases):
    L_T, dW0, _ = cases[0]
    n = len(dW0)
    streams_c, streams_s = [], []
    for _, dW, res in cases:
        dW = np.resize(dW, n).astype(np.float32)
        res = np.resize(res, n).astype(np.float32)
        p = cref.pack(dW, res.copy(), L_T)
        cnt, words, scale, _, _ = scalar.pack(dW, res, L_T)
        streams_c.append(p.raw)
        streams_s.append((cnt, words, scale))
    got = cref.unpack_sum(streams_c, n)
    want = np.array(scalar.unpack_sum(streams_s, n, L_T), np.float32)
    assert got.tobytes() == want.tobytes()
