"""CUDA path vs the CPU oracle through the C ABI, element by element.

Integer outputs (indices, signs, packed bytes, counts, directory) must match
bit for bit; so must scale and residue: both sides take the same single
binary32 operations and the scale comes from an exact sum, so the tolerance
the task allows (1e-6 relative, 1e-7 absolute near zero) is only checked as a
fallback statement of that bar."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from paper_1712_02679_b200 import synth
from tests.gpu_util import GpuLayer, assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-6, 1e-7       # the stated floating-point bar; the tests below are stricter (bits)


def run_steps(n, L_T, dws, flags=0, residue0=None):
    """Carried-residue run on both sides; compares every step."""
    r_cpu = np.zeros(n, np.float32) if residue0 is None else residue0.copy()
    layer = GpuLayer(n, L_T, residue0)
    streams = []
    for step, dW in enumerate(dws):
        want = cref.pack(dW, r_cpu, L_T, flags=flags & 1)
        raw, n_sel, used = layer.compress(dW, flags)
        what = f"n={n} L_T={L_T} flags={flags} step={step}"
        assert (n_sel, used) == (want.n_sel, want.bytes_used), what
        assert_stream_equal(raw, want, what)
        got_r = layer.residue_host()
        assert_f32_bits_equal(got_r, r_cpu, what + " residue")
        np.testing.assert_allclose(got_r, r_cpu, rtol=RTOL, atol=ATOL)
        streams.append(raw)
    assert B.adacomp_device_status() == 0
    return layer, streams


def test_config1_fc_layer_ten_steps():
    n, L_T = 100352, 50
    dws = [synth.make_dw(1, 0, 0, s, n, heavy=False, sigma=1e-3) for s in range(10)]
    run_steps(n, L_T, dws)
    run_steps(n, L_T, dws[:3], flags=B.ADACOMP_FLAG_GENERIC_PATH)


def test_config2_small_conv_net_twenty_steps():
    for t, spec in enumerate(synth.config2_tensors()):
        dws = [synth.make_dw(2, 0, t, s, spec.n, heavy=True) for s in range(20)]
        run_steps(spec.n, spec.L_T, dws)


@pytest.mark.parametrize("L_T", [1, 2, 3, 7, 25, 49, 50, 51, 63, 64, 65, 100, 333, 499, 500, 501,
                                 1000, 1001, 4096, 5000, 16384])
def test_bin_lengths_and_ragged_tails(L_T):
    rng = np.random.default_rng(L_T)
    for n in sorted({1, L_T - 1, L_T, L_T + 1, 4001, 3 * 4000 + 17, 10 * max(L_T, 40) + 3}):
        if n <= 0:
            continue
        dws = [rng.normal(0, 1e-3, n).astype(np.float32) for _ in range(3)]
        run_steps(n, L_T, dws)


@pytest.mark.parametrize("L_T", [50, 100, 125, 200, 250, 500, 1000])
@pytest.mark.parametrize("n", [4000, 8000, 7999, 8001, 4000 * 150 + 1, 4000 * 1500 - 3])
def test_fast_path_tile_boundaries(L_T, n):
    rng = np.random.default_rng(n + L_T)
    dws = [synth.heavy_dw(n, 1e-3, rng) for _ in range(4)]
    run_steps(n, L_T, dws)
    run_steps(n, L_T, dws[:2], flags=B.ADACOMP_FLAG_LITERAL)
    run_steps(n, L_T, dws[:2], flags=B.ADACOMP_FLAG_GENERIC_PATH | B.ADACOMP_FLAG_LITERAL)


@pytest.mark.parametrize("L_T", [41, 52, 64, 65, 96, 300, 333, 400, 800, 999, 1004, 1500, 2000, 3000, 3996, 4000])
def test_any_bin_tile_pass_tile_boundaries(L_T):
    """Bin lengths whose bins do not line up with the threads' 25-element segments: the tile pass
    finds each segment's one or two bins at run time.  Whole tiles, ragged tails, many tiles; with a
    scale-factor; and against the warp-per-bin kernel on the same inputs."""
    T = 4 * (1000 // L_T) * L_T if L_T <= 1000 else L_T        # a tile (one bin where L_T > 1000)
    for n in (T, 2 * T, 2 * T - 1, 2 * T + 1, T * 150 + 1, T * 301 - L_T - 3):
        rng = np.random.default_rng(n + L_T)
        dws = [synth.heavy_dw(n, 1e-3, rng) for _ in range(3)]
        run_steps(n, L_T, dws)
        run_steps(n, L_T, dws[:2], flags=B.ADACOMP_FLAG_GENERIC_PATH)


def test_empty_tensor_writes_a_header_only():
    layer = GpuLayer(0, 50)
    raw, n_sel, used = layer.compress(np.zeros(0, np.float32))
    want = cref.pack(np.zeros(0, np.float32), np.zeros(0, np.float32), 50)
    assert (n_sel, used) == (0, 80)
    assert_stream_equal(raw, want)


def test_degenerate_values():
    n, L_T = 9000, 50
    rng = np.random.default_rng(4)
    zeros = np.zeros(n, np.float32)
    run_steps(n, L_T, [zeros, zeros])                              # nothing to send at all
    dw = rng.normal(0, 1e-3, n).astype(np.float32)
    dw[:150] = 0                                                   # zero bins inside
    dw[200:250] = np.float32(1e-3)                                 # a bin of ties: all sent
    dw[300:350] = np.float32(-0.0)
    run_steps(n, L_T, [dw, -dw, dw])                               # -dw cancels: exact zeros
    tiny = (rng.normal(0, 1, n) * 1e-42).astype(np.float32)        # denormals must survive
    run_steps(n, L_T, [tiny, tiny])
    huge = (rng.normal(0, 1, n) * 1e37).astype(np.float32)
    run_steps(n, L_T, [huge])
    wide = (rng.normal(0, 1, n) * 10.0 ** rng.uniform(-40, 30, n)).astype(np.float32)
    run_steps(n, 500, [wide, wide])                                # scale sum over 70 decades
    res0 = rng.normal(0, 5e-3, n).astype(np.float32)
    run_steps(n, 500, [np.zeros(n, np.float32)], residue0=res0)    # dW = 0: only maxima go


def test_metamorphic_on_gpu_scale_is_order_independent():
    L_T, Bn = 50, 4000
    rng = np.random.default_rng(9)
    dW = rng.normal(0, 1e-3, L_T * Bn).astype(np.float32)
    dW[::977] *= np.float32(1e4)
    perm = rng.permutation(Bn)
    dWp = dW.reshape(Bn, L_T)[perm].ravel().copy()
    a, _ = run_steps(L_T * Bn, L_T, [dW])
    b, _ = run_steps(L_T * Bn, L_T, [dWp])
    sa = a.packed[48:52].cpu().numpy().tobytes()
    sb = b.packed[48:52].cpu().numpy().tobytes()
    assert sa == sb


def test_same_inputs_twice_give_the_same_bytes():
    n = 4000 * 300 + 11
    rng = np.random.default_rng(21)
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    res = rng.normal(0, 3e-3, n).astype(np.float32)
    outs = []
    for _ in range(3):
        layer = GpuLayer(n, 50, res)
        raw, _, _ = layer.compress(dW)
        outs.append((raw.tobytes(), layer.residue_host().tobytes()))
    assert outs[0] == outs[1] == outs[2]


# --------------------------------------------------------------------------
# unpack()-and-sum
# --------------------------------------------------------------------------

def gpu_decode(streams, n):
    dev = torch.device("cuda:0")
    bufs = [torch.from_numpy(s.copy()).to(dev) for s in streams]
    # pad each to a 16-byte aligned allocation (torch already aligns to 512)
    dst = torch.full((max(n, 4),), float("nan"), dtype=torch.float32, device=dev)
    B.adacomp_decompress_accumulate(bufs, len(bufs), dst)
    torch.cuda.synchronize()
    return dst[:n].cpu().numpy()


@pytest.mark.parametrize("L_T,n,k", [(50, 100352, 1), (50, 5120, 4), (500, 147456, 8), (50, 4000 * 40 + 7, 16),
                                     (3, 9001, 3), (64, 70000, 2), (65, 70000, 2), (1000, 50001, 5),
                                     (1001, 50001, 5), (5000, 123457, 3), (16384, 100001, 4),
                                     (16384, 100, 2), (500, 12, 64),
                                     # every lane-to-bin arrangement of the warp decoder: 24 / 20 bins per warp by word,
                                     # then 16, 10, 8, 4, 2 and 1 bins per warp with 2 .. 32 lanes per bin
                                     (41, 96 * 41 * 9 + 5, 3), (48, 80 * 48 * 7 + 1, 4), (49, 80 * 49 * 5, 2),
                                     (62, 64 * 62 * 6 + 9, 3), (100, 40 * 100 * 5 + 7, 3), (125, 32 * 125 * 5 + 3, 5),
                                     (250, 16 * 250 * 6 + 11, 3), (400, 8 * 400 * 7 + 2, 9), (1000, 4 * 1000 * 6 + 13, 3),
                                     # bin-count runs of a tile that are not a multiple of 16 bytes; 3, 5 and 15 bins per warp
                                     (52, 76 * 52 * 9 + 3, 4), (58, 68 * 58 * 7 + 50, 3), (63, 60 * 63 * 8 + 1, 5),
                                     (66, 60 * 66 * 5 + 65, 2), (200, 20 * 200 * 9 + 199, 4), (300, 12 * 300 * 7 + 8, 3),
                                     (800, 4 * 800 * 11 + 5, 6),
                                     # one bin per tile: the warps share it, in one to four chunks
                                     (1001, 1001 * 23 + 17, 5), (2000, 2000 * 40 + 3, 4), (2001, 2001 * 21 + 1999, 3),
                                     (4096, 4096 * 9 + 1, 3), (4097, 4097 * 7 + 5, 3), (5000, 5000 * 30 + 123, 6),
                                     (8192, 8192 * 5, 2), (12345, 12345 * 9 + 12000, 3), (16384, 16384 * 6 + 11, 4)])
def test_decode_sum_matches_oracle(L_T, n, k):
    rng = np.random.default_rng(L_T + n + k)
    streams_gpu, streams_cpu = [], []
    for l in range(k):
        r = rng.normal(0, 2e-3, n).astype(np.float32)
        dW = rng.normal(0, 1e-3 * (1 + l), n).astype(np.float32)
        want = cref.pack(dW, r.copy(), L_T)
        raw, _, _ = GpuLayer(n, L_T, r).compress(dW)
        assert_stream_equal(raw, want)
        streams_gpu.append(raw)
        streams_cpu.append(want.raw)
    want_dst = cref.unpack_sum(streams_cpu, n)
    got = gpu_decode(streams_gpu, n)
    assert_f32_bits_equal(got, want_dst, f"decode L_T={L_T} n={n} k={k}")
    np.testing.assert_allclose(got, want_dst, rtol=RTOL, atol=ATOL)
    assert B.adacomp_device_status() == 0


def test_decode_sum_dense_streams_overflow_the_prefetch_stage():
    """Every element sent (all ties): 4000 words per tile and learner, so only a few learners'
    words fit the decoder's staging buffer and the rest take its one-at-a-time path."""
    rng = np.random.default_rng(8)
    for L_T, n, k in [(50, 4000 * 9 + 123, 12), (500, 4000 * 5 + 77, 7), (5000, 5000 * 5 + 77, 5), (16384, 16384 * 3 + 5, 3)]:
        streams = []
        for l in range(k):
            sign = np.where(rng.random(n) < 0.5, -1.0, 1.0).astype(np.float32)
            dW = sign * np.float32(2.0 ** -(l % 5))
            want = cref.pack(dW, np.zeros(n, np.float32), L_T)
            assert want.n_sel == n
            raw, _, _ = GpuLayer(n, L_T).compress(dW)
            assert_stream_equal(raw, want)
            streams.append(raw)
        got = gpu_decode(streams, n)
        assert_f32_bits_equal(got, cref.unpack_sum(streams, n), f"dense decode L_T={L_T} k={k}")
    assert B.adacomp_device_status() == 0


def test_decode_sum_uneven_density_and_many_learners():
    """The decoder sizes a learner's staging region from its average words per tile.  A learner that is
    dense in a few tiles only overflows it there; forty sparse learners share one staging slot (more
    learners than a warp has lanes); forty denser ones need several slots per tile."""
    rng = np.random.default_rng(77)
    cases = []
    for L_T in (50, 500):
        n = 4000 * 12 + 5
        layers = []
        for l in range(5):
            dW = rng.normal(0, 1e-3, n).astype(np.float32)
            if l == 2:      # every element of tiles 3..5 ties for its bin's maximum: all of them are sent
                dW[12000:24000] = np.where(rng.random(12000) < 0.5, -1.0, 1.0).astype(np.float32) * np.float32(0.25)
            layers.append((dW, np.zeros(n, np.float32)))
        cases.append((L_T, n, layers))
    n = 4000 * 6 + 9
    sparse = []
    for l in range(40):     # a few large entries per learner on a floor of tiny ones: few words per tile
        dW = rng.normal(0, 1e-6, n).astype(np.float32)
        at = rng.choice(n, 60, replace=False)
        dW[at] = rng.normal(0, 1.0, 60).astype(np.float32)
        sparse.append((dW, rng.normal(0, 1e-6, n).astype(np.float32)))
    cases.append((500, n, sparse))
    cases.append((50, n, [(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32)) for _ in range(40)]))
    for L_T, n, layers in cases:
        streams = []
        for dW, r in layers:
            want = cref.pack(dW, r.copy(), L_T)
            raw, _, _ = GpuLayer(n, L_T, r).compress(dW)
            assert_stream_equal(raw, want)
            streams.append(raw)
        got = gpu_decode(streams, n)
        assert_f32_bits_equal(got, cref.unpack_sum(streams, n), f"decode L_T={L_T} k={len(layers)}")
    assert B.adacomp_device_status() == 0


def test_decode_with_shape_hint_matches_and_rejects_wrong_hints():
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(31)
    for L_T, n in [(50, 777), (500, 4000 * 12 + 5), (7, 3000), (50, 4000 * 300)]:
        raws = []
        for l in range(3):
            dW = rng.normal(0, 1e-3 * (l + 1), n).astype(np.float32)
            raws.append(cref.pack(dW, np.zeros(n, np.float32), L_T).raw)
        bufs = [torch.from_numpy(r.copy()).to(dev) for r in raws]
        dst = torch.full((n,), float("nan"), device=dev)
        B.adacomp_decompress_accumulate_ex(bufs, 3, dst, n, L_T)
        torch.cuda.synchronize()
        assert_f32_bits_equal(dst.cpu().numpy(), cref.unpack_sum(raws, n), f"hinted decode L_T={L_T} n={n}")
        dsts = [torch.empty(n, device=dev) for _ in range(2)]
        B.adacomp_decompress_accumulate_multi_ex(bufs + bufs, 3, dsts, [n, n], [L_T, L_T], 2)
        torch.cuda.synchronize()
        assert torch.equal(dsts[0], dst) and torch.equal(dsts[1], dst)
        assert B.adacomp_device_status() == 0
        dst.fill_(float("nan"))
        B.adacomp_decompress_accumulate_ex(bufs, 3, dst, n + 1, L_T)       # wrong n: flagged, dst untouched
        assert B.adacomp_device_status() & B.ADACOMP_DEV_HEADER_MISMATCH
        assert bool(torch.isnan(dst).all())
        B.adacomp_device_status_reset()


def test_decode_sum_seeded_four_learners_crosscheck():
    import zlib
    spec = synth.config2_tensors()[7]
    streams = []
    for l in range(4):
        dW = synth.make_dw(2, l, 7, 0, spec.n, heavy=True)
        raw, _, _ = GpuLayer(spec.n, spec.L_T).compress(dW)
        streams.append(raw)
    dst = gpu_decode(streams, spec.n)
    assert zlib.crc32(dst.astype("<f4").tobytes()) & 0xFFFFFFFF == 0x4FC334F2
    assert int(np.count_nonzero(dst)) == 2589


def test_decoder_flags_bad_streams_without_faulting():
    n, L_T = 20000, 50
    rng = np.random.default_rng(2)
    a = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L_T)
    b = cref.pack(rng.normal(0, 1e-3, n + 50).astype(np.float32), np.zeros(n + 50, np.float32), L_T)
    B.adacomp_device_status_reset()
    assert B.adacomp_device_status() == 0
    got = gpu_decode([a.raw, b.raw], n)                       # n differs between the streams
    assert B.adacomp_device_status() & B.ADACOMP_DEV_HEADER_MISMATCH
    assert np.all(np.isnan(got))                              # dst left untouched
    B.adacomp_device_status_reset()
    bad = a.raw.copy()
    first_word = a.bytes_used - 16 * ((a.n_sel + 15) // 16)
    bad[first_word] = (bad[first_word] & 0xFC) | 0b10         # reserved ternary code
    got = gpu_decode([bad], n)
    assert B.adacomp_device_status() == B.ADACOMP_DEV_RESERVED_CODE
    want = cref.unpack_sum([a.raw], n)
    pos, _ = a.positions_and_codes()
    want[pos[0]] = 0.0                                        # the bad word is skipped
    assert_f32_bits_equal(got, want)
    B.adacomp_device_status_reset()
    assert B.adacomp_device_status() == 0


@pytest.mark.parametrize("L_T,n", [(50, 4000 * 6 + 77), (62, 3968 * 5 + 9), (200, 4000 * 4 + 150), (500, 4000 * 5 + 3),
                                   (1001, 4096 * 5 + 100), (5000, 5000 * 7 + 11), (16384, 16384 * 3 + 5)])
def test_decoder_flags_out_of_range_words_and_inflated_counts(L_T, n):
    """Streams that disagree with themselves (every read they ask for stays inside the stream): a word
    whose index is past its bin is skipped and flagged; a bin count that makes a tile's counts exceed
    its directory entry is flagged and costs at most that tile's neighbourhood."""
    rng = np.random.default_rng(L_T + n)
    good = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L_T)
    a = cref.pack(rng.normal(0, 1e-3, n).astype(np.float32), np.zeros(n, np.float32), L_T)
    w = a.w
    n_tiles_bytes = 8 * (a.n_tiles + 1)
    bin_cnt_at = (64 + n_tiles_bytes + 15) & ~15
    payload_at = (bin_cnt_at + a.n_bins * w + 15) & ~15
    pos, codes = a.positions_and_codes()
    alone = cref.unpack_sum([good.raw], n)
    both = cref.unpack_sum([good.raw, a.raw], n)

    # a word in the middle of the stream gets the index L_T (one past its bin's last element)
    j = a.n_sel // 2
    word = (L_T << 2) | int(codes[j])
    if word < (1 << (8 * w)):                                 # (L_T = 16384: every index a word can hold is inside the bin)
        bad = a.raw.copy()
        bad[payload_at + j * w: payload_at + (j + 1) * w] = np.frombuffer(int(word).to_bytes(w, "little"), dtype=np.uint8)
        B.adacomp_device_status_reset()
        got = gpu_decode([good.raw, bad], n)
        assert B.adacomp_device_status() == B.ADACOMP_DEV_BAD_STREAM
        want = both.copy()
        want[pos[j]] = alone[pos[j]]                          # the bad word is skipped
        assert_f32_bits_equal(got, want, f"L_T={L_T} out-of-range word")

    # a bin of a middle tile claims one word more than it has
    b = (a.n_bins // 2)
    bad = a.raw.copy()
    cnt = int(a.bin_cnt[b]) + 1
    bad[bin_cnt_at + b * w: bin_cnt_at + (b + 1) * w] = np.frombuffer(cnt.to_bytes(w, "little"), dtype=np.uint8)
    B.adacomp_device_status_reset()
    got = gpu_decode([good.raw, bad], n)
    assert B.adacomp_device_status() & B.ADACOMP_DEV_BAD_STREAM
    # everything farther than a tile (and a 4096-element work item) from that bin is untouched by it
    reach = max(a.tile_bins * L_T, 4096) + L_T
    lo, hi = max(0, b * L_T - reach), min(n, (b + 1) * L_T + reach)
    assert_f32_bits_equal(got[:lo], both[:lo], f"L_T={L_T} inflated count, before")
    assert_f32_bits_equal(got[hi:], both[hi:], f"L_T={L_T} inflated count, after")
    assert np.all(np.isfinite(got))
    B.adacomp_device_status_reset()
    assert B.adacomp_device_status() == 0


def test_nonfinite_gradient_sets_a_status_bit_and_returns():
    n = 8000
    dW = np.full(n, 1e-3, np.float32)
    dW[17] = np.inf
    dW[4100] = np.nan
    B.adacomp_device_status_reset()
    GpuLayer(n, 50).compress(dW)
    assert B.adacomp_device_status() & B.ADACOMP_DEV_NONFINITE
    B.adacomp_device_status_reset()


def test_multi_tensor_calls_match_single_calls():
    # a mix: small and mid-size layers (batched launches: the layer and its bin length change from tile to
    # tile), an empty one, bin lengths outside the batched range and one layer beyond the batch's size limit
    # (the single-layer kernels)
    specs = synth.resnet50_tensors()[:30] + [
        synth.TensorSpec("empty", 0, 50, "fc"), synth.TensorSpec("odd_bins", 12345, 7, "fc"),
        synth.TensorSpec("long_bins", 54321, 5000, "fc"), synth.TensorSpec("big", (1 << 22) + 4321, 50, "fc"),
        synth.TensorSpec("tail_of_one", 4001, 500, "conv"), synth.TensorSpec("lt42", 9999, 42, "fc"),
        synth.TensorSpec("lt1000", 99999, 1000, "fc"), synth.TensorSpec("lt333", 3996 * 7 + 5, 333, "fc"),
        synth.TensorSpec("alone", (1 << 25) + 7, 500, "fc"), synth.TensorSpec("lt64", 3840 * 3, 64, "conv")]
    dev = torch.device("cuda:0")
    layers, singles, dws = [], [], []
    for t, spec in enumerate(specs):
        dW = synth.make_dw(3, 0, t, 0, spec.n, heavy=True)
        dws.append(dW)
        L = GpuLayer(spec.n, spec.L_T)
        L.grad[:spec.n].copy_(torch.from_numpy(dW))
        layers.append(L)
    descs = [dict(grad=L.grad, residue=L.residue, n=L.n, L_T=L.L_T, packed_out=L.packed,
                  count_out=L.count) for L in layers]
    B.adacomp_compress_multi(descs, len(descs))
    torch.cuda.synchronize()
    for t, (L, spec) in enumerate(zip(layers, specs)):
        r = np.zeros(spec.n, np.float32)
        want = cref.pack(dws[t], r, spec.L_T)
        used = int(L.count[1])
        assert_stream_equal(L.packed[:used].cpu().numpy(), want, f"tensor {t}")
        assert_f32_bits_equal(L.residue_host(), r)
    # decode every layer from two "learners" (the same stream twice) in one call
    dsts = [torch.empty(max(L.n, 4), dtype=torch.float32, device=dev) for L in layers]
    packed = [p for L in layers for p in (L.packed, L.packed)]
    B.adacomp_decompress_accumulate_multi(packed, 2, dsts, len(layers))
    torch.cuda.synchronize()
    for t, L in enumerate(layers):
        used = int(L.count[1])
        raw = L.packed[:used].cpu().numpy()
        assert_f32_bits_equal(dsts[t][:L.n].cpu().numpy(), cref.unpack_sum([raw, raw], L.n))


def test_multi_tensor_calls_with_more_layers_than_one_batch_holds():
    """200 small layers: two pack batches of 100 and two decode launches; every stream and sum equals the oracle's."""
    rng = np.random.default_rng(200)
    dev = torch.device("cuda:0")
    shapes = [(int(rng.integers(1, 9000)), int(rng.choice([50, 500, 64, 333]))) for _ in range(200)]
    layers, dws = [], []
    for n, L_T in shapes:
        L = GpuLayer(n, L_T)
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        L.grad[:n].copy_(torch.from_numpy(dW))
        layers.append(L)
        dws.append(dW)
    descs = [dict(grad=L.grad, residue=L.residue, n=L.n, L_T=L.L_T, packed_out=L.packed, count_out=L.count) for L in layers]
    B.adacomp_compress_multi(descs, len(descs))
    torch.cuda.synchronize()
    raws = []
    for t, (L, (n, L_T)) in enumerate(zip(layers, shapes)):
        r = np.zeros(n, np.float32)
        want = cref.pack(dws[t], r, L_T)
        raw = L.packed[:int(L.count[1])].cpu().numpy()
        assert_stream_equal(raw, want, f"tensor {t} n={n} L_T={L_T}")
        assert_f32_bits_equal(L.residue_host(), r, f"residue {t}")
        raws.append(raw)
    dsts = [torch.empty(max(L.n, 4), dtype=torch.float32, device=dev) for L in layers]
    packed = [p for L in layers for p in (L.packed, L.packed)]
    B.adacomp_decompress_accumulate_multi_ex(packed, 2, dsts, [n for n, _ in shapes], [l for _, l in shapes], len(layers))
    torch.cuda.synchronize()
    for t, L in enumerate(layers):
        assert_f32_bits_equal(dsts[t][:L.n].cpu().numpy(), cref.unpack_sum([raws[t], raws[t]], L.n), f"sum {t}")
    assert B.adacomp_device_status() == 0


def test_random_shapes_against_the_oracle():
    """Seeded fuzz over (n, L_T, k): two carried pack() steps per learner and one dense sum."""
    rng = np.random.default_rng(20261125)
    for case in range(40):
        L_T = int(rng.choice([int(rng.integers(1, 130)), int(rng.integers(130, 1100)),
                              int(rng.integers(1100, 16385)), 50, 500]))
        n = int(rng.integers(1, 60000))
        k = int(rng.integers(1, 7))
        streams = []
        for l in range(k):
            sigma = 10.0 ** rng.uniform(-5, 1)
            dws = [synth.heavy_dw(n, sigma, rng) if rng.random() < 0.5 else
                   rng.normal(0, sigma, n).astype(np.float32) for _ in range(2)]
            layer, raws = run_steps(n, L_T, dws)
            streams.append(raws[-1])
        got = gpu_decode(streams, n)
        assert_f32_bits_equal(got, cref.unpack_sum(streams, n), f"fuzz case {case}: n={n} L_T={L_T} k={k}")
    assert B.adacomp_device_status() == 0
