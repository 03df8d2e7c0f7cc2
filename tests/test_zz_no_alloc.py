"""adacomp_compress_static: pack() for callers that are not allowed to allocate.

Some users of this library sit where cudaMalloc is unavailable: inside a runtime that
owns a fixed memory arena, in a step loop that must never trigger a device-wide
synchronisation, or behind an interface that passes them nothing but input and output
buffers.  For them the library carries its own 8 MiB scratch array; the call must then
produce exactly what adacomp_compress produces.  This file is collected last on purpose,
so that a run stopping at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_1712_02679_b200 import binding as B

STATIC_SCRATCH_BYTES = 8 << 20


def stream_bound(n, L_T):
    """Bytes of the stream alone when every element is sent (formula of include/adacomp.h)."""
    w = 1 if L_T <= 64 else 2
    tile_bins = 4 * (1000 // L_T) if L_T <= 1000 else 1
    n_bins = -(-n // L_T)
    n_tiles = -(-n_bins // tile_bins)
    r16 = lambda x: (x + 15) & ~15
    return r16(r16(r16(64 + 8 * (n_tiles + 1)) + w * n_bins) + w * n)


def test_oversized_tensor_is_refused_on_the_host():
    """The size check needs no GPU: nothing is enqueued for a tensor beyond the array."""
    lib = B.lib()
    A = 0x1000      # fake aligned pointers; never dereferenced because the check comes first
    n_too_big = STATIC_SCRATCH_BYTES + 4000
    assert lib.adacomp_compress_static(A, A, n_too_big, 50, A, A, None) == -8
    assert lib.adacomp_compress_static(A, A, n_too_big // 2 + 4000, 500, A, A, None) == -8
    assert "built-in" in B.adacomp_strerror(-8)
    assert lib.adacomp_compress_static(None, A, 10, 50, A, A, None) == -1
    assert lib.adacomp_compress_static(A, A, 10, 0, A, A, None) == -2
    assert lib.adacomp_compress_static(A + 4, A, 10, 50, A, A, None) == -3


@pytest.mark.gpu
@pytest.mark.parametrize("L_T,n", [(50, 100352), (500, 2359296), (7, 30011), (5000, 123457), (64, 3840 * 31 + 5), (333, 3996 * 9 + 1),
                                   (200, 4000 * 12 + 150), (3000, 3000 * 17 + 2), (1001, 50001)])
def test_static_scratch_matches_adacomp_compress_on_two_calls_in_a_row(L_T, n):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(L_T * 31 + n)
    res0 = torch.from_numpy(rng.normal(0, 2e-3, n).astype(np.float32)).to(dev)
    res_a, res_b = res0.clone(), res0.clone()
    cap = B.adacomp_packed_capacity(n, L_T)
    packed_a = torch.empty(cap, dtype=torch.uint8, device=dev)
    # the caller of the static variant brings only the stream's worst-case bytes
    packed_b = torch.empty(stream_bound(n, L_T), dtype=torch.uint8, device=dev)
    assert packed_b.numel() < cap
    cnt_a = torch.zeros(2, dtype=torch.int64, device=dev)
    cnt_b = torch.zeros(2, dtype=torch.int64, device=dev)
    for call in range(2):          # two calls in a row: the shared array carries stale contents
        dW = torch.from_numpy(rng.normal(0, 1e-3, n).astype(np.float32)).to(dev)
        packed_b.fill_(0xCD)
        B.adacomp_compress(dW, res_a, n, L_T, packed_a, cnt_a)
        B.adacomp_compress_static(dW, res_b, n, L_T, packed_b, cnt_b)
        torch.cuda.synchronize()
        assert torch.equal(cnt_a, cnt_b), f"call {call}"
        used = int(cnt_a[1])
        assert used <= packed_b.numel() and int(cnt_a[0]) > 0
        assert torch.equal(packed_a[:used], packed_b[:used]), f"call {call}: stream bytes differ"
        # scale and residue: the tolerance the parity tests state (1e-6 relative, 1e-7
        # absolute); the two paths run the same kernels, so the bits agree as well
        np.testing.assert_allclose(res_b.cpu().numpy(), res_a.cpu().numpy(), rtol=1e-6, atol=1e-7)
        assert torch.equal(res_a.view(torch.int32), res_b.view(torch.int32)), f"call {call}: residue"
    assert B.adacomp_device_status() == 0


@pytest.mark.gpu
def test_static_scratch_stale_contents_of_another_shape_never_leak():
    """The shared array keeps whatever the last call left.  A dense call with many tiles (every element sent)
    fills its counts and word slots; the sparse calls after it, each of another shape, must come out exactly
    as the CPU oracle packs them - streams, counts and residues byte for byte - so a count or a slot that some
    path forgot to rewrite would show.  Also the empty tensor and a tensor of a single short tile."""
    from oracle import cref
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(2024)

    def static_call(dW, res, L_T):
        n = dW.size
        g = torch.from_numpy(dW).to(dev) if n else torch.zeros(4, device=dev)
        r = torch.from_numpy(res).to(dev) if n else torch.zeros(4, device=dev)
        packed = torch.full((max(stream_bound(n, L_T), 64),), 0xCD, dtype=torch.uint8, device=dev)
        cnt = torch.zeros(2, dtype=torch.int64, device=dev)
        B.adacomp_compress_static(g, r, n, L_T, packed, cnt)
        torch.cuda.synchronize()
        n_sel, used = (int(v) for v in cnt.cpu())
        return packed[:used].cpu().numpy(), n_sel, r[:n].cpu().numpy()

    def dense_call():
        n = 4000 * 600 + 37                  # every element ties for its bin's maximum: all of them are sent
        dW = (np.where(rng.random(n) < 0.5, -1.0, 1.0) * 0.25).astype(np.float32)
        raw, n_sel, _ = static_call(dW, np.zeros(n, np.float32), 50)
        assert n_sel == n
        return raw

    dense_call()
    for L_T, n in [(500, 4000 * 150 + 11), (7, 30011), (5000, 5000 * 40 + 123), (50, 100352), (50, 0), (50, 37), (500, 499)]:
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        res = rng.normal(0, 2e-3, n).astype(np.float32)
        want_res = res.copy()
        want = cref.pack(dW, want_res, L_T)
        raw, n_sel, got_res = static_call(dW, res, L_T)
        assert n_sel == want.n_sel and raw.size == want.bytes_used, (L_T, n)
        assert np.array_equal(raw, want.raw), f"L_T={L_T} n={n}: stream differs from the oracle's"
        assert np.array_equal(got_res.view(np.uint32), want_res.view(np.uint32)), f"L_T={L_T} n={n}: residue"
        dense_call()                         # and dirty the array again before the next shape
    assert B.adacomp_device_status() == 0


@pytest.mark.gpu
def test_static_scratch_largest_supported_and_first_refused_size():
    dev = torch.device("cuda:0")
    # largest n whose scratch still fits the array (the scratch grows with n), by bisection
    lo, hi = 4000, STATIC_SCRATCH_BYTES + 4000
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if scratch_bytes(mid, 50) <= STATIC_SCRATCH_BYTES:
            lo = mid
        else:
            hi = mid
    n = lo
    dW = torch.randn(n, device=dev) * 1e-3
    res_a = torch.zeros(n, device=dev)
    res_b = torch.zeros(n, device=dev)
    pa = torch.empty(B.adacomp_packed_capacity(n, 50), dtype=torch.uint8, device=dev)
    pb = torch.empty(stream_bound(n, 50), dtype=torch.uint8, device=dev)
    ca = torch.zeros(2, dtype=torch.int64, device=dev)
    cb = torch.zeros(2, dtype=torch.int64, device=dev)
    B.adacomp_compress(dW, res_a, n, 50, pa, ca)
    B.adacomp_compress_static(dW, res_b, n, 50, pb, cb)
    torch.cuda.synchronize()
    used = int(ca[1])
    assert torch.equal(ca, cb) and torch.equal(pa[:used], pb[:used])
    assert torch.equal(res_a.view(torch.int32), res_b.view(torch.int32))
    with pytest.raises(B.AdaCompError) as e:
        B.adacomp_compress_static(dW, res_b, hi, 50, pb, cb)
    assert e.value.code == -8


def scratch_bytes(n, L_T):
    """Scratch the compressor needs: control block, group and tile counts, one slot per tile."""
    w = 1 if L_T <= 64 else 2
    tile_bins = 4 * (1000 // L_T) if L_T <= 1000 else 1
    n_bins = -(-n // L_T)
    n_tiles = -(-n_bins // tile_bins)
    n_groups = -(-n_tiles // 32)
    slots_at = (256 + 8 * n_groups + 4 * n_tiles + 255) & ~255
    return slots_at + n_tiles * ((tile_bins * L_T * w + 15) & ~15)
