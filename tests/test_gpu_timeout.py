"""The bounded device-side waits, exercised without a fault: one CTA's copy engine is told to announce a copy and
never start it (adacomp_debug_waits), and the wait for it is cut to about a millisecond.  The kernel must raise
ADACOMP_DEV_TIMEOUT and return, the kernels behind it must stay inside their buffers, everything the other CTAs
did must be complete, and the library must work as before afterwards."""
import numpy as np
import pytest
import torch

from oracle import cref
from paper_1712_02679_b200 import binding as B
from tests.gpu_util import assert_f32_bits_equal, assert_stream_equal

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
LIMIT = 2_000_000          # cycles: about a millisecond


@pytest.fixture(autouse=True)
def restore_waits():
    yield
    B.adacomp_debug_waits(0, 0, 0)
    B.adacomp_device_status_reset()


def sms():
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("L_T,lazy", [(50, False), (500, False), (50, True)])
def test_tile_pass_times_out_on_a_withheld_load_and_everything_else_is_done(L_T, lazy):
    grid = 2 * sms()                                  # CTAs of the pipelined tile pass
    n_tiles = 5 * grid + 7
    n = 4000 * n_tiles - 123
    rng = np.random.default_rng(L_T)
    r0 = rng.normal(0, 2e-3, n).astype(np.float32)
    dW = rng.normal(0, 1e-3, n).astype(np.float32)
    res = torch.from_numpy(r0).to(DEV)
    g = torch.from_numpy(dW).to(DEV)
    packed = torch.empty(B.adacomp_packed_capacity(n, L_T), dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(2, dtype=torch.int64, device=DEV)
    state = None
    if lazy:
        state = torch.empty(B.adacomp_lazy_state_bytes(n, L_T), dtype=torch.uint8, device=DEV)
        B.adacomp_lazy_state_init(state, n, L_T)
    B.adacomp_device_status_reset()
    B.adacomp_debug_waits(LIMIT, 2, 0)                # CTA 0 never gets its third tile
    B.adacomp_compress_opt(g, res, n, L_T, packed, cnt, lazy_state=state)
    torch.cuda.synchronize()                          # the kernels returned
    assert B.adacomp_device_status() & B.ADACOMP_DEV_TIMEOUT
    B.adacomp_debug_waits(0, 0, 0)
    n_sel, used = (int(v) for v in cnt.cpu())
    assert 0 < n_sel < n and 0 < used <= packed.numel()
    got = res.cpu().numpy()
    G = r0 + dW                                       # (one rounded binary32 addition, as Algorithm 2's first line)
    tile_of = np.arange(n) // 4000
    mine = tile_of % grid == 0                        # CTA 0's tiles: 0, grid, 2 grid, ...
    untouched = mine & (tile_of >= 2 * grid)          # from the withheld one on: nothing written
    assert_f32_bits_equal(got[untouched], r0[untouched], "tiles CTA 0 never finished")
    done = ~untouched
    # every other tile was processed: the elements nobody sent hold G exactly (the sent ones were finished with the
    # scale of an incomplete sum, or, in lazy-scale mode, hold G as well)
    same = got[done].view(np.uint32) == G[done].view(np.uint32)
    assert same.mean() > 0.75
    if lazy:
        assert same.all()
    # the stream is self-consistent: the directory is monotone and ends at n_sel
    geo_tiles = n_tiles
    tile_off = packed[64:64 + 8 * (geo_tiles + 1)].cpu().numpy().view(np.uint64)
    assert np.all(np.diff(tile_off.astype(np.int64)) >= 0) and int(tile_off[-1]) == n_sel
    # and the library is as good as new: the same call again, on fresh data, matches the oracle bit for bit
    B.adacomp_device_status_reset()
    r1 = rng.normal(0, 2e-3, n).astype(np.float32)
    res.copy_(torch.from_numpy(r1))
    if lazy:
        B.adacomp_lazy_state_init(state, n, L_T)
    want = cref.pack(dW, r1, L_T)
    B.adacomp_compress_opt(g, res, n, L_T, packed, cnt, lazy_state=state)
    torch.cuda.synchronize()
    assert_stream_equal(packed[:int(cnt[1])].cpu().numpy(), want, "after the time-out")
    assert B.adacomp_device_status() == 0


@pytest.mark.parametrize("L_T,n_items_per_cta", [(50, 6), (500, 6), (5000, 6)])
def test_decoder_times_out_on_a_withheld_slot_and_every_other_item_is_written(L_T, n_items_per_cta):
    k = 3
    rng = np.random.default_rng(L_T + 1)
    # enough work items for every CTA of the decoder to take several (items: pairs of tiles at L_T = 50 from 256
    # tiles on, tiles at 500, 4096 elements at 5000)
    n = 4096 * 8 * sms() * n_items_per_cta + 321
    raws = []
    for l in range(k):
        dW = rng.normal(0, 1e-3, n).astype(np.float32)
        raws.append(cref.pack(dW, np.zeros(n, np.float32), L_T).raw)
    bufs = [torch.from_numpy(r.copy()).to(DEV) for r in raws]
    want = cref.unpack_sum(raws, n)
    dst = torch.full((n,), float("nan"), device=DEV)
    B.adacomp_device_status_reset()
    B.adacomp_debug_waits(LIMIT, 0, 2)                # CTA 0's loader leaves out its third item
    B.adacomp_decompress_accumulate_ex(bufs, k, dst, n, L_T)
    torch.cuda.synchronize()
    assert B.adacomp_device_status() & B.ADACOMP_DEV_TIMEOUT
    B.adacomp_debug_waits(0, 0, 0)
    got = dst.cpu().numpy()
    written = ~np.isnan(got)
    assert 0.5 < written.mean() < 1.0                 # CTA 0's later items stay unwritten, nothing else does
    assert_f32_bits_equal(got[written], want[written], "items that were decoded")
    # the first element of the tensor belongs to CTA 0's first item, which was decoded before the time-out
    assert written[0] and written[100]
    B.adacomp_device_status_reset()
    B.adacomp_decompress_accumulate_ex(bufs, k, dst, n, L_T)
    torch.cuda.synchronize()
    assert_f32_bits_equal(dst.cpu().numpy(), want, "after the time-out")
    assert B.adacomp_device_status() == 0
