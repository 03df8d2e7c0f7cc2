// Batched decode-sum: the kernels of the *_multi decode entry points and their launcher (see decode_batch.cuh).
#include "internal.h"

namespace adacomp_impl {

struct DecodeBatchSmem {
    DecodeSmem d;
    Geometry geo[kDecBatchLayers];
    u32 first[kDecBatchLayers + 1];                  // global index of each layer's first tile
};

__global__ void __launch_bounds__(kDecodeThreads)
decode_batch(const __grid_constant__ DecodeBatchArgs b)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecodeBatchSmem &sm = *reinterpret_cast<DecodeBatchSmem *>(smem_raw);
    const int tid = threadIdx.x;
    u32 bad = 0;
    // every CTA checks every layer's k headers against the shape the caller gave and indexes the
    // tiles of the layers that pass; a layer that fails is skipped (dst untouched) and reported
    for (int t = tid; t < (int)b.n_layers; t += kDecodeThreads) {
        const Geometry g = make_geometry(b.n[t], b.L_T[t]);
        bool ok = true;
        for (u32 l = 0; l < b.k; l++) {     // (no early exit: the k headers' loads go out together)
            const u32 *h = reinterpret_cast<const u32 *>(b.stream[t * b.k + l]);
            const u64 *h64 = reinterpret_cast<const u64 *>(h);
            ok &= h[0] == kMagic && (h[1] & 0xffffu) == 1u && h[2] == g.L_T && h64[2] == g.n &&
                  ((h[1] >> 16) & 0xffu) == g.w && h[3] == g.tile_bins && h64[3] == g.n_bins &&
                  h64[4] == g.n_tiles && h64[5] <= g.n;
        }
        if (!ok) bad |= ADACOMP_DEV_HEADER_MISMATCH;
        sm.geo[t] = g;
        sm.first[t + 1] = ok ? (u32)g.n_tiles : 0u;
    }
    for (int i = tid; i < kDecodeChunk; i += kDecodeThreads) sm.d.acc[i] = 0.f;
    consumer_barrier();
    if (tid == 0) {
        u32 run = 0;
        sm.first[0] = 0;
        for (u32 t = 0; t < b.n_layers; t++) {
            run += sm.first[t + 1];
            sm.first[t + 1] = run;
        }
    }
    consumer_barrier();
    const u32 total = sm.first[b.n_layers];
    for (u32 gt = blockIdx.x; gt < total; gt += gridDim.x) {
        int lo = 0, hi = (int)b.n_layers;            // largest t with first[t] <= gt and a tile of its own
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (sm.first[mid] <= gt) lo = mid; else hi = mid;
        }
        const Geometry &geo = sm.geo[lo];
        const u64 tile = gt - sm.first[lo];
        const unsigned char *const *streams = &b.stream[lo * b.k];
        const Epilogue ep = {b.opt ? b.dst[lo] : nullptr, b.opt ? b.aux[lo] : nullptr, b.opt == 2u ? b.aux2[lo] : nullptr,
                             b.lr, b.mu, b.beta2, b.eps, (float)b.k, b.opt == 2u ? 1u : 0u,
                             (b.k & (b.k - 1u)) == 0u ? __frcp_rn((float)b.k) : 0.f};
        if (geo.w == 1u) {
            decode_item_staged<unsigned char, true>(streams, b.k, geo, tile, b.dst[lo], ep, sm.d, bad);
        } else if (geo.tile_bins >= 32) {
            decode_item_staged<unsigned short, true>(streams, b.k, geo, tile, b.dst[lo], ep, sm.d, bad);
        } else {
            decode_item_staged<unsigned short, false>(streams, b.k, geo, tile, b.dst[lo], ep, sm.d, bad);
        }
    }
    if (bad && blockIdx.x == 0) raise_status(bad & ADACOMP_DEV_HEADER_MISMATCH);
    if (bad & ~ADACOMP_DEV_HEADER_MISMATCH) raise_status(bad & ~ADACOMP_DEV_HEADER_MISMATCH);
}

// ---------------------------------------------------------------------------------
// Batched decode-sum, warp path: the loader warp and the four free-running decoding warps of
// decode_warps over the tiles of a whole batch of layers (global tile gt belongs to the layer whose
// first tile is the largest not above it).  What decode_warps takes from one tensor's shape travels
// per layer in shared memory; the slots are laid out once per launch, with the learners' word regions
// sized from the batch-wide average bytes per tile (1.5 times it plus slack) and the room for the bin
// counts from the largest count run among the layers; a learner's scale and word total come into the
// slot with its directory entries.  Every layer here has 42 <= L_T <= 1000.  OPT: 0 the finished tiles go
// to dst; 1 (SGD) / 2 (Adam) they feed the optimizer step on the layer's weights instead (see Epilogue), the
// warp reading and writing its share of the optimizer's arrays itself.
// ---------------------------------------------------------------------------------
struct BatchLayerCtx {
    u64 n, n_bins, bin_cnt_at, payload_at;
    u32 L_T, TB, T, w;
};
// (as WarpDecSmem, without the ring: it is dynamic shared memory here, sized by the launcher from k)
struct WarpBatchCtl {
    u32 tmp[4][32];
    unsigned short coff[ADACOMP_MAX_STREAMS], wcap[ADACOMP_MAX_STREAMS];
    unsigned char rfirst[ADACOMP_MAX_STREAMS], rcount[ADACOMP_MAX_STREAMS];
    u64 full[kSlots], empty[kSlots];
    u32 slot_bytes, n_slots, n_rounds, abort;
};
struct WarpBatchSmem {
    WarpBatchCtl ws;
    BatchLayerCtx ctx[kDecBatchLayers];
    u32 first[kDecBatchLayers + 1];                  // global index of each layer's first tile
    unsigned long long bytes_total[ADACOMP_MAX_STREAMS];   // payload bytes of learner l over the batch
    u64 layer_bar;                                   // the decoding warps meet here when the layer changes
    u32 count_room_max, bad;
};

template <int OPT>
__global__ void __launch_bounds__(kDecodeLaunch, 4)
decode_batch_warps(const __grid_constant__ DecodeBatchArgs b, u32 ring_bytes)
{
    constexpr int NW = 4;
    constexpr u32 full_mask = 0xffffffffu;
    extern __shared__ __align__(16) unsigned char ring[];           // ring_bytes: the slots
    __shared__ __align__(16) float s_acc[kDecodeChunk];
    __shared__ __align__(16) WarpBatchSmem sm;
    WarpBatchCtl &ws = sm.ws;
    const u32 slot_max = ring_bytes / 2;        // a slot never takes more: two items are always in flight
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u32 k = b.k, n_layers = b.n_layers;

    // ---- every CTA checks every layer's k headers against the shape the caller gave and indexes the
    // tiles of the layers that pass; a layer that fails is skipped (dst untouched) and reported ----
    if (tid < (int)ADACOMP_MAX_STREAMS) sm.bytes_total[tid] = 0;
    if (tid == 0) {
        sm.count_room_max = 16;
        sm.bad = 0;
    }
    for (int i = tid; i < kDecodeChunk; i += blockDim.x) s_acc[i] = 0.f;
    __syncthreads();
    for (u32 t = tid; t < n_layers; t += blockDim.x) {
        const Geometry g = make_geometry(b.n[t], b.L_T[t]);
        bool ok = g.tile_bins >= 4u && g.tile_bins <= (u32)kSmallBins && g.tile_bins % 4u == 0 && g.tile_elems <= (u32)kDecodeChunk;
        // (no early exit: the k headers' loads go out together; a failing layer's words only widen the regions)
        for (u32 l = 0; l < k; l++) {
            const u32 *h = reinterpret_cast<const u32 *>(b.stream[t * k + l]);
            const u64 *h64 = reinterpret_cast<const u64 *>(h);
            const u64 n_sel = h64[5];
            ok &= h[0] == kMagic && (h[1] & 0xffffu) == 1u && h[2] == g.L_T && h64[2] == g.n &&
                  ((h[1] >> 16) & 0xffu) == g.w && h[3] == g.tile_bins && h64[3] == g.n_bins &&
                  h64[4] == g.n_tiles && n_sel <= g.n;
            atomicAdd(&sm.bytes_total[l], min(n_sel, g.n) * (u64)g.w);
        }
        if (ok) {
            const u32 run = g.tile_bins * g.w;
            atomicMax(&sm.count_room_max, run % 16u == 0 ? run : (u32)align_up(run + 15u, 16));
        } else {
            atomicOr(&sm.bad, (u32)ADACOMP_DEV_HEADER_MISMATCH);
        }
        sm.ctx[t] = BatchLayerCtx{g.n, g.n_bins, g.bin_cnt_at, g.payload_at, g.L_T, g.tile_bins, g.tile_elems, g.w};
        sm.first[t + 1] = ok ? (u32)g.n_tiles : 0u;
    }
    __syncthreads();
    if (tid == 0) {
        u32 run = 0;
        sm.first[0] = 0;
        for (u32 t = 0; t < n_layers; t++) {
            run += sm.first[t + 1];
            sm.first[t + 1] = run;
        }
        for (int s = 0; s < kSlots; s++) {
            mbar_init(&ws.full[s], 32);
            mbar_init(&ws.empty[s], NW);
        }
        mbar_init(&sm.layer_bar, NW);
        ws.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (sm.bad && blockIdx.x == 0) raise_status(sm.bad);
    }
    __syncthreads();
    const u32 total = sm.first[n_layers];
    const u32 count_bytes = sm.count_room_max;                     // room of a learner's bin counts in a slot
    const u32 k8 = (k + 7u) & ~7u;
    const u32 meta_bytes = kSlotHead + 8u * k8;                    // slot header + u16 cnt[k8], u16 head[k8], u32 scale bits[k8]
    if (warp == NW) {
        // the learners' regions (as decode_warps_any, from the batch's totals), then the rounds
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const u32 l = (u32)lane + 32u * h;
            if (l < k) {
                const u64 avg = total ? sm.bytes_total[l] / total : 0;
                const u64 cap = min((u64)kDecodeChunk * 2u, avg + avg / 2 + 128);
                ws.wcap[l] = (unsigned short)min(align_up(cap + 16, 16), (u64)((slot_max - meta_bytes - count_bytes) & ~15u));
            }
        }
        __syncwarp();
        if (lane == 0) {
            u32 r = 0, used = meta_bytes, most = 0, r0 = 0;
            for (u32 l = 0; l < k; l++) {
                const u32 need = count_bytes + ws.wcap[l];
                if (used + need > slot_max && l > r0) {
                    ws.rfirst[r] = (unsigned char)r0;
                    ws.rcount[r] = (unsigned char)(l - r0);
                    r++;
                    r0 = l;
                    used = meta_bytes;
                }
                ws.coff[l] = (unsigned short)used;
                used += need;
                most = max(most, used);
            }
            ws.rfirst[r] = (unsigned char)r0;
            ws.rcount[r] = (unsigned char)(k - r0);
            ws.n_rounds = r + 1u;
            ws.slot_bytes = most;
            ws.n_slots = min((u32)kSlots, ring_bytes / most);
        }
    }
    __syncthreads();

    const u32 first = blockIdx.x, stride = gridDim.x;
    const u32 my_tiles = total > first ? (total - first + stride - 1) / stride : 0;
    const u32 NR = ws.n_rounds, slot_bytes = ws.slot_bytes, S = ws.n_slots;
    auto seek = [&](u32 gt, u32 &li) {      // (tiles only go up; layers without tiles are stepped over)
        while (li + 1 < n_layers && sm.first[li + 1] <= gt) li++;
    };

    if (warp == NW) {
        // ================================ loader warp ================================
        // An item is one round of one tile; lane j (and j + 32) looks after the j-th learner of the round.
        // Its directory entries, word total and scale are read two items ahead.
        u64 da0[2] = {0, 0}, da1[2] = {0, 0}, db0[2] = {0, 0}, db1[2] = {0, 0}, dan[2] = {0, 0}, dbn[2] = {0, 0};
        u32 das[2] = {0, 0}, dbs[2] = {0, 0};
        u32 pli = 0, pgt = first, pit = 0, pr = 0;          // the item two ahead: its layer, tile, index and round
        auto load_dir = [&](u64 *d0, u64 *d1, u64 *dn, u32 *ds) {
            if (pit >= my_tiles) return;
            seek(pgt, pli);
            const u32 lt = pgt - sm.first[pli];
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const u32 j = (u32)lane + 32u * h;
                if (j < (u32)ws.rcount[pr]) {
                    const unsigned char *st = b.stream[pli * k + (u32)ws.rfirst[pr] + j];
                    const u64 *dir = reinterpret_cast<const u64 *>(st + kHeaderBytes);
                    d0[h] = dir[lt];
                    d1[h] = dir[lt + 1];
                    dn[h] = reinterpret_cast<const u64 *>(st)[5];
                    ds[h] = reinterpret_cast<const u32 *>(st)[12];
                }
            }
        };
        auto step_ahead = [&]() {
            if (++pr == NR) {
                pr = 0;
                pgt += stride;
                pit++;
            }
        };
        load_dir(da0, da1, dan, das);
        step_ahead();
        load_dir(db0, db1, dbn, dbs);
        step_ahead();
        u32 issued = 0, s = 0, use = 0, li = 0;
        bool failed = false;
        for (u32 it = 0; it < my_tiles && !failed; it++) {
            const u32 gt = first + it * stride;
            seek(gt, li);
            const BatchLayerCtx c = sm.ctx[li];
            const u32 lt = gt - sm.first[li];
            const u64 bin0 = (u64)lt * c.TB;
            const u32 live = (u32)min((u64)c.TB, c.n_bins - bin0);
            // the tile's bin counts start `clead` bytes behind a 16-byte boundary: the copy starts at the boundary
            const u32 clead = (u32)(bin0 * c.w) & 15u;
            const u32 cbytes = (u32)align_up(clead + live * c.w, 16);
            for (u32 r = 0; r < NR; r++, s = s + 1u == S ? 0u : s + 1u, use += s == 0u) {
                if (use > 0 && !mbar_wait(&ws.empty[s], (use - 1u) & 1u)) {
                    ws.abort = 1;
                    raise_status(ADACOMP_DEV_TIMEOUT);
                    failed = true;      // the decoding warps time out on the full barrier in turn
                    break;
                }
                if (*reinterpret_cast<volatile u32 *>(&ws.abort)) {
                    failed = true;
                    break;
                }
                unsigned char *sl = ring + s * slot_bytes;
                unsigned short *m_cnt = reinterpret_cast<unsigned short *>(sl + kSlotHead), *m_head = m_cnt + k8;
                u32 *m_scale = reinterpret_cast<u32 *>(m_head + k8);
                const u32 l0 = ws.rfirst[r], nl = ws.rcount[r];
                u64 src[2] = {0, 0};
                u32 wbytes[2] = {0, 0}, coff[2] = {0, 0};
                u32 staged = 0, bad = 0;
                bool open = true;
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const u32 j = (u32)lane + 32u * h;
                    const bool active = j < nl;
                    bool ok = true, fit = false;
                    if (active) {
                        const u32 l = l0 + j;
                        ok = da1[h] >= da0[h] && da1[h] - da0[h] <= c.T && da1[h] <= dan[h];
                        const u32 cnt = ok ? (u32)(da1[h] - da0[h]) : 0u;
                        src[h] = (u64)(uintptr_t)(b.stream[li * k + l] + c.payload_at) + da0[h] * c.w;
                        const u32 head = (u32)(src[h] & 15u);
                        wbytes[h] = cnt ? (u32)align_up(head + cnt * c.w, 16) : 0u;
                        fit = wbytes[h] <= (u32)ws.wcap[l];
                        coff[h] = ws.coff[l];
                        m_cnt[j] = (unsigned short)cnt;
                        m_head[j] = (unsigned short)head;
                        m_scale[j] = das[h];
                    }
                    if (__any_sync(full_mask, active && !ok)) bad |= ADACOMP_DEV_BAD_STREAM;
                    const u32 fits = __ballot_sync(full_mask, active && open && fit);
                    const int lead = __ffs(~fits) - 1;
                    const int staged_lanes = lead < 0 ? 32 : lead;
                    staged += (u32)staged_lanes;
                    if (staged_lanes < 32) open = false;
                    if (nl <= 32u) break;
                }
                if (lane == 0) {
                    reinterpret_cast<u32 *>(sl)[0] = staged;
                    reinterpret_cast<u32 *>(sl)[1] = bad;
                }
                __syncwarp();
                u32 expect = 0;
#pragma unroll
                for (int h = 0; h < 2; h++)
                    if ((u32)lane + 32u * h < staged) expect += cbytes + wbytes[h];
                if (expect) mbar_arrive_expect_tx(&ws.full[s], expect);
                else mbar_arrive(&ws.full[s]);
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const u32 j = (u32)lane + 32u * h;
                    if (j < staged) {
                        bulk_load(sl + coff[h], b.stream[li * k + l0 + j] + c.bin_cnt_at + (bin0 * c.w - clead), cbytes, &ws.full[s]);
                        if (wbytes[h])
                            bulk_load(sl + coff[h] + count_bytes, reinterpret_cast<const void *>(src[h] & ~(u64)15u), wbytes[h],
                                      &ws.full[s]);
                    }
                }
                issued++;
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    da0[h] = db0[h];
                    da1[h] = db1[h];
                    dan[h] = dbn[h];
                    das[h] = dbs[h];
                }
                load_dir(db0, db1, dbn, dbs);
                step_ahead();
            }
        }
        if (*reinterpret_cast<volatile u32 *>(&ws.abort)) {
            // after a timeout the copies already started must land (or time out in turn) before
            // this CTA's shared memory is given back
            for (u32 j = issued > S ? issued - S : 0; j < issued; j++) mbar_wait(&ws.full[j % S], (j / S) & 1u);    // (rare)
        }
        return;
    }

    // =============================== decoding warps ===============================
    u32 *const tmp = ws.tmp[warp];
    u32 li = 0, at_li = 0xffffffffu, s = 0, use = 0, bad = 0, switches = 0;
    // what depends on the layer (see decode_warps)
    u32 L_T = 0, wb = 1, quarter = 0, acc_at = 0, mine_at = 0;
    int TB = 0, nb = 0, b0 = 0, G = 1, my_bin = 0, my_r = 0;
    bool by_bin = true, vec_store = false;
    float *my_acc = s_acc;
    bool failed = false;
    for (u32 it = 0; it < my_tiles; it++) {
        const u32 gt = first + it * stride;
        seek(gt, li);
        const BatchLayerCtx &c = sm.ctx[li];
        if (li != at_li) {
            // (layers of one bin length and word width, as most neighbours in a list are, cut the tile alike)
            if (at_li != 0xffffffffu && !(c.L_T == L_T && (int)c.TB == TB && c.w == wb)) {
                // a warp's share of the output tile moves with the bin length: every warp has stored and
                // zeroed its old share before any adds into its new one (a bounded wait, as all of them)
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.layer_bar);
                if (!mbar_wait(&sm.layer_bar, switches & 1u)) {
                    ws.abort = 1;
                    bad |= ADACOMP_DEV_TIMEOUT;
                    break;
                }
                switches++;
            }
            at_li = li;
            L_T = c.L_T;
            wb = c.w;
            TB = (int)c.TB;
            nb = TB / NW;
            b0 = warp * nb;
            quarter = (u32)nb * L_T;
            acc_at = smem_addr(s_acc) + (u32)warp * quarter * 4u;
            my_acc = s_acc + (u32)warp * quarter;
            vec_store = (quarter & 3u) == 0 && (c.T & 3u) == 0;
            by_bin = wb == 2u || TB <= 64;
            G = nb <= 32 ? 32 / nb : 1;
            const int my_local = lane / G;
            my_r = lane % G;
            my_bin = my_local < nb ? b0 + my_local : TB;
            mine_at = smem_addr(s_acc) + (u32)my_bin * L_T * 4u;
        }
        const u32 lt = gt - sm.first[li];
        const u64 bin0 = (u64)lt * (u64)TB;
        const u32 live = (u32)min((u64)TB, c.n_bins - bin0);
        const u32 clead = (u32)(bin0 * wb) & 15u;
        const u64 out0 = (u64)lt * (u64)c.T + (u64)warp * quarter;
        const u32 len = out0 < c.n ? (u32)min((u64)quarter, c.n - out0) : 0u;
        const bool whole = vec_store && len == quarter;
        float *const dst = b.dst[li];
        for (u32 r = 0; r < NR; r++, s = s + 1u == S ? 0u : s + 1u, use += s == 0u) {
            if (!mbar_wait(&ws.full[s], use & 1u)) {
                ws.abort = 1;
                bad |= ADACOMP_DEV_TIMEOUT;
                failed = true;
                break;
            }
            const unsigned char *sl = ring + s * slot_bytes;
            const u32 l0 = ws.rfirst[r], nl = ws.rcount[r];
            const u32 staged = min(reinterpret_cast<const u32 *>(sl)[0], nl);
            if (warp == 0) bad |= reinterpret_cast<const u32 *>(sl)[1];
            const unsigned short *m_cnt = reinterpret_cast<const unsigned short *>(sl + kSlotHead), *m_head = m_cnt + k8;
            const u32 *m_scale = reinterpret_cast<const u32 *>(m_head + k8);
            const u32 sl_at = smem_addr(sl);

            // ---- the round's learners whose words wait in the slot, four at a time ----
            for (u32 g0 = 0; g0 < staged; g0 += kRoundMax) {
                const int R = (int)min((u32)kRoundMax, staged - g0);
                GroupSrc<u32> src = {0u, 0u, 0u, 0u};
                if (lane < R) {
                    const u32 j = g0 + (u32)lane, l = l0 + j;
                    src.counts = sl_at + ws.coff[l] + clead;
                    src.words = sl_at + ws.coff[l] + count_bytes + m_head[j];
                    src.limit = m_cnt[j];
                    src.sbits = m_scale[j];
                }
                if (wb == 2u) bad |= warp_add_group_by_bin<unsigned short, true, u32>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else if (by_bin) bad |= warp_add_group_by_bin<unsigned char, true, u32>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else bad |= warp_add_group<unsigned char, true, u32>(src, R, b0, nb, live, L_T, acc_at, tmp, lane);
            }
            // the scales of the round's other learners, before the slot goes back
            u32 rest_scale[2] = {0u, 0u};
#pragma unroll
            for (int h = 0; h < 2; h++)
                if ((u32)lane + 32u * h < nl) rest_scale[h] = m_scale[(u32)lane + 32u * h];
            __syncwarp();
            if (lane == 0) mbar_arrive(&ws.empty[s]);

            // ---- the round's others: read from global memory ----
            for (u32 g0 = staged; g0 < nl; g0 += kRoundMax) {
                const int R = (int)min((u32)kRoundMax, nl - g0);
                GroupSrc<u64> src = {0ull, 0ull, 0u, 0u};
                bool ok = true;
                const u32 sb_lo = __shfl_sync(full_mask, rest_scale[0], (g0 + (u32)lane) & 31u);
                const u32 sb_hi = __shfl_sync(full_mask, rest_scale[1], (g0 + (u32)lane) & 31u);
                if (lane < R) {
                    const u32 j = g0 + (u32)lane, l = l0 + j;
                    const unsigned char *st = b.stream[li * k + l];
                    const u64 *dir = reinterpret_cast<const u64 *>(st + kHeaderBytes);
                    const u64 w0 = dir[lt], w1 = dir[lt + 1];
                    ok = w1 >= w0 && w1 - w0 <= c.T && w1 <= reinterpret_cast<const u64 *>(st)[5];
                    src.counts = (u64)__cvta_generic_to_global(st + c.bin_cnt_at) + bin0 * wb;
                    src.words = (u64)__cvta_generic_to_global(st + c.payload_at) + (ok ? w0 : 0) * wb;
                    src.limit = ok ? (u32)(w1 - w0) : 0u;
                    src.sbits = j < 32u ? sb_lo : sb_hi;
                }
                if (__any_sync(full_mask, !ok)) bad |= ADACOMP_DEV_BAD_STREAM;
                if (wb == 2u) bad |= warp_add_group_by_bin_global<unsigned short>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else if (by_bin) bad |= warp_add_group_by_bin_global<unsigned char>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else bad |= warp_add_group_global<unsigned char>(src, R, b0, nb, live, L_T, acc_at, tmp, lane);
            }
        }
        if (failed) break;

        // ---- store the warp's quarter of the tile (and leave it zeroed for the next one) ----
        if (OPT != 0) {
            // averageGradients() + updateWeights() on the warp's quarter; dst is the layer's weights
            const Epilogue ep = {dst, b.aux[li], OPT == 2 ? b.aux2[li] : nullptr, b.lr, b.mu, b.beta2, b.eps, (float)k,
                                 OPT == 2 ? 1u : 0u, (k & (k - 1u)) == 0u ? __frcp_rn((float)k) : 0.f};
            if (whole) {
                float4 *w4 = reinterpret_cast<float4 *>(ep.weights + out0), *v4 = reinterpret_cast<float4 *>(ep.momentum + out0);
                float4 *u4 = OPT == 2 ? reinterpret_cast<float4 *>(ep.second + out0) : nullptr;
                float4 *s4 = reinterpret_cast<float4 *>(my_acc);
                for (int at = lane; at < (int)(quarter >> 2); at += 32) {
                    float4 w = w4[at], v = v4[at];
                    if (OPT == 2) {
                        float4 u = u4[at];
                        adam_step4(s4[at], w, v, u, ep);
                        u4[at] = u;
                    } else {
                        sgd_step4(s4[at], w, v, ep);
                    }
                    s4[at] = make_float4(0.f, 0.f, 0.f, 0.f);
                    v4[at] = v;
                    w4[at] = w;
                }
            } else {
                for (u32 i = lane; i < quarter; i += 32) {
                    if (i < len) {
                        float w = ep.weights[out0 + i], v = ep.momentum[out0 + i];
                        if (OPT == 2) {
                            float u = ep.second[out0 + i];
                            adam_step(my_acc[i], w, v, u, ep);
                            ep.second[out0 + i] = u;
                        } else {
                            sgd_step(my_acc[i], w, v, ep);
                        }
                        ep.momentum[out0 + i] = v;
                        ep.weights[out0 + i] = w;
                    }
                    my_acc[i] = 0.f;
                }
            }
        } else if (whole) {
            fence_async_smem();                     // this lane's adds, for the copy engine
            __syncwarp();
            if (lane == 0) {
                bulk_store(dst + out0, my_acc, quarter * 4u);
                bulk_commit();
                bulk_wait_read_all();               // shared memory has been read: it can be zeroed
            }
            __syncwarp();
            float4 *s4 = reinterpret_cast<float4 *>(my_acc);
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int at = lane; at < (int)(quarter >> 2); at += 32) s4[at] = zero;
        } else {
            for (u32 i = lane; i < quarter; i += 32) {
                if (i < len) dst[out0 + i] = my_acc[i];
                my_acc[i] = 0.f;
            }
        }
        __syncwarp();                               // zeroed before the next tile's adds
    }
    if (lane == 0) bulk_wait_all();                // the last copies leave shared memory before the CTA ends
    if (bad) raise_status(bad);
}


void init_decode_batch_info(DeviceInfo &d)
{
    if (cudaFuncSetAttribute(decode_batch, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)sizeof(DecodeBatchSmem)) == cudaSuccess) {
        int per = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, decode_batch, kDecodeThreads, sizeof(DecodeBatchSmem));
        d.dec_batch_per_sm = per;
        auto batch_warps_ready = [&](auto kernel, int o) {
            int q = 0;
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&q, kernel, kDecodeLaunch, kBatchRingBytes);
            d.dec_batch_warps_per_sm[o] = q;
        };
        batch_warps_ready(decode_batch_warps<0>, 0);
        batch_warps_ready(decode_batch_warps<1>, 1);
        batch_warps_ready(decode_batch_warps<2>, 2);
    }
}

// One launch for the layers of `batch` (batch_tiles work items over all of them).
int launch_decode_batch(const DecodeBatchArgs &batch, u64 batch_tiles, const DeviceInfo &info, cudaStream_t st)
{
    if (info.dec_batch_warps_per_sm[batch.opt] > 0) {
        const u32 ring = kBatchRingBytes;
        const u64 cap = (u64)info.sms * info.dec_batch_warps_per_sm[batch.opt];
        const unsigned grid = (unsigned)(batch_tiles < cap ? (batch_tiles ? batch_tiles : 1) : cap);
        if (batch.opt == 2u) decode_batch_warps<2><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
        else if (batch.opt == 1u) decode_batch_warps<1><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
        else decode_batch_warps<0><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
    } else {
        const u64 cap = (u64)info.sms * info.dec_batch_per_sm;
        const unsigned grid = (unsigned)(batch_tiles < cap ? (batch_tiles ? batch_tiles : 1) : cap);
        decode_batch<<<grid, kDecodeThreads, sizeof(DecodeBatchSmem), st>>>(batch);
    }
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

ADACOMP_STATUS_HOOKS(decode_batch)

}  // namespace adacomp_impl
