// Batched pack(): the kernels of adacomp_compress_multi and their launcher (see pack_batch.cuh).
#include "internal.h"

namespace adacomp_impl {

// Largest i with layer[i].tile_first <= gt (layers without tiles are skipped by construction).
template <int N>
__device__ inline int batch_layer_of(const BatchArgsT<N> &b, u32 gt)
{
    int lo = 0, hi = (int)b.n_layers;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (b.layer[mid].tile_first <= gt) lo = mid; else hi = mid;
    }
    return lo;
}

template <int N>
__global__ void __launch_bounds__(128)
batch_clear(const __grid_constant__ BatchArgsT<N> b)
{
    const BatchLayer &L = b.layer[blockIdx.x];
    u64 *z = reinterpret_cast<u64 *>(L.packed + L.geo.scratch_at);
    const u64 words = kCtlBytes / 8 + L.geo.n_groups;
    for (u64 i = threadIdx.x; i < words; i += blockDim.x) z[i] = 0;
}

template <int N>
__global__ void __launch_bounds__(kGenericThreads)
batch_tile_pass(const __grid_constant__ BatchArgsT<N> b)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 s_tmp[33];
    __shared__ u64 s_acc[kWindows + 1];
    const int tid = threadIdx.x;
    if (tid < kWindows + 1) s_acc[tid] = 0;
    __syncthreads();
    int cur = -1;
    auto flush = [&]() {        // this CTA's share of the current layer's exact sum
        if (cur >= 0 && tid < kWindows) {
            const u64 v = s_acc[tid];
            if (v) atomicAdd(reinterpret_cast<u64 *>(b.layer[cur].packed + b.layer[cur].geo.scratch_at) + tid, v);
            s_acc[tid] = 0;
        }
    };
    for (u32 gt = blockIdx.x; gt < b.total_tiles; gt += gridDim.x) {
        const int li = batch_layer_of(b, gt);
        if (li != cur) {
            flush();
            cur = li;
        }
        const BatchLayer &L = b.layer[li];
        const TileIo io{L.grad, L.residue, L.packed, L.packed + L.geo.scratch_at, 0u, L.factor, L.grad_type, 0u, nullptr};
        if (L.geo.w == 1u) generic_tile<unsigned char>(io, L.geo, gt - L.tile_first, smem_raw, s_tmp, s_acc);
        else generic_tile<unsigned short>(io, L.geo, gt - L.tile_first, smem_raw, s_tmp, s_acc);
    }
    flush();
}

// The pipelined tile pass (any-bin form: fp32 gradient, eager, no flags) over the tiles of a whole batch of
// layers: global tile gt belongs to the layer whose tile_first is the largest not above it.  The CTA's
// tiles go up, so each thread (and, for the loads two tiles ahead, the service lane) keeps a cursor
// into the layer table; what depends on the layer's bin length (the place of a thread's 25 elements among
// the bins) is recomputed when the cursor moves, and the CTA's share of a layer's exact g_max sum is added
// to that layer's windows when the CTA leaves the layer.  Every layer here has 41 <= L_T <= 1000.
// LAZY: lazy-scale mode, every layer with its own state (see tile_pass_fast); a layer whose state is not its
// own is flagged, left untouched and reports empty tiles.
// OPTS: some layer has a 16-bit gradient or a factor (else both are compile-time constants: plain lists keep
// the shorter code).
// USPB: not 0 when every layer of the batch has the bin length 25 * USPB (tiles of exactly 4000 elements, a bin
// USPB whole segments): the tile's shape, a thread's place among the bins and the word width are then
// compile-time constants, as in the single-layer kernel, and the tile code is two thirds as long.
template <int N, bool LAZY, bool OPTS, int USPB = 0>
__global__ void __launch_bounds__(kFastThreads, 2)
batch_tile_pass_fast(const __grid_constant__ BatchArgsT<N> b)
{
    constexpr bool UNI = USPB != 0;
    constexpr int USPB1 = UNI ? USPB : 1;           // (a divisor that is never 0)
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *s_words = smem + FastSmem::kWordsAt;
    u32 *s_incl = reinterpret_cast<u32 *>(smem + FastSmem::kInclAt);
    u32 *s_wtot = reinterpret_cast<u32 *>(smem + FastSmem::kWtotAt);
    float *s_segmax = reinterpret_cast<float *>(smem + FastSmem::kSegmaxAt);   // (layers whose bins are whole segments) the segments' maxima
    u32 *s_anymax = reinterpret_cast<u32 *>(smem + FastSmem::kBinmaxAt);    // [2][kSmallBins] bits of the bin maxima, by tile parity
    u32 *s_anycnt = s_anymax + 2 * kSmallBins;                               // [2][kSmallBins] words per bin
    u64 *s_acc = reinterpret_cast<u64 *>(smem + FastSmem::kAccAt);
    u64 *s_full = reinterpret_cast<u64 *>(smem + FastSmem::kBarAt);
    volatile u32 *s_abort = reinterpret_cast<volatile u32 *>(smem + FastSmem::kAbortAt);
    // the layers' first tiles, copied out of the kernel parameters: a CTA's next tile is often several layers on, and a
    // walk through the parameter table is a chain of dependent constant-cache misses that every warp waits for
    u32 *s_tile_first = reinterpret_cast<u32 *>(smem + FastSmem::kBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const u32 first = blockIdx.x, stride = gridDim.x;
    const u32 my_tiles = b.total_tiles > first ? (b.total_tiles - first + stride - 1) / stride : 0;
    const int n_layers = (int)b.n_layers;
    for (int l = tid; l < n_layers; l += kFastThreads) s_tile_first[l] = b.layer[l].tile_first;
    auto seek = [&](u32 gt, int &li) {      // (tiles only go up)
        while (li + 1 < n_layers && s_tile_first[li + 1] <= gt) li++;
    };
    auto state_ok = [&](const BatchLayer &L) {      // (LAZY) the state is this layer's
        const LazyHeader *lh = reinterpret_cast<const LazyHeader *>(L.lazy);
        return lh->magic == kLazyMagic && lh->n == L.geo.n && lh->L_T == L.geo.L_T;
    };

    if (tid < kWindows + 1) s_acc[tid] = 0;
    for (int i = tid; i < 4 * kSmallBins; i += kFastThreads) s_anymax[i] = 0;
    if (tid == 0) {
        *s_abort = 0;
        for (int st = 0; st < kStages; st++) mbar_init(&s_full[st], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    u32 issued = 0;                     // service lane 0: loads issued for tiles [0, issued)
    int load_li = 0, load_checked = -1;
    bool load_ok = true;
    auto issue_load = [&](u32 i) {
        if (i >= my_tiles) return;
        const u32 gt = first + i * stride;
        seek(gt, load_li);
        const BatchLayer &L = b.layer[load_li];
        if (LAZY && load_li != load_checked) {
            load_checked = load_li;
            load_ok = state_ok(L);
        }
        if (LAZY && !load_ok) return;                   // nothing of such a layer is read
        const u32 lt = gt - L.tile_first, T = L.geo.tile_elems;
        // a ragged last tile is read with plain loads (no division: the layer's tiles cover n exactly or all but the last are whole)
        if ((u64)lt + 1 >= L.geo.n_tiles && L.geo.n != L.geo.n_tiles * (u64)T) return;
        const bool g16 = OPTS && L.grad_type != ADACOMP_GRAD_F32;
        if (g16 && T % 8u != 0) return;                 // 16-bit tiles off the 16-byte boundaries: plain loads as well
        const u32 gbytes = g16 ? 2u * T : 4u * T;
        unsigned char *st = smem + (i % kStages) * kStageBytes;
        u64 *bar = &s_full[i % kStages];
        mbar_arrive_expect_tx(bar, gbytes + 4u * T + (LAZY ? kMaskBytes : 0u));
        bulk_load(st, reinterpret_cast<const unsigned char *>(L.grad) + (u64)lt * gbytes, gbytes, bar);
        bulk_load(st + kTileBytes, L.residue + (u64)lt * T, 4u * T, bar);
        if (LAZY) bulk_load(st + 2 * kTileBytes, L.lazy + kLazyHeaderBytes + (u64)lt * kMaskBytes, kMaskBytes, bar);
        issued = i + 1;
    };
    if (service && lane == 0) {
        issue_load(0);
        issue_load(1);
    }

    int li = 0, at_li = -1;             // the tile's layer; the layer the values below belong to
    u32 phase = 0;                      // bit s: parity of stage s's next completion (ragged tiles use no barrier)
    int T = 0, TB = 0, b0 = 0, cut = kSeg, off0 = 0, vcount = 0;
    u32 full_tiles = 0, wbytes = 1;
    u32 gtype = 0;                      // the layer's gradient format
    float factor = 0.f;                 // the layer's factor of the selection test (0: two additions)
    int SPB = 0;                        // (aligned) segments per bin
    bool aligned = false;               // every segment of the layer's tiles lies in one bin and exists whole
    bool layer_ok = true;               // (LAZY) the layer's state is its own
    u32 prev_scale_bits = 0;            // (LAZY) last step's scale of the layer
    u32 *lazy_mask = nullptr;
    auto flush = [&]() {                // (service warp) this CTA's share of layer at_li's exact sum
        if (at_li >= 0 && lane < kWindows) {
            const u64 v = s_acc[lane];
            if (v) atomicAdd(reinterpret_cast<u64 *>(b.layer[at_li].packed + b.layer[at_li].geo.scratch_at) + lane, v);
            s_acc[lane] = 0;
        }
        __syncwarp();
    };
    u32 i = 0;
    for (; i < my_tiles; i++) {
        const u32 gt = first + i * stride;
        seek(gt, li);
        const BatchLayer &L = b.layer[li];
        const Geometry &geo = L.geo;
        if (li != at_li) {
            if (service) flush();
            at_li = li;
            T = (int)geo.tile_elems;
            TB = (int)geo.tile_bins;
            full_tiles = (u32)geo.n_tiles - (geo.n != geo.n_tiles * (u64)T ? 1u : 0u);      // (no division)
            wbytes = geo.w;
            // the thread's elements [0, cut) lie in bin b0 of the tile, from place off0 of it on, the others
            // in bin b0 + 1; only the first `vcount` of them exist (tiles of less than 4000 elements)
            const int Lt = (int)geo.L_T, e0 = tid * kSeg;
            b0 = (int)__umulhi((u32)e0, L.inv_L_T);         // e0 / L_T (the host's ceil(2^32 / L_T): exact for e0 < 4000, L_T <= 1000)
            off0 = e0 - b0 * Lt;
            cut = min(kSeg, Lt - off0);
            vcount = max(0, min(kSeg, T - e0));
#ifdef ADACOMP_BATCH_NO_ALIGNED_FORM
            aligned = false;
#else
            aligned = T == kFastTile && Lt % kSeg == 0;     // (then cut = vcount = 25 in every thread)
#endif
            SPB = Lt / kSeg;
            gtype = OPTS ? L.grad_type : (u32)ADACOMP_GRAD_F32;
            factor = OPTS ? L.factor : 0.f;
            // (16-bit gradient tiles that do not start on 16-byte boundaries: every tile by plain loads)
            if (gtype != ADACOMP_GRAD_F32 && T % 8 != 0) full_tiles = 0;
            if (LAZY) {
                layer_ok = state_ok(L);
                if (layer_ok) {
                    prev_scale_bits = __float_as_uint(reinterpret_cast<const LazyHeader *>(L.lazy)->scale) & 0x7fffffffu;
                    lazy_mask = reinterpret_cast<u32 *>(L.lazy + kLazyHeaderBytes);
                } else if (tid == 0) {
                    raise_status(ADACOMP_DEV_HEADER_MISMATCH);
                }
            }
        }
        // (UNI: what the layer-change block worked out is known at compile time)
        const int kT = UNI ? kFastTile : T, kTB = UNI ? kTileSegs / USPB1 : TB, kSPB = UNI ? USPB : SPB;
        const bool kAl = UNI || aligned;
        const u32 kWb = UNI ? (USPB == 2 ? 1u : 2u) : wbytes;
        const int kB0 = UNI ? tid / USPB1 : b0, kCut = UNI ? kSeg : cut, kOff0 = UNI ? (tid % USPB1) * kSeg : off0;
        unsigned char *scratch = L.packed + geo.scratch_at;
        const u32 lt = gt - L.tile_first;
        if (LAZY && !layer_ok) {
            // the same hand-over as for a real tile, nothing read or computed: the tile counts as empty
            __syncthreads();
            if (tid < kSmallBins) {
                s_anymax[((i & 1) ^ 1) * kSmallBins + tid] = 0;
                s_anycnt[((i & 1) ^ 1) * kSmallBins + tid] = 0;
            }
            if (service && lane == 0) {
                reinterpret_cast<u32 *>(scratch + geo.tile_cnt_at)[lt] = 0;
                bulk_wait_read_all();
                issue_load(i + 2);
            }
            __syncthreads();
            continue;
        }
        const u64 base = (u64)lt * (u64)kT;
        float *s_d = reinterpret_cast<float *>(smem + (i % kStages) * kStageBytes);
        float *s_r = s_d + kFastTile;
        const bool whole = lt < full_tiles;
        const int elems = whole ? kT : (int)min((u64)kT, geo.n - base);      // (plain loads: the ragged last tile, or 16-bit tiles off the 16-byte boundaries)
        u32 *const any_max = s_anymax + (i & 1) * kSmallBins, *const any_cnt = s_anycnt + (i & 1) * kSmallBins;

        if (whole) {
            const u32 stage = i % kStages;
            if (!mbar_wait(&s_full[stage], (phase >> stage) & 1u)) {
                *s_abort = 1;                      // every thread that times out says so
                raise_status(ADACOMP_DEV_TIMEOUT);
            }
            phase ^= 1u << stage;
        } else {
            // the ragged last tile of a layer: plain loads, zero fill past the end (all of a thread's loads are
            // started before the first value is used: one trip to memory, not twenty-one)
            constexpr int kPer = (kFastTile + kFastThreads - 1) / kFastThreads;
            float dv[kPer], rv[kPer];
            const bool g16 = OPTS && gtype != ADACOMP_GRAD_F32;
#pragma unroll
            for (int q = 0; q < kPer; q++) {
                const int e = tid + q * kFastThreads;
                dv[q] = rv[q] = 0.f;
                if (e < elems) {
                    if (g16) dv[q] = __uint_as_float((u32) reinterpret_cast<const unsigned short *>(L.grad)[base + e]);    // (the 16 bits, as they are)
                    else dv[q] = L.grad[base + e];
                    rv[q] = L.residue[base + e];
                }
            }
#pragma unroll
            for (int q = 0; q < kPer; q++) {
                const int e = tid + q * kFastThreads;
                if (e < kFastTile) {
                    if (g16) reinterpret_cast<unsigned short *>(s_d)[e] = (unsigned short)__float_as_uint(dv[q]);
                    else s_d[e] = dv[q];
                    s_r[e] = rv[q];
                }
            }
            if (LAZY && tid < kTileSegs) reinterpret_cast<u32 *>(s_r + kFastTile)[tid] = lazy_mask[(u64)lt * kTileSegs + tid];
            __syncthreads();
        }

        // ---- G = residue + dW, H = G + dW; the maxima of |G| over the segment's part of each bin ----
        float g[kSeg], key[kSeg];
        float gm = 0.f, gm1 = 0.f;
        u32 selmask = 0, cnt = 0, incl = 0;
        if (!service) {
            const float *pd = s_d + tid * kSeg;
            const float *pr = s_r + tid * kSeg;
            float m = 0.f, m1 = 0.f;
            const u32 prev = LAZY ? reinterpret_cast<const u32 *>(s_r + kFastTile)[tid] : 0u;
            // (the loop twice: where the segments line up with the bins, as in the lists' bin lengths 50 and
            // 500, the tests on `vcount` and `kCut` fold away)
            auto form = [&](auto lined_up, auto sixteen) {
                constexpr bool AL = decltype(lined_up)::value, G16 = decltype(sixteen)::value;
                const int vc = AL ? kSeg : vcount, ct = AL ? kSeg : kCut;
                // 16-bit values: thirteen kAl 32-bit loads cover the segment's 50 bytes, a funnel shift lines the pairs up
                u32 pair[G16 ? 13 : 1];
                if (G16) {
                    const u32 *pw = reinterpret_cast<const u32 *>(s_d) + ((tid * kSeg) >> 1);
                    const u32 sh = (tid & 1) * 16u;
                    u32 w[14];
#pragma unroll
                    for (int q = 0; q < 13; q++) w[q] = pw[q];
                    w[13] = 0;
#pragma unroll
                    for (int q = 0; q < 13; q++) pair[q] = __funnelshift_r(w[q], w[q + 1], sh);
                }
#pragma unroll
                for (int j = 0; j < kSeg; j++) {
                    float d, r = pr[j];
                    if (G16) {
                        const u32 v16 = (j & 1) ? pair[j >> 1] >> 16 : pair[j >> 1] & 0xffffu;
                        d = gtype == ADACOMP_GRAD_BF16 ? __uint_as_float(v16 << 16) : __half2float(__ushort_as_half((unsigned short)v16));
                    } else {
                        d = pd[j];
                    }
                    if (j >= vc) d = r = 0.f;               // past the tile's end
                    if (LAZY) {
                        // r holds last step's G: finish "residue = G - sign(G) * scale" where it was sent
                        const float q = __uint_as_float(prev_scale_bits | (__float_as_uint(r) & 0x80000000u));
                        const float fixed = __fsub_rn(r, q);
                        r = (prev >> j & 1u) ? fixed : r;
                    }
                    g[j] = __fadd_rn(r, d);
                    const float h = OPTS && factor != 0.f ? __fadd_rn(r, __fmul_rn(factor, d)) : __fadd_rn(g[j], d);
                    if (j >= ct) m1 = fmaxf(m1, fabsf(g[j]));
                    else m = fmaxf(m, fabsf(g[j]));
                    key[j] = fmaxf(fabsf(h), fabsf(g[j]));
                }
            };
            if (!OPTS || gtype == ADACOMP_GRAD_F32) {
                if (kAl) form(TrueType{}, FalseType{});
                else form(FalseType{}, FalseType{});
            } else {
                if (kAl) form(TrueType{}, TrueType{});
                else form(FalseType{}, TrueType{});
            }
            if (kAl) {
                // a bin is kSPB whole segments: no atomics, the maximum goes through a shuffle (two segments)
                // or through the segments' maxima in shared memory
                if (kSPB == 2) gm = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                else s_segmax[tid] = m;
            } else {
                // (non-negative floats order like their bits)
                if (m > 0.f && kB0 < kTB) atomicMax(&any_max[kB0], __float_as_uint(m));
                if (m1 > 0.f && kB0 + 1 < kTB) atomicMax(&any_max[kB0 + 1], __float_as_uint(m1));
            }
        }
        if (!(kAl && kSPB == 2)) __syncthreads();                // barrier A (uniform: the layer's shape)
        if (!service) {
            if (!kAl) {
                gm = kB0 < kTB ? __uint_as_float(any_max[kB0]) : 0.f;
                gm1 = kB0 + 1 < kTB ? __uint_as_float(any_max[kB0 + 1]) : 0.f;
            } else if (kSPB != 2) {
                const int s0 = kB0 * kSPB;
                for (int sgm = 0; sgm < kSPB; sgm++) gm = fmaxf(gm, s_segmax[s0 + sgm]);
            }
            // ---- selection (a zero bin has G == 0 everywhere and sends nothing) ----
            if (kAl) {
#pragma unroll
                for (int j = 0; j < kSeg; j++)
                    if (key[j] >= gm && g[j] != 0.f) selmask |= 1u << j;
            } else {
#pragma unroll
                for (int j = 0; j < kSeg; j++)
                    if (key[j] >= (j >= kCut ? gm1 : gm) && g[j] != 0.f) selmask |= 1u << j;
            }
            cnt = __popc(selmask);
            if (!kAl) {
                const u32 c0 = __popc(selmask & ((1u << kCut) - 1u));
                if (c0) atomicAdd(&any_cnt[kB0], c0);
                if (cnt - c0) atomicAdd(&any_cnt[kB0 + 1], cnt - c0);
            } else if (tid == kB0 * kSPB) {
                any_max[kB0] = __float_as_uint(gm);                  // for the exact sum (the service warp reads it after barrier B)
            }
            incl = warp_inclusive_scan(cnt, lane);
            s_incl[tid] = incl;
            if (lane == 31) s_wtot[warp] = incl;
        }
        __syncthreads();                                            // barrier B
        // the other parity's buffers are free: tile i - 1 is done with them, tile i + 1 starts after barrier D
        if (tid < kSmallBins) {
            s_anymax[((i & 1) ^ 1) * kSmallBins + tid] = 0;
            s_anycnt[((i & 1) ^ 1) * kSmallBins + tid] = 0;
        }

        u32 total = 0;
        if (!service) {
            // ---- words into the staging area, G back into the residue stage ----
            u32 wpre_all[6];
            wpre_all[0] = 0;
#pragma unroll
            for (int wv = 0; wv < 5; wv++) wpre_all[wv + 1] = wpre_all[wv] + s_wtot[wv];
            const u32 wpre = wpre_all[warp];
            float *pr = s_r + tid * kSeg;
#pragma unroll
            for (int j = 0; j < kSeg; j++) pr[j] = g[j];
            u32 at = wpre + incl - cnt;
            u32 mask = selmask;
            while (mask) {
                const int j = __ffs(mask) - 1;
                mask &= mask - 1;
                const u32 neg = __float_as_uint(pr[j]) >> 31;
                const u32 idx = j >= kCut ? (u32)(j - kCut) : (u32)(kOff0 + j);        // the element's place in its bin
                const u32 word = (idx << 2) | 1u | (neg << 1);
                if (kWb == 1u) s_words[at] = (unsigned char)word;
                else reinterpret_cast<unsigned short *>(s_words)[at] = (unsigned short)word;
                at++;
            }
            if (LAZY) lazy_mask[(u64)lt * kTileSegs + tid] = selmask;
            if (kAl) {
                // the bin's first thread: the words between its own first one and the last one of the bin's last segment
                if (tid == kB0 * kSPB) {
                    const u64 bin = (u64)lt * (u64)kTB + (u32)kB0;
                    const int t1 = tid + kSPB - 1;
                    const u32 last = wpre_all[t1 >> 5] + s_incl[t1], count = last - (wpre + incl) + cnt;
                    if (bin < geo.n_bins) {
                        unsigned char *bc = L.packed + geo.bin_cnt_at;
                        if (kWb == 1u) bc[bin] = (unsigned char)count;
                        else reinterpret_cast<unsigned short *>(bc)[bin] = (unsigned short)count;
                    }
                }
            } else if (tid < kTB) {
                const u64 bin = (u64)lt * (u64)kTB + tid;
                if (bin < geo.n_bins) {
                    unsigned char *bc = L.packed + geo.bin_cnt_at;
                    if (kWb == 1u) bc[bin] = (unsigned char)any_cnt[tid];
                    else reinterpret_cast<unsigned short *>(bc)[bin] = (unsigned short)any_cnt[tid];
                }
            }
            fence_async_smem();          // the bulk store below reads what was just written
        } else {
            total = s_wtot[0] + s_wtot[1] + s_wtot[2] + s_wtot[3] + s_wtot[4];
            for (int bb = 0; bb < kTB; bb += 32) {       // every lane takes part each round
                const int bq = bb + lane;
                const bool valid = bq < kTB && (u64)lt * (u64)kTB + bq < geo.n_bins;
                warp_accumulate(s_acc, valid ? __uint_as_float(any_max[bq]) : 0.f, valid);
            }
            if (lane == 0) {
                bulk_wait_read_all();    // the store of tile i - 1 has drained its stage
                issue_load(i + 2);
            }
        }
        __syncthreads();                                            // barrier D

        const bool aborted = *s_abort != 0;
        if (service && !aborted) {
            if (whole) {
                if (lane == 0) {
                    bulk_store(L.residue + base, s_r, 4u * (u32)kT);
                    bulk_commit();
                }
            } else {
                for (int e = lane; e < elems; e += 32) L.residue[base + e] = s_r[e];
            }
            uint4 *slot = reinterpret_cast<uint4 *>(scratch + geo.slots_at + (u64)lt * geo.slot_bytes);
            const int chunks = (int)((total * kWb + 15) / 16);
            for (int c = lane; c < chunks; c += 32) slot[c] = reinterpret_cast<uint4 *>(s_words)[c];
            if (lane == 0) {
                reinterpret_cast<u32 *>(scratch + geo.tile_cnt_at)[lt] = total;
                if (total) atomicAdd(&reinterpret_cast<u64 *>(scratch + geo.group_at)[lt / kGroupTiles], (u64)total);
            }
        }
        if (aborted) break;          // uniform: the flag was set before barrier D
    }

    if (service) {
        if (lane == 0) {
            bulk_wait_all();
            if (*s_abort) {
                // after a timeout: loads still in flight must land (or time out in turn) before this CTA's
                // shared memory is given back, and the tiles it never finished count as empty so that the
                // kernels after this one stay inside their buffers
                int zl = 0;
                for (u32 j = i; j < my_tiles; j++) {
                    const u32 gt = first + j * stride;
                    seek(gt, zl);
                    const BatchLayer &Z = b.layer[zl];
                    const u32 zt = gt - Z.tile_first;
                    if (j > i && j < issued && (u64)zt < Z.geo.n / Z.geo.tile_elems)       // (a load was started for it)
                        mbar_wait(&s_full[j % kStages], (phase >> (j % kStages)) & 1u);
                    reinterpret_cast<u32 *>(Z.packed + Z.geo.scratch_at + Z.geo.tile_cnt_at)[zt] = 0;
                }
            }
        }
        __syncwarp();
        flush();
    }
}

template <int N>
__global__ void __launch_bounds__(1024)
batch_finalize(const __grid_constant__ BatchArgsT<N> b)
{
    const BatchLayer &L = b.layer[blockIdx.x];
    finalize_body(L.packed, L.packed + L.geo.scratch_at, L.geo, L.factor != 0.f ? kFlagFactor : 0u, L.count_out, L.lazy);
}

// FIXUP: also finishes the sent elements' residues (eager mode; lazy-scale mode leaves G).
template <int N, bool FIXUP>
__global__ void __launch_bounds__(kGatherThreads)
batch_gather(const __grid_constant__ BatchArgsT<N> b)
{
    __shared__ u32 s_pre_all[kGatherThreads / 32][kSmallBins + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 warps = gridDim.x * (kGatherThreads / 32);
    // Last tile first: the tile pass wrote the residues front to back, so the tail is what the L2 still holds.
    for (u32 item = blockIdx.x * (kGatherThreads / 32) + warp; item < b.total_tiles; item += warps) {
        const u32 gt = b.total_tiles - 1u - item;
        const BatchLayer &L = b.layer[batch_layer_of(b, gt)];
        const unsigned char *scratch = L.packed + L.geo.scratch_at;
        if (L.geo.w == 1u)
            gather_tile_small<unsigned char, FIXUP>(L.residue, L.packed, scratch, L.geo, gt - L.tile_first, lane, s_pre_all[warp]);
        else
            gather_tile_small<unsigned short, FIXUP>(L.residue, L.packed, scratch, L.geo, gt - L.tile_first, lane, s_pre_all[warp]);
    }
}


void init_pack_batch_info(DeviceInfo &d)
{
    const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
    const int bytes = (int)FastSmem::kBytes + 4 * kBatchMax;
    if (cudaFuncSetAttribute(batch_tile_pass<kBatchMax>, at, (int)kBatchSmemBytes) == cudaSuccess &&
        cudaFuncSetAttribute(batch_tile_pass<kBatchSmall>, at, (int)kBatchSmemBytes) == cudaSuccess) {
        int per = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, batch_tile_pass<kBatchMax>, kGenericThreads, kBatchSmemBytes);
        d.batch_per_sm = per;
    }
    d.batch_fast_ready = d.fast_ready &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, false, false>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, false, false>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, true, false>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, true, false>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, false, true>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, false, true>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, true, true>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, true, true>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, false, false, 2>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, false, false, 2>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, true, false, 2>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, true, false, 2>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, false, false, 20>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, false, false, 20>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, true, false, 20>, at, bytes) == cudaSuccess &&
                         cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, true, false, 20>, at, bytes) == cudaSuccess;
}

// lazy: lazy-scale mode (every layer carries its state; needs the pipelined batch tile pass).
template <int N>
int launch_batch_sized(const BatchArgsT<N> &b, const DeviceInfo &info, cudaStream_t st, bool lazy)
{
    batch_clear<N><<<b.n_layers, 128, 0, st>>>(b);
    if (b.total_tiles) {
        if (info.batch_fast_ready) {
            const u64 cap = (u64)info.sms * 2;
            const unsigned grid = (unsigned)(b.total_tiles < cap ? b.total_tiles : cap);
            bool opts = false;
            for (u32 i = 0; i < b.n_layers; i++) opts = opts || b.layer[i].grad_type != ADACOMP_GRAD_F32 || b.layer[i].factor != 0.f;
            // (one bin length, 50 or 500, throughout the batch: the form with the tile's shape compiled in)
            u32 lt_all = b.layer[0].geo.L_T;
            for (u32 i = 1; i < b.n_layers; i++) lt_all = b.layer[i].geo.L_T == lt_all ? lt_all : 0u;
            if (lazy && opts) batch_tile_pass_fast<N, true, true><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (opts) batch_tile_pass_fast<N, false, true><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (lazy && lt_all == 50u) batch_tile_pass_fast<N, true, false, 2><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (lazy && lt_all == 500u) batch_tile_pass_fast<N, true, false, 20><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (lazy) batch_tile_pass_fast<N, true, false><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (lt_all == 50u) batch_tile_pass_fast<N, false, false, 2><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else if (lt_all == 500u) batch_tile_pass_fast<N, false, false, 20><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
            else batch_tile_pass_fast<N, false, false><<<grid, kFastThreads, FastSmem::kBytes + 4 * N, st>>>(b);
        } else {
            const u64 cap = (u64)info.sms * info.batch_per_sm;
            const unsigned grid = (unsigned)(b.total_tiles < cap ? b.total_tiles : cap);
            batch_tile_pass<N><<<grid, kGenericThreads, kBatchSmemBytes, st>>>(b);
        }
    }
    batch_finalize<N><<<b.n_layers, 1024, 0, st>>>(b);
    if (b.total_tiles) {
        const u64 want = ((u64)b.total_tiles + 3) / 4, cap = (u64)info.sms * 16;
        const unsigned grid = (unsigned)(want < cap ? want : cap);
        if (lazy) batch_gather<N, false><<<grid, kGatherThreads, 0, st>>>(b);
        else batch_gather<N, true><<<grid, kGatherThreads, 0, st>>>(b);
    }
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

// Launches one batch (at most kBatchMax layers, all batchable) on the stream.
int launch_batch(const BatchArgs &b, const DeviceInfo &info, cudaStream_t st, bool lazy)
{
    if (b.n_layers == 0) return ADACOMP_OK;
    if (b.n_layers == 1) {      // a batch of one gains nothing over the single-layer kernels
        const BatchLayer &L = b.layer[0];
        return compress_impl(L.grad, L.residue, L.geo.n, L.geo.L_T, L.packed, reinterpret_cast<uint64_t *>(L.count_out),
                             st, 0, nullptr, L.lazy, L.factor, L.grad_type);
    }
    // a list that fits on the chip: the control blocks cleared, then one kernel (pack_onchip_list.cu)
    const bool onchip = !lazy && debug_waits().withhold_pack == 0 && onchip_list_takes(b, info);
    if (b.n_layers <= (u32)kBatchSmall) {
        BatchArgsT<kBatchSmall> small;
        small.n_layers = b.n_layers;
        small.total_tiles = b.total_tiles;
        for (u32 i = 0; i < b.n_layers; i++) small.layer[i] = b.layer[i];
        if (!onchip) return launch_batch_sized(small, info, st, lazy);
        batch_clear<kBatchSmall><<<small.n_layers, 128, 0, st>>>(small);
    } else {
        if (!onchip) return launch_batch_sized(b, info, st, lazy);
        batch_clear<kBatchMax><<<b.n_layers, 128, 0, st>>>(b);
    }
    return launch_pack_onchip_list(b, info, debug_waits().limit, st);
}


ADACOMP_STATUS_HOOKS(pack_batch)

}  // namespace adacomp_impl
