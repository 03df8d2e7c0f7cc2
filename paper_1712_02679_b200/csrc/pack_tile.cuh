// pack(): the tile code shared by the single-layer and the batched kernels (Algorithm 2 with the scale of Section 2.5).
#pragma once

#include "common.cuh"

namespace adacomp_impl {

// ---------------------------------------------------------------------------------
// tile_pass, fast path: L_T = 25 * SPB for SPB = 2, 4, 5, 8, 10, 20, 40 (L_T = 50 ... 1000), tiles of 4000 elements;
// and, as SPB = 0, every other L_T from 41 to 1000 (tiles of 3200 to 4000 elements, bins anywhere) and the
// multiples of 4 up to 4000 (a tile is one bin).
//
// Thread t < 160 owns the 25 consecutive elements of segment t (stride 25 words in
// shared memory: odd, so a warp's accesses are bank-conflict free); a bin is SPB
// adjacent segments.  SPB = 0: a bin is L_T consecutive elements wherever the segments' edges
// are; L_T > 25, so a segment lies in one bin or straddles one edge between two, and the
// threads meet in shared-memory atomics on per-bin maxima and counts.  Warp 5 (the service warp) owns no segment: its lane 0 issues
// every bulk copy, and the warp feeds the exact g_max accumulator and copies the
// tile's words to the scratch slot.
//
// Ring: tile i of this CTA lives in stage i % 3.  Loads for tile i + 2 are issued
// during tile i, after the bulk store that drained that stage (tile i - 1) has
// finished reading shared memory.
// ---------------------------------------------------------------------------------

struct PassArgs {
    const float *grad;
    float *residue;
    unsigned char *packed;      // the stream under construction
    unsigned char *scratch;     // control block, group counts, tile counts, word slots
    Geometry geo;
    u32 literal;
    unsigned char *lazy_state;  // lazy mode: header + per-segment masks of the elements sent last step
    float factor;               // 0: H = G + dW (Algorithm 2); else H = residue + factor * dW (Section 2.4's scale-factor)
    u32 grad_type;              // ADACOMP_GRAD_*: `grad` points to binary32 values, or to bfloat16 / binary16 ones (widened exactly on load)
    u32 quantiser;              // 0: scale = mean of the bin maxima (Section 2.5); 1: mean |G| of the sent elements
    long long wait_limit;       // cycles a wait for a stage may take (kWaitCycles unless a test shortened it)
    u32 withhold;               // testing aid: CTA 0 starts no copies for its tile number `withhold` (0: none)
};

// Lazy-mode state: 64-byte header, then one u32 per 25-element segment (bit j = element j
// of the segment was sent by the last step and its residue still holds G).
constexpr u32 kLazyMagic = 0x314c4441u;     // "ADL1"
constexpr u32 kLazyHeaderBytes = 64;
struct LazyHeader {
    u32 magic, L_T;
    u64 n;
    float scale;        // last step's scale
    u32 steps;          // lazy steps since the last flush
};

__host__ __device__ inline u64 lazy_state_bytes(const Geometry &g)
{
    return kLazyHeaderBytes + align_up(g.n_tiles * (u64)kMaskBytes, 16);
}

// Shared memory of the pipelined tile pass: NS stages of STAGE bytes, then the tile's words and the small tables.
template <int NS, u32 STAGE>
struct FastSmemT {
    static constexpr u32 kWordsAt = NS * STAGE;                       // (3 stages of 32640: 97920)
    static constexpr u32 kInclAt = kWordsAt + 2 * kFastTile;          // + 8000 (16-bit words)
    static constexpr u32 kWtotAt = kInclAt + 4 * kTileSegs;
    static constexpr u32 kSegmaxAt = kWtotAt + 4 * 8;
    static constexpr u32 kBinmaxAt = kSegmaxAt + 4 * kTileSegs;
    static constexpr u32 kAccAt = kBinmaxAt + 4 * 4 * kSmallBins;     // (SPB = 0: two buffers each of bin maxima and counts) 8-byte aligned
    static constexpr u32 kAcc2At = kAccAt + 8 * (kWindows + 1);       // (second quantiser) exact sum of the sent |G|
    static constexpr u32 kBarAt = kAcc2At + 8 * (kWindows + 1);
    static constexpr u32 kAbortAt = kBarAt + 8 * NS;
    static constexpr u32 kBytes = kAbortAt + 16;
};
typedef FastSmemT<kStages, kStageBytes> FastSmem;
static_assert(FastSmem::kAccAt % 8 == 0, "accumulator must be 8-byte aligned");
// The form with three CTAs per SM (16-bit gradients): two stages, the 8000-byte gradient tile packed against the residue.
constexpr u32 kStageBytes16 = kTileBytes / 2 + kTileBytes + kMaskBytes;     // 24640
typedef FastSmemT<2, kStageBytes16> FastSmem3;
static_assert(FastSmem3::kAccAt % 8 == 0 && kStageBytes16 % 16 == 0 && 3 * (FastSmem3::kBytes + 1024) <= 227 * 1024, "three CTAs per SM");

// GT: ADACOMP_GRAD_F32, or the gradient arrives in 16 bits per value (bfloat16 / binary16: tiles of half the
// bytes, widened exactly as they are read).
// CTAS: CTAs per SM the kernel is built for.  2: three stages of a whole gradient tile and a residue tile.  3 (16-bit
// gradients only): two stages with the half-size gradient tile packed against the residue; the next tile's load
// is then issued at the top of a tile instead of at its end, so that it has the whole tile to land.
template <int SPB, typename Word, bool LAZY, int GT = 0, int CTAS = 2>
__global__ void __launch_bounds__(kFastThreads, CTAS)
tile_pass_fast(PassArgs a)
{
    static_assert(CTAS == 2 || (CTAS == 3 && GT != 0), "three CTAs per SM: 16-bit gradients");
    constexpr int NS = CTAS == 3 ? 2 : kStages;
    constexpr u32 STAGE = CTAS == 3 ? kStageBytes16 : kStageBytes;
    constexpr u32 kResAt = CTAS == 3 ? kTileBytes / 2 : kTileBytes, kMaskAt = kResAt + kTileBytes;     // inside a stage
    typedef FastSmemT<NS, STAGE> FS;
    extern __shared__ __align__(128) unsigned char smem[];
    Word *s_words = reinterpret_cast<Word *>(smem + FS::kWordsAt);
    u32 *s_incl = reinterpret_cast<u32 *>(smem + FS::kInclAt);
    u32 *s_wtot = reinterpret_cast<u32 *>(smem + FS::kWtotAt);
    float *s_segmax = reinterpret_cast<float *>(smem + FS::kSegmaxAt);
    float *s_binmax = reinterpret_cast<float *>(smem + FS::kBinmaxAt);
    u64 *s_acc = reinterpret_cast<u64 *>(smem + FS::kAccAt);
    u64 *s_acc2 = reinterpret_cast<u64 *>(smem + FS::kAcc2At);
    u64 *s_full = reinterpret_cast<u64 *>(smem + FS::kBarAt);
    volatile u32 *s_abort = reinterpret_cast<volatile u32 *>(smem + FS::kAbortAt);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const Geometry &geo = a.geo;
    constexpr bool ANY = SPB == 0;
    constexpr bool G16 = GT != 0;       // 16-bit gradient values (ANY: the launcher sees to it that a tile of them is a multiple of 16 bytes)
    constexpr int kBins = ANY ? kSmallBins : kTileSegs / (ANY ? 1 : SPB);
    const int T = ANY ? (int)geo.tile_elems : kFastTile;            // elements of a tile (a multiple of 4)
    const int TB = ANY ? (int)geo.tile_bins : kBins;
    const u32 tile_bytes = (u32)T * 4u;
    // ANY: the thread's elements [0, cut) lie in bin b0 of the tile, from place off0 of it on, the
    // others in bin b0 + 1; only the first `vcount` of them exist (tiles of less than 4000 elements)
    int b0 = 0, cut = kSeg, off0 = 0, vcount = kSeg;
    if (ANY) {
        const int L = (int)geo.L_T, e0 = tid * kSeg;
        b0 = e0 / L;
        off0 = e0 - b0 * L;
        cut = min(kSeg, L - off0);
        vcount = max(0, min(kSeg, T - e0));
    }
    u32 *s_anymax = reinterpret_cast<u32 *>(s_binmax);              // ANY: [2][kSmallBins] bits of the bin maxima, by tile parity
    u32 *s_anycnt = s_anymax + 2 * kSmallBins;                      // ANY: [2][kSmallBins] words per bin
    Word *bin_cnt = reinterpret_cast<Word *>(a.packed + geo.bin_cnt_at);
    u32 *tile_cnt = reinterpret_cast<u32 *>(a.scratch + geo.tile_cnt_at);
    u64 *group_cnt = reinterpret_cast<u64 *>(a.scratch + geo.group_at);

    // tiles of this CTA: blockIdx.x + i * gridDim.x
    const u64 first = blockIdx.x, stride = gridDim.x;
    const u64 my_tiles = geo.n_tiles > first ? (geo.n_tiles - first + stride - 1) / stride : 0;
    const u64 full_tiles = geo.n / (u64)T;          // tiles below this index are complete

    // Lazy mode: the residue buffer holds last step's G; the elements sent then still owe
    // "- sign(G) * scale" (Algorithm 2's G - Gq), applied here as they are loaded.
    u32 prev_scale_bits = 0;
    u32 *lazy_mask = nullptr;
    if (LAZY) {
        const LazyHeader *lh = reinterpret_cast<const LazyHeader *>(a.lazy_state);
        if (lh->magic != kLazyMagic || lh->n != a.geo.n || lh->L_T != a.geo.L_T) {
            // not the state of this tensor (the same decision in every CTA): touch neither residue
            // nor state, and report every tile as empty so that the kernels after this one see a
            // consistent, empty stream
            if (threadIdx.x == 0) {
                if (blockIdx.x == 0) raise_status(ADACOMP_DEV_HEADER_MISMATCH);
                u32 *counts = reinterpret_cast<u32 *>(a.scratch + a.geo.tile_cnt_at);
                for (u64 t = blockIdx.x; t < a.geo.n_tiles; t += gridDim.x) counts[t] = 0;
            }
            return;
        }
        prev_scale_bits = __float_as_uint(lh->scale) & 0x7fffffffu;
        lazy_mask = reinterpret_cast<u32 *>(a.lazy_state + kLazyHeaderBytes);
    }

    if (tid < kWindows + 1) s_acc[tid] = s_acc2[tid] = 0;
    if (ANY)
        for (int b = tid; b < 4 * kSmallBins; b += kFastThreads) s_anymax[b] = 0;
    if (tid == 0) {
        *s_abort = 0;
        for (int s = 0; s < NS; s++) mbar_init(&s_full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    u64 issued = 0;                     // service lane 0: loads issued for tiles [0, issued)
    auto issue_load = [&](u64 i) {
        const u64 tile = first + i * stride;
        if (i >= my_tiles || tile >= full_tiles) return;
        unsigned char *st = smem + (i % NS) * STAGE;
        u64 *bar = &s_full[i % NS];
        const u32 grad_bytes = G16 ? tile_bytes / 2 : tile_bytes;
        mbar_arrive_expect_tx(bar, grad_bytes + tile_bytes + (LAZY ? kMaskBytes : 0u));
        if (a.withhold != 0u && blockIdx.x == 0 && i == (u64)a.withhold) {
            issued = i + 1;             // (testing aid) bytes are expected and never sent: the wait for this stage runs out
            return;
        }
        bulk_load(st, reinterpret_cast<const unsigned char *>(a.grad) + tile * (u64)grad_bytes, grad_bytes, bar);
        bulk_load(st + kResAt, a.residue + tile * (u64)T, tile_bytes, bar);
        if (LAZY) bulk_load(st + kMaskAt, lazy_mask + tile * (u64)kTileSegs, kMaskBytes, bar);
        issued = i + 1;
    };
    if (service && lane == 0) {
        issue_load(0);
        if (NS > 2) issue_load(1);
    }

    u64 i = 0;
    for (; i < my_tiles; i++) {
        const u64 tile = first + i * stride;
        const u64 base = tile * (u64)T;
        float *s_d = reinterpret_cast<float *>(smem + (i % NS) * STAGE);
        float *s_r = reinterpret_cast<float *>(smem + (i % NS) * STAGE + kResAt);
        const u32 *s_prev = reinterpret_cast<const u32 *>(s_r + kFastTile);
        const bool whole = tile < full_tiles;
        const int elems = whole ? T : (int)(geo.n - base);
        u32 *const any_max = s_anymax + (i & 1) * kSmallBins, *const any_cnt = s_anycnt + (i & 1) * kSmallBins;
        if (NS == 2 && service && lane == 0) {
            bulk_wait_read_all();        // the store of tile i - 1 has drained the other stage
            issue_load(i + 1);
        }

        if (whole) {
            if (!mbar_wait(&s_full[i % NS], (u32)(i / NS) & 1u, a.wait_limit)) {
                *s_abort = 1;                      // every thread that times out says so
                raise_status(ADACOMP_DEV_TIMEOUT);
            }
        } else {
            // the ragged last tile of the tensor: plain loads, zero fill past the end
            for (int e = tid; e < kFastTile; e += kFastThreads) {
                float d = 0.f, r = 0.f;
                unsigned short d16 = 0;
                if (e < elems) {
                    if (G16) d16 = reinterpret_cast<const unsigned short *>(a.grad)[base + e];
                    else d = a.grad[base + e];
                    r = a.residue[base + e];
                }
                if (G16) reinterpret_cast<unsigned short *>(s_d)[e] = d16;
                else s_d[e] = d;
                s_r[e] = r;
            }
            if (LAZY && tid < kTileSegs)
                const_cast<u32 *>(s_prev)[tid] = lazy_mask[tile * (u64)kTileSegs + tid];
            __syncthreads();
        }

        // ---- G = residue + dW, H = G + dW; the segment's maximum |G| ----
        float g[kSeg], key[kSeg];
        float gm = 0.f, gm1 = 0.f;      // the bin maximum (ANY: of the segment's first and second bin)
        u32 selmask = 0, cnt = 0, incl = 0;
        if (!service) {
            const float *pd = s_d + tid * kSeg;
            const float *pr = s_r + tid * kSeg;
            float m = 0.f, m1 = 0.f;
            const u32 prev = LAZY ? s_prev[tid] : 0u;
            // 16-bit values: the segment's 50 bytes start on a 4-byte boundary for even threads and two bytes
            // past one for odd threads; thirteen aligned 32-bit loads cover them either way, and a funnel
            // shift by 0 or 16 bits lines the pairs up (half as many shared-memory accesses as 25 16-bit loads)
            u32 pair[G16 ? 13 : 1];
            if (G16) {
                const u32 *pw = reinterpret_cast<const u32 *>(s_d) + ((tid * kSeg) >> 1);
                const u32 sh = (tid & 1) * 16u;
                u32 w[14];
#pragma unroll
                for (int q = 0; q < 13; q++) w[q] = pw[q];
                w[13] = 0;
#pragma unroll
                for (int q = 0; q < 13; q++) pair[q] = __funnelshift_r(w[q], w[q + 1], sh);    // elements 2q, 2q + 1
            }
#pragma unroll
            for (int j = 0; j < kSeg; j++) {
                float d;
                if (GT == ADACOMP_GRAD_BF16) d = __uint_as_float((j & 1) ? pair[j >> 1] & 0xffff0000u : pair[j >> 1] << 16);
                else if (GT == ADACOMP_GRAD_F16) d = __half2float(__ushort_as_half((unsigned short)((j & 1) ? pair[j >> 1] >> 16 : pair[j >> 1] & 0xffffu)));
                else d = pd[j];
                float r = pr[j];
                if (ANY && j >= vcount) d = r = 0.f;        // past the tile's end
                if (LAZY) {
                    // r holds last step's G: finish "residue = G - sign(G) * scale" where it was sent
                    const float q = __uint_as_float(prev_scale_bits | (__float_as_uint(r) & 0x80000000u));
                    const float fixed = __fsub_rn(r, q);
                    r = (prev >> j & 1u) ? fixed : r;
                }
                g[j] = __fadd_rn(r, d);
                const float h = a.factor != 0.f ? __fadd_rn(r, __fmul_rn(a.factor, d)) : __fadd_rn(g[j], d);
                if (ANY && j >= cut) m1 = fmaxf(m1, fabsf(g[j]));
                else m = fmaxf(m, fabsf(g[j]));
                // |G| never exceeds the bin maximum, so "|H| >= g_max or |G| == g_max"
                // is "max(|H|, |G|) >= g_max"
                key[j] = fmaxf(fabsf(h), fabsf(g[j]));
            }
            if (ANY) {
                // (non-negative floats order like their bits)
                if (m > 0.f && b0 < TB) atomicMax(&any_max[b0], __float_as_uint(m));
                if (m1 > 0.f && b0 + 1 < TB) atomicMax(&any_max[b0 + 1], __float_as_uint(m1));
            } else if (SPB == 2) {
                gm = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            } else {
                s_segmax[tid] = m;
            }
        }
        if (SPB != 2) {
            __syncthreads();                                        // barrier A
            if (ANY) {
                // the other parity's buffers are free: tile i - 1 is done with them, tile i + 1 starts after barrier D
                if (tid < kSmallBins) {
                    s_anymax[((i & 1) ^ 1) * kSmallBins + tid] = 0;
                    s_anycnt[((i & 1) ^ 1) * kSmallBins + tid] = 0;
                }
                if (!service) {
                    gm = b0 < TB ? __uint_as_float(any_max[b0]) : 0.f;
                    gm1 = b0 + 1 < TB ? __uint_as_float(any_max[b0 + 1]) : 0.f;
                }
            } else if (!service) {
                const int bin = tid / (ANY ? 1 : SPB);
#pragma unroll
                for (int s = 0; s < SPB; s++) gm = fmaxf(gm, s_segmax[bin * SPB + s]);
            }
        }
        if (!service) {
            if (!ANY && tid % (ANY ? 1 : SPB) == 0) s_binmax[tid / (ANY ? 1 : SPB)] = gm;
            // ---- selection (a zero bin has G == 0 everywhere and sends nothing) ----
#pragma unroll
            for (int j = 0; j < kSeg; j++)
                if (key[j] >= (ANY && j >= cut ? gm1 : gm) && g[j] != 0.f) selmask |= 1u << j;
            cnt = __popc(selmask);
            if (ANY) {
                const u32 c0 = __popc(selmask & ((1u << cut) - 1u));
                if (c0) atomicAdd(&any_cnt[b0], c0);
                if (cnt - c0) atomicAdd(&any_cnt[b0 + 1], cnt - c0);
            }
            incl = warp_inclusive_scan(cnt, lane);
            s_incl[tid] = incl;
            if (lane == 31) s_wtot[warp] = incl;
        }
        __syncthreads();                                            // barrier B

        u32 total = 0;
        if (!service) {
            // ---- words into the staging area, G back into the residue stage ----
            u32 wpre[6];
            wpre[0] = 0;
#pragma unroll
            for (int wv = 0; wv < 5; wv++) wpre[wv + 1] = wpre[wv] + s_wtot[wv];
            const u32 mine = wpre[warp] + incl;                     // inclusive position
            float *pr = s_r + tid * kSeg;
#pragma unroll
            for (int j = 0; j < kSeg; j++) pr[j] = g[j];
            u32 at = mine - cnt;
            const u32 seg_in_bin = ANY ? (u32)off0 : (u32)(tid % (ANY ? 1 : SPB)) * kSeg;
            u32 mask = selmask;
            while (mask) {
                const int j = __ffs(mask) - 1;
                mask &= mask - 1;
                const u32 neg = __float_as_uint(pr[j]) >> 31;
                const u32 idx = ANY && j >= cut ? (u32)(j - cut) : seg_in_bin + j;      // the element's place in its bin
                s_words[at++] = (Word)((idx << 2) | 1u | (neg << 1));
            }
            if (a.quantiser) {
                // the second quantiser: the exact sum of |G| over the sent elements, a sent element per lane and round
                const u32 rounds = __reduce_max_sync(0xffffffffu, cnt);
                u32 left = selmask;
                for (u32 r = 0; r < rounds; r++) {
                    const bool have = left != 0u;
                    const int j = have ? __ffs(left) - 1 : 0;
                    left &= left - 1u;
                    warp_accumulate_shared(s_acc2, fabsf(pr[j]), have);
                }
            }
            if (LAZY) lazy_mask[tile * (u64)kTileSegs + tid] = selmask;
            if (ANY) {
                if (tid < TB) {
                    const u64 bin = tile * (u64)TB + tid;
                    if (bin < geo.n_bins) bin_cnt[bin] = (Word)any_cnt[tid];
                }
            } else if (tid % (ANY ? 1 : SPB) == 0) {
                const u64 bin = tile * (u64)kBins + tid / (ANY ? 1 : SPB);
                const int t1 = tid + SPB - 1;
                const u32 last = wpre[t1 >> 5] + s_incl[t1];
                if (bin < geo.n_bins) bin_cnt[bin] = (Word)(last - mine + cnt);
            }
            fence_async_smem();          // the bulk store below reads what was just written
        } else {
            total = s_wtot[0] + s_wtot[1] + s_wtot[2] + s_wtot[3] + s_wtot[4];
            for (int bb = 0; bb < TB; bb += 32) {       // every lane takes part each round
                const int b = bb + lane;
                const bool valid = b < TB && tile * (u64)TB + b < geo.n_bins;
                warp_accumulate(s_acc, valid ? (ANY ? __uint_as_float(any_max[b]) : s_binmax[b]) : 0.f, valid);
            }
            if (NS > 2 && lane == 0) {
                bulk_wait_read_all();    // the store of tile i - 1 has drained its stage
                issue_load(i + 2);
            }
        }
        __syncthreads();                                            // barrier D

        const bool aborted = *s_abort != 0;
        if (service && !aborted) {
            if (whole) {
                if (lane == 0) {
                    bulk_store(a.residue + base, s_r, tile_bytes);
                    bulk_commit();
                }
            } else {
                for (int e = lane; e < elems; e += 32) a.residue[base + e] = s_r[e];
            }
            uint4 *slot = reinterpret_cast<uint4 *>(a.scratch + geo.slots_at + tile * geo.slot_bytes);
            const int chunks = (int)((total * sizeof(Word) + 15) / 16);
            for (int c = lane; c < chunks; c += 32) slot[c] = reinterpret_cast<uint4 *>(s_words)[c];
            if (lane == 0) {
                tile_cnt[tile] = total;
                if (total) atomicAdd(&group_cnt[tile / kGroupTiles], (u64)total);
            }
        }
        if (aborted) break;          // uniform: the flag was set before barrier D
    }

    if (service) {
        if (lane == 0) {
            bulk_wait_all();
            if (*s_abort) {
                // after a timeout: loads still in flight must land (or time out in turn) before
                // this CTA's shared memory is given back, and the tiles it never finished count
                // as empty so that the kernels after this one stay inside their buffers
                for (u64 j = i + 1; j < issued; j++) mbar_wait(&s_full[j % NS], (u32)(j / NS) & 1u, a.wait_limit);
                for (u64 j = i; j < my_tiles; j++) tile_cnt[first + j * stride] = 0;
            }
        }
        if (lane < kWindows) {
            const u64 v = s_acc[lane], v2 = s_acc2[lane];
            if (v) atomicAdd(reinterpret_cast<u64 *>(a.scratch) + lane, v);
            if (v2) atomicAdd(reinterpret_cast<u64 *>(a.scratch + kCtlSentSumAt) + lane, v2);
        }
    }
}

// ---------------------------------------------------------------------------------
// tile_pass, any L_T: a warp per bin, lanes strided over the bin's elements.
// Dynamic shared memory: H[tile_elems], G[tile_elems], words[tile_elems],
// gmax[units], cnt[units + 1], units = max(tile_bins, 8).
// ---------------------------------------------------------------------------------

// One tile of one layer.  Called by all 256 threads of the CTA; `s_acc` collects the CTA's share of
// the layer's exact g_max sum.
struct TileIo {                 // the buffers of one layer, as the generic tile code sees them
    const float *grad;
    float *residue;
    unsigned char *packed, *scratch;
    u32 literal;
    float factor;               // as in PassArgs
    u32 grad_type;
    u32 quantiser;              // as in PassArgs (then s_acc2 collects the exact sum of the sent |G|)
    u64 *s_acc2;
};

template <typename Word>
__device__ void generic_tile(const TileIo &a, const Geometry &geo, u64 tile, unsigned char *smem_raw, u32 *s_tmp,
                             u64 *s_acc)
{
    const int T = (int)geo.tile_elems, TB = (int)geo.tile_bins, L = (int)geo.L_T;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kGenericThreads / 32;
    // A unit is a warp's work: a bin or, in tiles of fewer bins than the CTA has warps, one of P equal
    // parts of a bin (whole 32-element steps each, so that the parts' words stay in ascending order).
    // (tiles have 1 bin or a multiple of 4: P is 8, 2 or 1)
    const int P = TB >= nwarp ? 1 : TB >= 4 ? 2 : 8, pshift = P == 8 ? 3 : P == 2 ? 1 : 0;
    const int part = P == 1 ? L : (((L + P - 1) / P + 31) & ~31);
    const int units = TB * P;
    float *s_d = reinterpret_cast<float *>(smem_raw);
    float *s_g = s_d + T;
    Word *s_words = reinterpret_cast<Word *>(s_g + T);
    float *s_gmax = reinterpret_cast<float *>(smem_raw + align_up((u64)T * (8 + sizeof(Word)), 16));    // [units]
    u32 *s_cnt = reinterpret_cast<u32 *>(s_gmax + units);                                                  // [units + 1]
    Word *bin_cnt = reinterpret_cast<Word *>(a.packed + geo.bin_cnt_at);
    u32 *tile_cnt = reinterpret_cast<u32 *>(a.scratch + geo.tile_cnt_at);
    u64 *group_cnt = reinterpret_cast<u64 *>(a.scratch + geo.group_at);

    const u64 base = tile * (u64)T;
    const u64 left = geo.n - base;
    const int elems = left < (u64)T ? (int)left : T;

    // G and H of the tile: four elements a thread and step where 4 divides the tile's length (every tile, and
    // the G array behind the H array in shared memory, then start on a 16-byte boundary)
    const int quads = (T & 3) == 0 && !a.grad_type ? elems >> 2 : 0;
    for (int i = tid; i < quads; i += kGenericThreads) {
        const float4 d = reinterpret_cast<const float4 *>(a.grad + base)[i];
        const float4 r = reinterpret_cast<const float4 *>(a.residue + base)[i];
        const float dv[4] = {d.x, d.y, d.z, d.w}, rv[4] = {r.x, r.y, r.z, r.w};
        float gv[4], hv[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            gv[q] = __fadd_rn(rv[q], dv[q]);
            hv[q] = a.factor != 0.f ? __fadd_rn(rv[q], __fmul_rn(a.factor, dv[q])) : __fadd_rn(gv[q], dv[q]);
        }
        reinterpret_cast<float4 *>(s_g)[i] = make_float4(gv[0], gv[1], gv[2], gv[3]);
        reinterpret_cast<float4 *>(s_d)[i] = make_float4(hv[0], hv[1], hv[2], hv[3]);
    }
    for (int i = 4 * quads + tid; i < T; i += kGenericThreads) {
        float d = 0.f, r = 0.f;
        if (i < elems) { d = load_grad(a.grad, base + i, a.grad_type); r = a.residue[base + i]; }
        const float g = __fadd_rn(r, d);
        s_g[i] = g;
        s_d[i] = a.factor != 0.f ? __fadd_rn(r, __fmul_rn(a.factor, d)) : __fadd_rn(g, d);      // H: dW is not needed again
    }
    __syncthreads();

    // words of unit u, whose bin's maximum is m; the bin's maximum joins the exact sum once
    auto count_unit = [&](int u, float m) {
        const int b = u >> pshift, j_lo = (u & (P - 1)) * part, j_hi = min(L, j_lo + part);
        u32 count = 0;
        if (m > 0.f) {
            for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
                const int j = j0 + lane;
                bool sel = false;
                if (j < j_hi) {
                    const float g = s_g[b * L + j];
                    const float h = s_d[b * L + j];
                    sel = (g != 0.f) && (fabsf(h) >= m || (!a.literal && fabsf(g) == m));
                }
                count += __popc(__ballot_sync(0xffffffffu, sel));
            }
        }
        if (lane == 0) {
            s_cnt[u] = count;
            if ((u & (P - 1)) == 0 && tile * (u64)TB + b < geo.n_bins) {
                u32 window;
                u64 lo, hi;
                if (split_for_sum(m, window, lo, hi)) {
                    atomicAdd(&s_acc[window], lo);
                    atomicAdd(&s_acc[window + 1], hi);
                }
            }
        }
    };
    // maxima of the units (a unit that is a whole bin goes on to count its words at once)
    for (int u = warp; u < units; u += nwarp) {
        const int b = u >> pshift, j_lo = (u & (P - 1)) * part, j_hi = min(L, j_lo + part);
        float m = 0.f;
        for (int j = j_lo + lane; j < j_hi; j += 32) m = fmaxf(m, fabsf(s_g[b * L + j]));
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        if (lane == 0) s_gmax[u] = m;
        if (P == 1) count_unit(u, m);
    }
    if (P > 1) {
        __syncthreads();
        for (int u = warp; u < units; u += nwarp) {
            float m = 0.f;
            for (int q = 0; q < P; q++) m = fmaxf(m, s_gmax[(u & ~(P - 1)) + q]);
            count_unit(u, m);
        }
    }
    __syncthreads();
    block_exclusive_scan(s_cnt, units, s_tmp);
    for (int b = tid; b < TB; b += kGenericThreads) {
        const u64 bin = tile * (u64)TB + b;
        if (bin < geo.n_bins) bin_cnt[bin] = (Word)(s_cnt[(b + 1) << pshift] - s_cnt[b << pshift]);
    }

    // words, in ascending order inside each bin
    for (int u = warp; u < units; u += nwarp) {
        const int b = u >> pshift, j_lo = (u & (P - 1)) * part, j_hi = min(L, j_lo + part);
        float m = 0.f;
        for (int q = 0; q < P; q++) m = fmaxf(m, s_gmax[(u & ~(P - 1)) + q]);
        if (!(m > 0.f)) continue;
        u32 at = s_cnt[u];
        for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
            const int j = j0 + lane;
            bool sel = false;
            float g = 0.f;
            if (j < j_hi) {
                g = s_g[b * L + j];
                const float h = s_d[b * L + j];
                sel = (g != 0.f) && (fabsf(h) >= m || (!a.literal && fabsf(g) == m));
            }
            const u32 mask = __ballot_sync(0xffffffffu, sel);
            if (sel) {
                const u32 pos = at + __popc(mask & ((1u << lane) - 1u));
                s_words[pos] = (Word)(((u32)j << 2) | (g < 0.f ? 3u : 1u));
            }
            if (a.quantiser && mask) warp_accumulate_shared(a.s_acc2, fabsf(g), sel);
            at += __popc(mask);
        }
    }
    __syncthreads();

    if (quads) {
        for (int i = tid; i < quads; i += kGenericThreads)
            reinterpret_cast<float4 *>(a.residue + base)[i] = reinterpret_cast<const float4 *>(s_g)[i];
        for (int i = 4 * quads + tid; i < elems; i += kGenericThreads) a.residue[base + i] = s_g[i];
    } else {
        for (int i = tid; i < elems; i += kGenericThreads) a.residue[base + i] = s_g[i];
    }
    const u32 total = s_cnt[units];
    Word *slot = reinterpret_cast<Word *>(a.scratch + geo.slots_at + tile * geo.slot_bytes);
    for (u32 i = tid; i < total; i += kGenericThreads) slot[i] = s_words[i];
    if (tid == 0) {
        tile_cnt[tile] = total;
        if (total) atomicAdd(&group_cnt[tile / kGroupTiles], (u64)total);
    }
    __syncthreads();
}

// A tile that is one bin (L_T > 1000), by the whole CTA.  Per element only a signed key stays in shared
// memory: max(|H|, |G|) (|H| alone under the literal flag) with G's sign, zero where G is zero; an element
// goes out when the key's magnitude reaches the bin's maximum, which is known once all of G has gone by.
// G itself is written to the residue as it is formed.  Dynamic shared memory: key[L_T], words[L_T].
template <typename Word>
__device__ void generic_tile_one_bin(const TileIo &a, const Geometry &geo, u64 tile, unsigned char *smem_raw, u32 *s_tmp,
                                     u64 *s_acc)
{
    const int L = (int)geo.L_T;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int nwarp = kGenericThreads / 32;
    float *s_key = reinterpret_cast<float *>(smem_raw);
    Word *s_words = reinterpret_cast<Word *>(s_key + L);
    const u64 base = tile * (u64)L;
    const u64 left = geo.n - base;
    const int elems = left < (u64)L ? (int)left : L;

    auto key_of = [&](float r, float d, float &g) {
        g = __fadd_rn(r, d);
        const float h = a.factor != 0.f ? __fadd_rn(r, __fmul_rn(a.factor, d)) : __fadd_rn(g, d);
        const float k = a.literal ? fabsf(h) : fmaxf(fabsf(h), fabsf(g));
        return g == 0.f ? 0.f : copysignf(k, g);
    };
    float m = 0.f;
    // (four elements a step where the bin starts on a 16-byte boundary)
    const int quads = (base & 3u) == 0 && !a.grad_type ? elems >> 2 : 0;
    for (int i = tid; i < quads; i += kGenericThreads) {
        const float4 d = reinterpret_cast<const float4 *>(a.grad + base)[i];
        const float4 r = reinterpret_cast<const float4 *>(a.residue + base)[i];
        float4 g, k;
        k.x = key_of(r.x, d.x, g.x);
        k.y = key_of(r.y, d.y, g.y);
        k.z = key_of(r.z, d.z, g.z);
        k.w = key_of(r.w, d.w, g.w);
        m = fmaxf(fmaxf(m, fmaxf(fabsf(g.x), fabsf(g.y))), fmaxf(fabsf(g.z), fabsf(g.w)));
        reinterpret_cast<float4 *>(a.residue + base)[i] = g;
        reinterpret_cast<float4 *>(s_key)[i] = k;
    }
    for (int i = 4 * quads + tid; i < L; i += kGenericThreads) {
        float k = 0.f;
        if (i < elems) {
            float g;
            k = key_of(a.residue[base + i], load_grad(a.grad, base + i, a.grad_type), g);
            m = fmaxf(m, fabsf(g));
            a.residue[base + i] = g;
        }
        s_key[i] = k;
    }
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) s_tmp[warp] = __float_as_uint(m);
    __syncthreads();
    m = 0.f;
    for (int q = 0; q < nwarp; q++) m = fmaxf(m, __uint_as_float(s_tmp[q]));
    __syncthreads();                                   // s_tmp is reused for the counts

    // a warp per eighth of the bin (whole 32-element steps, so that the words stay in ascending order)
    const int part = ((L + nwarp - 1) / nwarp + 31) & ~31;
    const int j_lo = warp * part, j_hi = min(L, j_lo + part);
    u32 count = 0;
    if (m > 0.f)
        for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
            const int j = j0 + lane;
            const float k = j < j_hi ? s_key[j] : 0.f;
            count += __popc(__ballot_sync(0xffffffffu, fabsf(k) >= m && k != 0.f));
        }
    if (lane == 0) s_tmp[warp] = count;
    __syncthreads();
    u32 at = 0, total = 0;
    for (int q = 0; q < nwarp; q++) {
        const u32 c = s_tmp[q];
        if (q < warp) at += c;
        total += c;
    }
    if (m > 0.f)
        for (int j0 = j_lo; j0 < j_hi; j0 += 32) {
            const int j = j0 + lane;
            const float k = j < j_hi ? s_key[j] : 0.f;
            const bool sel = fabsf(k) >= m && k != 0.f;
            const u32 mask = __ballot_sync(0xffffffffu, sel);
            if (sel) s_words[at + __popc(mask & ((1u << lane) - 1u))] = (Word)(((u32)j << 2) | (k < 0.f ? 3u : 1u));
            // (the second quantiser needs |G| itself: it was written through to the residue before the last barrier)
            if (a.quantiser && mask) warp_accumulate_shared(a.s_acc2, sel ? fabsf(a.residue[base + j]) : 0.f, sel);
            at += __popc(mask);
        }
    __syncthreads();

    Word *slot = reinterpret_cast<Word *>(a.scratch + geo.slots_at + tile * geo.slot_bytes);
    for (u32 i = tid; i < total; i += kGenericThreads) slot[i] = s_words[i];
    if (tid == 0) {
        reinterpret_cast<Word *>(a.packed + geo.bin_cnt_at)[tile] = (Word)total;       // (a tile is a bin)
        reinterpret_cast<u32 *>(a.scratch + geo.tile_cnt_at)[tile] = total;
        if (total) atomicAdd(&reinterpret_cast<u64 *>(a.scratch + geo.group_at)[tile / kGroupTiles], (u64)total);
        u32 window;
        u64 lo, hi;
        if (split_for_sum(m, window, lo, hi)) {
            atomicAdd(&s_acc[window], lo);
            atomicAdd(&s_acc[window + 1], hi);
        }
    }
    __syncthreads();
}

template <typename Word>
__global__ void __launch_bounds__(kGenericThreads)
tile_pass_generic(PassArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 s_tmp[33];
    __shared__ u64 s_acc[kWindows + 1], s_acc2[kWindows + 1];
    const int tid = threadIdx.x;
    if (tid < kWindows + 1) s_acc[tid] = s_acc2[tid] = 0;
    __syncthreads();
    const TileIo io{a.grad, a.residue, a.packed, a.scratch, a.literal, a.factor, a.grad_type, a.quantiser, s_acc2};
    for (u64 tile = blockIdx.x; tile < a.geo.n_tiles; tile += gridDim.x) {
        if (a.geo.tile_bins == 1u && sizeof(Word) == 2) generic_tile_one_bin<Word>(io, a.geo, tile, smem_raw, s_tmp, s_acc);
        else generic_tile<Word>(io, a.geo, tile, smem_raw, s_tmp, s_acc);
    }
    if (tid < kWindows) {
        const u64 v = s_acc[tid], v2 = s_acc2[tid];
        if (v) atomicAdd(reinterpret_cast<u64 *>(a.scratch) + tid, v);
        if (v2) atomicAdd(reinterpret_cast<u64 *>(a.scratch + kCtlSentSumAt) + tid, v2);
    }
}

// ---------------------------------------------------------------------------------
// finalize: one CTA.  Exact sum -> scale; group counts -> exclusive scan; header.
// ---------------------------------------------------------------------------------

// The nine windows hold the exact sum of the bin maxima in units of 2^-149.  Returns the
// double nearest to it (ties to even).
__device__ inline double windows_to_double(const u64 *win)
{
    u32 limb[kWindows + 2];
    u64 carry = 0;
    for (int i = 0; i < kWindows; i++) {
        const u64 s = win[i] + carry;
        limb[i] = (u32)s;
        carry = s >> 32;
    }
    limb[kWindows] = (u32)carry;
    limb[kWindows + 1] = (u32)(carry >> 32);
    int top = -1;
    for (int i = kWindows + 1; i >= 0 && top < 0; i--)
        if (limb[i]) top = 32 * i + 31 - __clz(limb[i]);
    if (top < 0) return 0.0;
    if (top <= 52) {
        const u64 v = ((u64)limb[1] << 32) | limb[0];
        return scalbn((double)v, -149);
    }
    const int low = top - 52;                    // lowest kept bit
    u64 mant = 0;
    for (int pos = top; pos >= low; pos--)
        mant = (mant << 1) | ((limb[pos >> 5] >> (pos & 31)) & 1u);
    const int rpos = low - 1;
    const u32 round_bit = (limb[rpos >> 5] >> (rpos & 31)) & 1u;
    bool sticky = false;
    for (int i = 0; i < (rpos >> 5); i++) sticky = sticky || limb[i] != 0;
    if (rpos & 31) sticky = sticky || (limb[rpos >> 5] & ((1u << (rpos & 31)) - 1u)) != 0;
    if (round_bit && (sticky || (mant & 1ull))) mant += 1;
    return scalbn((double)mant, low - 149);
}

// The whole CTA (any number of whole warps).  `prefix`: where the groups' running sums go: null for "in place, over the
// counts" (the finalize kernel), else an array of n_groups entries that the counts are scanned into (a gather
// kernel that does this work itself, every CTA into its own shared memory).  `head`: this CTA writes the header,
// count_out, the gaps and the lazy-scale state (exactly one CTA of a launch does).  Returns the scale (in thread 0).
__device__ inline float finalize_body(unsigned char *packed, unsigned char *scratch, const Geometry &geo, u32 flags,
                                      u64 *count_out, unsigned char *lazy_state, u64 *prefix = nullptr, bool head = true)
{
    __shared__ u64 s_warp[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const u64 *group = reinterpret_cast<const u64 *>(scratch + geo.group_at);
    u64 *const sums = prefix ? prefix : reinterpret_cast<u64 *>(scratch + geo.group_at);
    if (tid < 33) s_warp[tid] = 0;
    __syncthreads();

    // exclusive scan of the per-group word counts
    const u64 per = (geo.n_groups + blockDim.x - 1) / blockDim.x;
    const u64 lo = min((u64)tid * per, geo.n_groups), hi = min(lo + per, geo.n_groups);
    u64 sum = 0;
    for (u64 i = lo; i < hi; i++) sum += group[i];
    u64 inc = sum;
    for (int d = 1; d < 32; d <<= 1) {
        const u64 t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const u64 v = s_warp[lane];
        u64 s = v;
        for (int d = 1; d < 32; d <<= 1) {
            const u64 t = __shfl_up_sync(0xffffffffu, s, d);
            if (lane >= d) s += t;
        }
        s_warp[lane] = s - v;
        if (lane == 31) s_warp[32] = s;
    }
    __syncthreads();
    u64 run = s_warp[warp] + inc - sum;
    for (u64 i = lo; i < hi; i++) {
        const u64 c = group[i];
        sums[i] = run;
        run += c;
    }
    const u64 n_sel = s_warp[32];

    float scale = 0.f;
    if (tid == 0) {
        const u64 *win = reinterpret_cast<const u64 *>(scratch);
        if (flags & kFlagQuant) {
            // the second quantiser: the mean |G| of the sent elements
            if (n_sel) scale = __double2float_rn(__ddiv_rn(windows_to_double(win + kCtlSentSumAt / 8), (double)n_sel));
        } else if (geo.n_bins) {
            const double S = windows_to_double(win);
            scale = __double2float_rn(__ddiv_rn(S, (double)geo.n_bins));
        }
    }
    if (!head) return scale;
    if (tid == 0) {
        u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);
        tile_off[geo.n_tiles] = n_sel;
        const u64 bytes_used = geo.payload_at + align_up(n_sel * geo.w, 16);
        u32 *h32 = reinterpret_cast<u32 *>(packed);
        u64 *h64 = reinterpret_cast<u64 *>(packed);
        h32[0] = kMagic;
        h32[1] = 1u | (geo.w << 16) | ((flags & (ADACOMP_FLAG_LITERAL | kFlagFactor | kFlagQuant)) << 24);
        h32[2] = geo.L_T;
        h32[3] = geo.tile_bins;
        h64[2] = geo.n;
        h64[3] = geo.n_bins;
        h64[4] = geo.n_tiles;
        h64[5] = n_sel;
        h32[12] = __float_as_uint(scale);
        h32[13] = 0;
        h64[7] = bytes_used;
        count_out[0] = n_sel;
        count_out[1] = bytes_used;
        if (lazy_state) {
            LazyHeader *lh = reinterpret_cast<LazyHeader *>(lazy_state);
            if (lh->magic == kLazyMagic && lh->n == geo.n && lh->L_T == geo.L_T) {
                lh->scale = scale;      // the next step (or a flush) finishes the sent residues with it
                lh->steps += 1;
            }
        }
    }
    // zero padding behind the last word, and the alignment gaps of the directory sections
    const u64 pay_end = geo.payload_at + n_sel * geo.w;
    const u64 pad = align_up(pay_end, 16) - pay_end;
    if ((u64)tid < pad) packed[pay_end + tid] = 0;
    const u64 dir_end = geo.tile_off_at + 8 * (geo.n_tiles + 1);
    if ((u64)tid < geo.bin_cnt_at - dir_end) packed[dir_end + tid] = 0;
    const u64 cnt_end = geo.bin_cnt_at + geo.n_bins * geo.w;
    if ((u64)tid < geo.payload_at - cnt_end) packed[cnt_end + tid] = 0;
    return scale;
}

// ---------------------------------------------------------------------------------
// gather_fixup: per tile, copy the slot's words to the payload, write the tile's
// directory entry and finish the residue of the sent elements:
// residue = G - sign(G) * scale  (Algorithm 2, the "if" branch).
// ---------------------------------------------------------------------------------

// Words before `tile`: its group's scanned offset plus the counts of the tiles before it
// in the group.  Warp-collective; also returns the tile's own count.
__device__ inline u64 tile_offset(const unsigned char *scratch, const Geometry &geo, u64 tile, int lane,
                                  u32 &count, const u64 *group_sums = nullptr)
{
    const u32 *tile_cnt = reinterpret_cast<const u32 *>(scratch + geo.tile_cnt_at);
    const u64 *group = group_sums ? group_sums : reinterpret_cast<const u64 *>(scratch + geo.group_at);
    const u64 g = tile / kGroupTiles;
    const int me = (int)(tile % kGroupTiles);
    const u64 t = g * kGroupTiles + lane;
    const u32 c = t < geo.n_tiles ? tile_cnt[t] : 0u;
    u32 before = lane < me ? c : 0u;
    for (int d = 16; d > 0; d >>= 1) before += __shfl_xor_sync(0xffffffffu, before, d);
    count = min(__shfl_sync(0xffffffffu, c, me), geo.tile_elems);
    return group[g] + before;
}

#ifndef ADACOMP_GATHER_AHEAD
#define ADACOMP_GATHER_AHEAD 8
#endif
constexpr int kGatherAhead = ADACOMP_GATHER_AHEAD;     // words a lane of the gather has in flight

// One tile of at most 96 bins, handled by one warp.
// group_sums / scale_bits: null / unused where a finalize kernel ran before (the groups' running sums are in the
// scratch, the scale in the header); else the CTA's own copies.
template <typename Word, bool FIXUP>
__device__ void gather_tile_small(float *residue, unsigned char *packed, const unsigned char *scratch,
                                  const Geometry &geo, u64 tile, int lane, u32 *s_pre, const u64 *group_sums = nullptr,
                                  u32 scale_bits = 0u)
{
    const int TB = (int)geo.tile_bins;
    u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);
    const Word *bin_cnt = reinterpret_cast<const Word *>(packed + geo.bin_cnt_at);
    Word *payload = reinterpret_cast<Word *>(packed + geo.payload_at);
    const float scale = __uint_as_float(group_sums ? scale_bits : reinterpret_cast<const u32 *>(packed)[12]);
    u32 cnt;
    const u64 off0 = tile_offset(scratch, geo, tile, lane, cnt, group_sums);
    if (lane == 0) tile_off[tile] = off0;
    if (cnt == 0) return;
    // exclusive scan of the tile's bin counts, three bins per lane (only the fix-up needs bins)
    const u64 bin0 = tile * (u64)TB;
    u32 c[3], sum = 0;
    if (FIXUP) {
#pragma unroll
    for (int q = 0; q < 3; q++) {
        const int b = lane * 3 + q;
        c[q] = (b < TB && bin0 + b < geo.n_bins) ? (u32)bin_cnt[bin0 + b] : 0u;
        sum += c[q];
    }
    const u32 inc = warp_inclusive_scan(sum, lane);
    u32 run = inc - sum;
    __syncwarp();
#pragma unroll
    for (int q = 0; q < 3; q++) {
        const int b = lane * 3 + q;
        if (b < TB) s_pre[b] = run;
        run += c[q];
    }
    if (lane == 31) s_pre[TB] = inc;
    __syncwarp();
    }
    const Word *slot = reinterpret_cast<const Word *>(scratch + geo.slots_at + tile * geo.slot_bytes);
    const u64 base = tile * (u64)geo.tile_elems;
    for (u32 j0 = 0; j0 < cnt; j0 += 32 * kGatherAhead) {
        // kGatherAhead words per lane per round: their residue loads overlap
        u32 word[kGatherAhead];
        u64 pos[kGatherAhead];
        float g[kGatherAhead];
#pragma unroll
        for (int q = 0; q < kGatherAhead; q++) {
            const u32 j = j0 + q * 32 + lane;
            word[q] = 0;
            pos[q] = 0;
            g[q] = 0.f;
            if (j < cnt) {
                word[q] = slot[j];
                if (FIXUP) {
                    const int b = bin_of_word(s_pre, TB, j);
                    pos[q] = base + (u64)b * geo.L_T + (word[q] >> 2);
                    g[q] = residue[pos[q]];
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kGatherAhead; q++) {
            const u32 j = j0 + q * 32 + lane;
            if (j < cnt) {
                if (FIXUP) residue[pos[q]] = (word[q] & 2u) ? __fadd_rn(g[q], scale) : __fsub_rn(g[q], scale);
                payload[off0 + j] = (Word)word[q];
            }
        }
    }
    __syncwarp();
}

// Tiles of at most 96 bins: one warp per tile.
template <typename Word, bool FIXUP>
__global__ void __launch_bounds__(kGatherThreads)
gather_fixup_small(float *residue, unsigned char *packed, const unsigned char *scratch, Geometry geo)
{
    __shared__ u32 s_pre_all[kGatherThreads / 32][kSmallBins + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u64 warps = (u64)gridDim.x * (kGatherThreads / 32);
    // Last tile first: the tile pass wrote the residue front to back, so its tail is what the
    // L2 still holds when this kernel starts.
    for (u64 item = (u64)blockIdx.x * (kGatherThreads / 32) + warp; item < geo.n_tiles; item += warps)
        gather_tile_small<Word, FIXUP>(residue, packed, scratch, geo, geo.n_tiles - 1 - item, lane, s_pre_all[warp]);
}

// The same with finalize's work done here, for layers of at most kFoldGroups groups of 32 tiles (2^27 elements): every
// CTA scans the groups' counts into its shared memory and works the scale out (8 KB read from L2 and a microsecond,
// all CTAs at once) instead of waiting for a kernel of one CTA to do it; the first CTA also writes the header.
constexpr u32 kFoldGroups = 1024;
template <typename Word, bool FIXUP>
__global__ void __launch_bounds__(kGatherThreads)
gather_fixup_fold(float *residue, unsigned char *packed, unsigned char *scratch, Geometry geo, u32 flags, u64 *count_out,
                  unsigned char *lazy_state)
{
    __shared__ u32 s_pre_all[kGatherThreads / 32][kSmallBins + 1];
    __shared__ u64 s_sums[kFoldGroups];
    __shared__ u32 s_scale_bits;
    const float scale = finalize_body(packed, scratch, geo, flags, count_out, lazy_state, s_sums, blockIdx.x == 0);
    if (threadIdx.x == 0) s_scale_bits = __float_as_uint(scale);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u64 warps = (u64)gridDim.x * (kGatherThreads / 32);
    for (u64 item = (u64)blockIdx.x * (kGatherThreads / 32) + warp; item < geo.n_tiles; item += warps)
        gather_tile_small<Word, FIXUP>(residue, packed, scratch, geo, geo.n_tiles - 1 - item, lane, s_pre_all[warp], s_sums, s_scale_bits);
}

// Any tile shape: one CTA per tile.
template <typename Word>
__global__ void __launch_bounds__(kGatherThreads)
gather_fixup(float *residue, unsigned char *packed, const unsigned char *scratch, Geometry geo)
{
    __shared__ u32 s_pre[kMaxTileBins + 1];
    __shared__ u32 s_tmp[33];
    __shared__ u64 s_off0;
    __shared__ u32 s_count;
    const int tid = threadIdx.x;
    const int TB = (int)geo.tile_bins;
    u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);
    const Word *bin_cnt = reinterpret_cast<const Word *>(packed + geo.bin_cnt_at);
    Word *payload = reinterpret_cast<Word *>(packed + geo.payload_at);
    const float scale = __uint_as_float(reinterpret_cast<const u32 *>(packed)[12]);

    for (u64 tile = blockIdx.x; tile < geo.n_tiles; tile += gridDim.x) {
        if (tid < 32) {
            u32 c;
            const u64 o = tile_offset(scratch, geo, tile, tid, c);
            if (tid == 0) { s_off0 = o; s_count = c; tile_off[tile] = o; }
        }
        __syncthreads();
        const u64 off0 = s_off0;
        const u32 cnt = s_count;
        if (cnt == 0) { __syncthreads(); continue; }
        const u64 bin0 = tile * (u64)TB;
        for (int b = tid; b < TB; b += kGatherThreads)
            s_pre[b] = bin0 + b < geo.n_bins ? (u32)bin_cnt[bin0 + b] : 0u;
        __syncthreads();
        block_exclusive_scan(s_pre, TB, s_tmp);
        const Word *slot = reinterpret_cast<const Word *>(scratch + geo.slots_at + tile * geo.slot_bytes);
        const u64 base = tile * (u64)geo.tile_elems;
        for (u32 j = tid; j < cnt; j += kGatherThreads) {
            const u32 word = slot[j];
            const int b = bin_of_word(s_pre, TB, j);
            const u64 pos = base + (u64)b * geo.L_T + (word >> 2);
            const float g = residue[pos];
            residue[pos] = (word & 2u) ? __fadd_rn(g, scale) : __fsub_rn(g, scale);
            payload[off0 + j] = (Word)word;
        }
        __syncthreads();
    }
}


// The fast tile pass takes L_T = 25 * SPB for the divisors SPB of 40 but 1 (tiles of exactly 4000 elements):
// 50, 100, 125, 200, 250, 500 and 1000.
__host__ __device__ inline bool fast_L_T(u32 L_T)
{
    return L_T == 50u || L_T == 100u || L_T == 125u || L_T == 200u || L_T == 250u || L_T == 500u || L_T == 1000u;
}
constexpr u32 kFastL_T[] = {50u, 100u, 125u, 200u, 250u, 500u, 1000u};
// Every other L_T from 41 to 1000 (tiles of at most 96 bins, bins longer than a thread's 25 elements) takes
// the same kernel in its any-bin form (fp32 gradient), and so do the one-bin tiles of at most 4000 elements
// that start on 16-byte boundaries (L_T up to 4000, a multiple of 4).
__host__ __device__ inline bool any_fast_L_T(u32 L_T)
{
    return (L_T >= 41u && L_T <= 1000u && !fast_L_T(L_T)) || (L_T > 1000u && L_T <= (u32)kFastTile && L_T % 4u == 0);
}

}  // namespace adacomp_impl
