// One-kernel pack() for layers that fit on the chip: what the single-layer kernel (pack_onchip.cu) and the kernel for
// a whole parameter list (pack_onchip_list.cu) share: the shared-memory layout, one tile of phase 1, the header.
#pragma once

#include "internal.h"

namespace adacomp_impl {

constexpr int kOnchipSlots = 4;         // tiles a CTA keeps in shared memory
constexpr int kOnchipStages = 2;        // gradient tiles in flight
constexpr u32 kCtlMeetAt = 96;          // control block: the CTAs' meeting counter (u32), behind the nine windows

struct OnchipSmem {
    static constexpr u32 kSlotsAt = 0;                                       // [4][4000] floats: residue in, G, new residue out
    static constexpr u32 kGradAt = kOnchipSlots * kTileBytes;                // [2][4000] floats
    static constexpr u32 kWordsAt = kGradAt + kOnchipStages * kTileBytes;    // one tile's words (16-bit worst case)
    static constexpr u32 kInclAt = kWordsAt + 2 * kFastTile;
    static constexpr u32 kWtotAt = kInclAt + 4 * kTileSegs;
    static constexpr u32 kSegmaxAt = kWtotAt + 32;
    static constexpr u32 kBinmaxAt = kSegmaxAt + 4 * kTileSegs;              // [80] floats
    static constexpr u32 kMaskAt = kBinmaxAt + 4 * 80;                       // [4][160] u32: which of a thread's 25 elements are sent
    static constexpr u32 kSumsAt = kMaskAt + 4 * kTileSegs * kOnchipSlots;           // [6][2] u64: per-warp partial sums of tile counts
    static constexpr u32 kAccAt = kSumsAt + 8 * 6 * 2;                       // [10] u64 exact-sum windows
    static constexpr u32 kBarAt = kAccAt + 8 * (kWindows + 1);               // [4] residue + [2] gradient mbarriers
    static constexpr u32 kMiscAt = kBarAt + 8 * (kOnchipSlots + kOnchipStages);      // scale bits, abort flag
    static constexpr u32 kBytes = kMiscAt + 32;
};
static_assert(OnchipSmem::kAccAt % 8 == 0 && OnchipSmem::kSumsAt % 8 == 0 && OnchipSmem::kBarAt % 8 == 0, "8-byte aligned");
static_assert(2 * OnchipSmem::kBytes <= 227 * 1024, "two CTAs per SM");

// One tile of phase 1 (the whole CTA): G = residue + dW, the bins' maxima, the selection, the words into the staging
// area and from there into the tile's slot in the scratch, the bin counts into the stream, the tile's word count, the
// bins' maxima into the CTA's exact sum; G stays in shared-memory slot i, with a mask per thread of what was sent.
// This is tile_pass_fast's tile code for bins of SPB whole segments.
struct OnchipTile {
    const float *grad, *residue;        // the layer's arrays
    u64 tile;                           // the tile's number in its layer
    u64 n, n_bins;                      // the layer's elements and bins
    unsigned char *bin_cnt;             // the count section of the layer's stream
    unsigned char *slot;                // the tile's slot for words in the layer's scratch
    u32 *tile_cnt;                      // the layer's word counts per tile
    float factor;                       // 0: H = G + dW
    long long wait_limit;
    bool whole;                         // the tile came by bulk copies (else: the ragged last tile, plain loads)
};

template <int SPB, typename Word>
__device__ __forceinline__ void onchip_tile(unsigned char *smem, int i, const OnchipTile &t)
{
    Word *s_words = reinterpret_cast<Word *>(smem + OnchipSmem::kWordsAt);
    u32 *s_incl = reinterpret_cast<u32 *>(smem + OnchipSmem::kInclAt);
    u32 *s_wtot = reinterpret_cast<u32 *>(smem + OnchipSmem::kWtotAt);
    float *s_segmax = reinterpret_cast<float *>(smem + OnchipSmem::kSegmaxAt);
    float *s_binmax = reinterpret_cast<float *>(smem + OnchipSmem::kBinmaxAt);
    u32 *s_mask = reinterpret_cast<u32 *>(smem + OnchipSmem::kMaskAt);
    u64 *s_acc = reinterpret_cast<u64 *>(smem + OnchipSmem::kAccAt);
    u64 *s_res_bar = reinterpret_cast<u64 *>(smem + OnchipSmem::kBarAt);
    u64 *s_grad_bar = s_res_bar + kOnchipSlots;
    volatile u32 *s_misc = reinterpret_cast<volatile u32 *>(smem + OnchipSmem::kMiscAt);     // [0] scale bits, [1] abort
    volatile u32 *s_tcnt = s_misc + 4;                                                       // [4] words of the CTA's tiles
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    constexpr int kBins = kTileSegs / SPB;
    float *s_d = reinterpret_cast<float *>(smem + OnchipSmem::kGradAt) + (i % kOnchipStages) * kFastTile;
    float *s_r = reinterpret_cast<float *>(smem + OnchipSmem::kSlotsAt) + i * kFastTile;
    const u64 base = t.tile * (u64)kFastTile;
    Word *bin_cnt = reinterpret_cast<Word *>(t.bin_cnt);

    if (t.whole) {
        const bool ok = mbar_wait(&s_res_bar[i], 0u, t.wait_limit) &&
                        mbar_wait(&s_grad_bar[i % kOnchipStages], (u32)(i / kOnchipStages) & 1u, t.wait_limit);
        if (!ok) {
            s_misc[1] = 1;
            raise_status(ADACOMP_DEV_TIMEOUT);
        }
    } else {
        const int elems = (int)(t.n - base);
        for (int e = tid; e < kFastTile; e += kFastThreads) {
            float d = 0.f, r = 0.f;
            if (e < elems) { d = t.grad[base + e]; r = t.residue[base + e]; }
            s_d[e] = d;
            s_r[e] = r;
        }
        __syncthreads();
    }

    float g[kSeg], key[kSeg];
    float gm = 0.f;
    u32 selmask = 0, cnt = 0, incl = 0;
    if (!service) {
        const float *pd = s_d + tid * kSeg;
        const float *pr = s_r + tid * kSeg;
        float m = 0.f;
#pragma unroll
        for (int j = 0; j < kSeg; j++) {
            const float d = pd[j], r = pr[j];
            g[j] = __fadd_rn(r, d);
            const float h = t.factor != 0.f ? __fadd_rn(r, __fmul_rn(t.factor, d)) : __fadd_rn(g[j], d);
            m = fmaxf(m, fabsf(g[j]));
            // |G| never exceeds the bin maximum, so "|H| >= g_max or |G| == g_max" is "max(|H|, |G|) >= g_max"
            key[j] = fmaxf(fabsf(h), fabsf(g[j]));
        }
        if (SPB == 2) gm = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
        else s_segmax[tid] = m;
    }
    if (SPB != 2) {
        __syncthreads();                                        // barrier A
        if (!service) {
            const int bin = tid / SPB;
#pragma unroll
            for (int s = 0; s < SPB; s++) gm = fmaxf(gm, s_segmax[bin * SPB + s]);
        }
    }
    if (!service) {
        if (tid % SPB == 0) s_binmax[tid / SPB] = gm;
#pragma unroll
        for (int j = 0; j < kSeg; j++)
            if (key[j] >= gm && g[j] != 0.f) selmask |= 1u << j;
        cnt = __popc(selmask);
        s_mask[i * kTileSegs + tid] = selmask;
        incl = warp_inclusive_scan(cnt, lane);
        s_incl[tid] = incl;
        if (lane == 31) s_wtot[warp] = incl;
    }
    __syncthreads();                                            // barrier B

    u32 total = 0;
    if (!service) {
        u32 wpre[6];
        wpre[0] = 0;
#pragma unroll
        for (int wv = 0; wv < 5; wv++) wpre[wv + 1] = wpre[wv] + s_wtot[wv];
        const u32 mine = wpre[warp] + incl;                     // inclusive position
        float *pr = s_r + tid * kSeg;
#pragma unroll
        for (int j = 0; j < kSeg; j++) pr[j] = g[j];            // the slot now holds G
        u32 at = mine - cnt;
        const u32 seg_in_bin = (u32)(tid % SPB) * kSeg;
        u32 mask = selmask;
        while (mask) {
            const int j = __ffs(mask) - 1;
            mask &= mask - 1;
            const u32 neg = __float_as_uint(pr[j]) >> 31;
            s_words[at++] = (Word)(((seg_in_bin + j) << 2) | 1u | (neg << 1));
        }
        if (tid % SPB == 0) {
            const u64 bin = t.tile * (u64)kBins + tid / SPB;
            const int t1 = tid + SPB - 1;
            const u32 last = wpre[t1 >> 5] + s_incl[t1], count = last - mine + cnt;
            if (bin < t.n_bins) bin_cnt[bin] = (Word)count;
        }
    } else {
        total = s_wtot[0] + s_wtot[1] + s_wtot[2] + s_wtot[3] + s_wtot[4];
        for (int bb = 0; bb < kBins; bb += 32) {    // every lane takes part each round
            const int b = bb + lane;
            const bool valid = b < kBins && t.tile * (u64)kBins + b < t.n_bins;
            warp_accumulate(s_acc, valid ? s_binmax[b] : 0.f, valid);
        }
    }
    __syncthreads();                                            // barrier D
    if (service) {
        // the tile's words wait in its scratch slot for their place in the stream
        uint4 *slot = reinterpret_cast<uint4 *>(t.slot);
        const int chunks = (int)((total * sizeof(Word) + 15) / 16);
        for (int c = lane; c < chunks; c += 32) slot[c] = reinterpret_cast<uint4 *>(s_words)[c];
        if (lane == 0) {
            t.tile_cnt[t.tile] = total;
            s_tcnt[i] = total;
        }
    }
}

// The stream's header, count_out, the directory's last entry and the zeroes of the alignment gaps (the whole CTA).
__device__ inline void onchip_header(unsigned char *packed, const Geometry &geo, u32 header_flags, float scale, u64 n_sel,
                                     u64 *count_out)
{
    const int tid = threadIdx.x;
    if (tid == 0) {
        reinterpret_cast<u64 *>(packed + geo.tile_off_at)[geo.n_tiles] = n_sel;
        const u64 bytes_used = geo.payload_at + align_up(n_sel * geo.w, 16);
        u32 *h32 = reinterpret_cast<u32 *>(packed);
        u64 *h64 = reinterpret_cast<u64 *>(packed);
        h32[0] = kMagic;
        h32[1] = 1u | (geo.w << 16) | ((header_flags & (ADACOMP_FLAG_LITERAL | kFlagFactor | kFlagQuant)) << 24);
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
    }
    const u64 pay_end = geo.payload_at + n_sel * geo.w;
    const u64 pad = align_up(pay_end, 16) - pay_end;
    if ((u64)tid < pad) packed[pay_end + tid] = 0;
    const u64 dir_end = geo.tile_off_at + 8 * (geo.n_tiles + 1);
    if ((u64)tid < geo.bin_cnt_at - dir_end) packed[dir_end + tid] = 0;
    const u64 cnt_end = geo.bin_cnt_at + geo.n_bins * geo.w;
    if ((u64)tid < geo.payload_at - cnt_end) packed[cnt_end + tid] = 0;
}

}  // namespace adacomp_impl
