// libadacomp: AdaComp pack() / unpack()-and-sum for one B200 (sm_100a).
//
// pack() (Algorithm 2 of the paper) runs as three kernels on the caller's stream:
//   tile_pass     one read of dW and residue, one write of residue (= G everywhere);
//                 per-bin max |G|, selection, words compacted per tile into a scratch
//                 slot, per-bin counts, per-tile counts, exact partial sums of g_max
//   finalize      exact sum -> scale, scan of the tile counts, header, count_out
//   gather_fixup  moves each tile's words to their final place and subtracts
//                 sign * scale from the residue of the sent elements only
// The layer-wide scale (Section 2.5: mean of the g_max vector) is needed by every
// sent element's residue but is known only after every bin has been seen; that is
// why the residue of sent elements is finished by the third kernel.
//
// unpack()-and-sum is one kernel: each CTA owns an output tile in shared memory,
// adds the k learners' words into it in learner order and stores it once.
//
// HBM-bandwidth bound; no tensor cores (nothing here is a contraction).

#include <cuda_runtime.h>
#include <stdint.h>

#include "adacomp.h"

namespace {

typedef unsigned long long u64;
typedef unsigned int u32;

constexpr u32 kMagic = 0x31434441u;
constexpr u32 kHeaderBytes = 64;
constexpr u32 kCtlBytes = 256;       // control block at the start of the scratch area
constexpr int kWindows = 9;          // 32-bit windows of the exact g_max accumulator
constexpr int kSeg = 25;             // elements per thread on the fast path
constexpr int kTileSegs = 160;       // segments per tile on the fast path
constexpr int kFastTile = kSeg * kTileSegs;   // 4000 elements
constexpr int kFastThreads = 192;
constexpr int kGenericThreads = 256;
constexpr int kDecodeChunk = 4096;   // output elements per decode work item
constexpr int kDecodeThreads = 256;
constexpr int kGatherThreads = 128;
constexpr int kMaxTileBins = 4000;

__device__ u32 g_status;             // sticky ADACOMP_DEV_* bits of this device

__host__ __device__ inline u64 align_up(u64 x, u64 a) { return (x + a - 1) / a * a; }

// Section offsets of a packed stream and of the scratch behind it.
struct Geometry {
    u32 w, L_T, tile_bins, tile_elems;
    u64 n, n_bins, n_tiles;
    u64 tile_off_at, bin_cnt_at, payload_at, ctl_at, slots_at, slot_bytes, capacity;
};

__host__ __device__ inline Geometry make_geometry(u64 n, u32 L_T)
{
    Geometry g;
    g.n = n;
    g.L_T = L_T;
    g.w = L_T <= 64u ? 1u : 2u;
    g.tile_bins = L_T <= 1000u ? 4u * (1000u / L_T) : 1u;
    g.tile_elems = g.tile_bins * L_T;
    g.n_bins = (n + L_T - 1) / L_T;
    g.n_tiles = (g.n_bins + g.tile_bins - 1) / g.tile_bins;
    g.tile_off_at = kHeaderBytes;
    g.bin_cnt_at = align_up(g.tile_off_at + 8 * (g.n_tiles + 1), 16);
    g.payload_at = align_up(g.bin_cnt_at + g.n_bins * g.w, 16);
    g.ctl_at = align_up(g.payload_at + align_up(n * g.w, 16), 256);
    g.slots_at = g.ctl_at + kCtlBytes;
    g.slot_bytes = align_up((u64)g.tile_elems * g.w, 16);
    g.capacity = g.slots_at + g.n_tiles * g.slot_bytes;
    return g;
}

// ---------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------

__device__ inline void raise_status(u32 bits) { atomicOr(&g_status, bits); }

// Exclusive scan, in place, of a[0..count) in shared memory; a[count] receives the total.
// Called by every thread of the CTA; contains barriers.
__device__ inline void block_exclusive_scan(u32 *a, int count, u32 *warp_tmp /* >= 33 */)
{
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int per = (count + nthr - 1) / nthr;
    const int lo = min(tid * per, count), hi = min(lo + per, count);
    u32 sum = 0;
    for (int i = lo; i < hi; i++) sum += a[i];
    // scan of the per-thread sums: warp shuffles, then the warp totals
    const int lane = tid & 31, warp = tid >> 5, nwarp = (nthr + 31) >> 5;
    u32 inc = sum;
    for (int d = 1; d < 32; d <<= 1) {
        u32 t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) warp_tmp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        u32 v = lane < nwarp ? warp_tmp[lane] : 0u;
        u32 s = v;
        for (int d = 1; d < 32; d <<= 1) {
            u32 t = __shfl_up_sync(0xffffffffu, s, d);
            if (lane >= d) s += t;
        }
        warp_tmp[lane] = s - v;
        if (lane == 31) warp_tmp[32] = s;
    }
    __syncthreads();
    u32 run = warp_tmp[warp] + inc - sum;
    for (int i = lo; i < hi; i++) {
        u32 v = a[i];
        a[i] = run;
        run += v;
    }
    if (tid == 0) a[count] = warp_tmp[32];
    __syncthreads();
}

// Largest b in [0, bins) with prefix[b] <= j  (prefix is an exclusive scan, prefix[bins] > j).
__device__ inline int bin_of_word(const u32 *prefix, int bins, u32 j)
{
    int lo = 0, hi = bins;           // invariant: prefix[lo] <= j < prefix[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (prefix[mid] <= j) lo = mid; else hi = mid;
    }
    return lo;
}

// A non-negative finite binary32 value is m * 2^(sh - 149) with m < 2^24.  The exact
// accumulator keeps the sum of all bin maxima as nine 64-bit counters of 32-bit windows.
__device__ inline bool split_for_sum(float gm, u32 &window, u64 &lo, u64 &hi)
{
    const u32 bits = __float_as_uint(gm) & 0x7fffffffu;
    const u32 e = bits >> 23;
    if (e == 255u) { raise_status(ADACOMP_DEV_NONFINITE); return false; }
    const u64 m = e ? ((bits & 0x7fffffu) | 0x800000u) : (bits & 0x7fffffu);
    if (m == 0) return false;
    const u32 sh = e ? e - 1u : 0u;
    const u64 v = m << (sh & 31u);
    window = sh >> 5;
    lo = v & 0xffffffffull;
    hi = v >> 32;
    return true;
}

// Warp-collective add of one value per lane into the CTA's accumulator, which only this
// warp touches.  Lanes whose values fall into one window are summed by shuffles first.
__device__ inline void warp_accumulate(u64 *acc, float gm, bool valid)
{
    const u32 full = 0xffffffffu;
    u32 window = 0;
    u64 lo = 0, hi = 0;
    valid = valid && split_for_sum(gm, window, lo, hi);
    const u32 vm = __ballot_sync(full, valid);
    if (vm == 0) return;
    const u32 w0 = __shfl_sync(full, window, __ffs(vm) - 1);
    if (__all_sync(full, !valid || window == w0)) {
        if (!valid) { lo = 0; hi = 0; }
        for (int d = 16; d > 0; d >>= 1) {
            lo += __shfl_down_sync(full, lo, d);
            hi += __shfl_down_sync(full, hi, d);
        }
        if ((threadIdx.x & 31) == 0) { acc[w0] += lo; acc[w0 + 1] += hi; }
    } else if (valid) {
        atomicAdd(&acc[window], lo);
        atomicAdd(&acc[window + 1], hi);
    }
    __syncwarp();
}

// ---------------------------------------------------------------------------------
// tile_pass, fast path: L_T = 25 * SPB (50 and 500), tiles of 4000 elements.
// Thread t < 160 owns the 25 consecutive elements of segment t (stride 25 words in
// shared memory: odd, so the warp's accesses are bank-conflict free); a bin is SPB
// adjacent segments.  Warp 5 has no segment: it feeds the exact g_max accumulator.
// ---------------------------------------------------------------------------------

struct PassArgs {
    const float *grad;
    float *residue;
    unsigned char *packed;
    Geometry geo;
    u32 literal;
};

template <int SPB, typename Word>
__global__ void __launch_bounds__(kFastThreads)
tile_pass_fast(PassArgs a)
{
    __shared__ __align__(16) float s_d[kFastTile];     // dW, later the word staging area
    __shared__ __align__(16) float s_r[kFastTile];     // residue, later G
    __shared__ float s_segmax[kTileSegs];
    __shared__ u32 s_off[kTileSegs + 1];
    __shared__ u64 s_acc[kWindows + 1];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const Geometry &geo = a.geo;
    constexpr int kBins = kTileSegs / SPB;
    u64 *tile_cnt = reinterpret_cast<u64 *>(a.packed + geo.tile_off_at);
    Word *bin_cnt = reinterpret_cast<Word *>(a.packed + geo.bin_cnt_at);
    Word *s_words = reinterpret_cast<Word *>(s_d);

    if (tid < kWindows + 1) s_acc[tid] = 0;

    for (u64 tile = blockIdx.x; tile < geo.n_tiles; tile += gridDim.x) {
        const u64 base = tile * (u64)kFastTile;
        const u64 left = geo.n - base;
        const int elems = left < (u64)kFastTile ? (int)left : kFastTile;

        // ---- load the tile (128-bit, coalesced; zero fill past the end) ----
        const float4 *gd = reinterpret_cast<const float4 *>(a.grad + base);
        const float4 *gr = reinterpret_cast<const float4 *>(a.residue + base);
        for (int i = tid; i < kFastTile / 4; i += kFastThreads) {
            float4 d = make_float4(0.f, 0.f, 0.f, 0.f), r = d;
            if (4 * i + 3 < elems) {
                d = __ldcs(gd + i);
                r = __ldcs(gr + i);
            } else {
                float *pd = &d.x, *pr = &r.x;
                for (int c = 0; c < 4; c++)
                    if (4 * i + c < elems) {
                        pd[c] = a.grad[base + 4 * i + c];
                        pr[c] = a.residue[base + 4 * i + c];
                    }
            }
            reinterpret_cast<float4 *>(s_d)[i] = d;
            reinterpret_cast<float4 *>(s_r)[i] = r;
        }
        __syncthreads();

        // ---- G = residue + dW; maximum |G| of the segment ----
        float g[kSeg];
        if (tid < kTileSegs) {
            float m = 0.f;
#pragma unroll
            for (int j = 0; j < kSeg; j++) {
                g[j] = __fadd_rn(s_r[tid * kSeg + j], s_d[tid * kSeg + j]);
                m = fmaxf(m, fabsf(g[j]));
            }
            s_segmax[tid] = m;
        }
        __syncthreads();

        // ---- bin maximum, selection; warp 5 adds the bin maxima to the exact sum ----
        u32 selmask = 0, negmask = 0;
        if (tid < kTileSegs) {
            const int bin = tid / SPB;
            float gm = 0.f;
#pragma unroll
            for (int s = 0; s < SPB; s++) gm = fmaxf(gm, s_segmax[bin * SPB + s]);
            if (gm > 0.f) {
#pragma unroll
                for (int j = 0; j < kSeg; j++) {
                    const float h = __fadd_rn(g[j], s_d[tid * kSeg + j]);
                    const float ag = fabsf(g[j]);
                    const bool sel = (g[j] != 0.f) &&
                                     (fabsf(h) >= gm || (!a.literal && ag == gm));
                    selmask |= (u32)sel << j;
                    negmask |= (u32)(g[j] < 0.f) << j;
                }
            }
            s_off[tid] = __popc(selmask);
        } else {
            for (int b0 = 0; b0 < kBins; b0 += 32) {    // every lane takes part each round
                const int b = b0 + lane;
                float gm = 0.f;
                if (b < kBins) {
#pragma unroll
                    for (int s = 0; s < SPB; s++) gm = fmaxf(gm, s_segmax[b * SPB + s]);
                }
                const bool valid = b < kBins && tile * (u64)kBins + b < geo.n_bins;
                warp_accumulate(s_acc, gm, valid);
            }
        }
        __syncthreads();    // s_d (dW) is dead from here on: it becomes the word staging area

        // ---- exclusive scan of the 160 segment counts (warp 0, five per lane) ----
        if (warp == 0) {
            u32 c[5], sum = 0;
#pragma unroll
            for (int q = 0; q < 5; q++) { c[q] = s_off[lane * 5 + q]; sum += c[q]; }
            u32 inc = sum;
            for (int d = 1; d < 32; d <<= 1) {
                u32 t = __shfl_up_sync(0xffffffffu, inc, d);
                if (lane >= d) inc += t;
            }
            u32 run = inc - sum;
#pragma unroll
            for (int q = 0; q < 5; q++) { s_off[lane * 5 + q] = run; run += c[q]; }
            if (lane == 31) s_off[kTileSegs] = inc;
        }
        __syncthreads();

        // ---- words into the staging area, G back into shared memory, bin counts ----
        if (tid < kTileSegs) {
            u32 at = s_off[tid];
            const u32 seg_in_bin = (u32)(tid % SPB) * kSeg;
#pragma unroll
            for (int j = 0; j < kSeg; j++) {
                if (selmask >> j & 1u) {
                    const u32 code = (negmask >> j & 1u) ? 3u : 1u;
                    s_words[at++] = (Word)(((seg_in_bin + j) << 2) | code);
                }
                s_r[tid * kSeg + j] = g[j];
            }
            if (tid % SPB == 0) {
                const u64 bin = tile * (u64)kBins + tid / SPB;
                if (bin < geo.n_bins) bin_cnt[bin] = (Word)(s_off[tid + SPB] - s_off[tid]);
            }
        }
        __syncthreads();

        // ---- store residue = G (coalesced) and the tile's words into its slot ----
        float4 *out = reinterpret_cast<float4 *>(a.residue + base);
        for (int i = tid; i < kFastTile / 4; i += kFastThreads) {
            if (4 * i + 3 < elems) {
                out[i] = reinterpret_cast<float4 *>(s_r)[i];
            } else {
                for (int c = 0; c < 4; c++)
                    if (4 * i + c < elems) a.residue[base + 4 * i + c] = s_r[4 * i + c];
            }
        }
        const u32 total = s_off[kTileSegs];
        uint4 *slot = reinterpret_cast<uint4 *>(a.packed + geo.slots_at + tile * geo.slot_bytes);
        const int chunks = (int)((total * sizeof(Word) + 15) / 16);
        for (int i = tid; i < chunks; i += kFastThreads) slot[i] = reinterpret_cast<uint4 *>(s_d)[i];
        if (tid == 0) tile_cnt[tile + 1] = total;
        __syncthreads();
    }

    // ---- this CTA's share of the exact sum of g_max ----
    if (warp == 5 && lane < kWindows) {
        const u64 v = s_acc[lane];
        if (v) atomicAdd(reinterpret_cast<u64 *>(a.packed + geo.ctl_at) + lane, v);
    }
}

// ---------------------------------------------------------------------------------
// tile_pass, any L_T: a warp per bin, lanes strided over the bin's elements.
// Dynamic shared memory: dW[tile_elems], G[tile_elems], words[tile_elems],
// gmax[tile_bins], cnt[tile_bins + 1].
// ---------------------------------------------------------------------------------

template <typename Word>
__global__ void __launch_bounds__(kGenericThreads)
tile_pass_generic(PassArgs a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ u32 s_tmp[33];
    __shared__ u64 s_acc[kWindows + 1];

    const Geometry &geo = a.geo;
    const int T = (int)geo.tile_elems, TB = (int)geo.tile_bins, L = (int)geo.L_T;
    float *s_d = reinterpret_cast<float *>(smem_raw);
    float *s_g = s_d + T;
    Word *s_words = reinterpret_cast<Word *>(s_g + T);
    float *s_gmax = reinterpret_cast<float *>(smem_raw + align_up((u64)T * (8 + sizeof(Word)), 16));
    u32 *s_cnt = reinterpret_cast<u32 *>(s_gmax + TB);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kGenericThreads / 32;
    u64 *tile_cnt = reinterpret_cast<u64 *>(a.packed + geo.tile_off_at);
    Word *bin_cnt = reinterpret_cast<Word *>(a.packed + geo.bin_cnt_at);

    if (tid < kWindows + 1) s_acc[tid] = 0;
    __syncthreads();

    for (u64 tile = blockIdx.x; tile < geo.n_tiles; tile += gridDim.x) {
        const u64 base = tile * (u64)T;
        const u64 left = geo.n - base;
        const int elems = left < (u64)T ? (int)left : T;

        for (int i = tid; i < T; i += kGenericThreads) {
            float d = 0.f, r = 0.f;
            if (i < elems) { d = a.grad[base + i]; r = a.residue[base + i]; }
            s_d[i] = d;
            s_g[i] = __fadd_rn(r, d);
        }
        __syncthreads();

        // bin maxima and per-bin counts
        for (int b = warp; b < TB; b += nwarp) {
            float m = 0.f;
            for (int j = lane; j < L; j += 32) m = fmaxf(m, fabsf(s_g[b * L + j]));
            for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
            u32 count = 0;
            if (m > 0.f) {
                for (int j0 = 0; j0 < L; j0 += 32) {
                    const int j = j0 + lane;
                    bool sel = false;
                    if (j < L) {
                        const float g = s_g[b * L + j];
                        const float h = __fadd_rn(g, s_d[b * L + j]);
                        sel = (g != 0.f) && (fabsf(h) >= m || (!a.literal && fabsf(g) == m));
                    }
                    count += __popc(__ballot_sync(0xffffffffu, sel));
                }
            }
            if (lane == 0) {
                s_gmax[b] = m;
                s_cnt[b] = count;
                const u64 bin = tile * (u64)TB + b;
                if (bin < geo.n_bins) {
                    bin_cnt[bin] = (Word)count;
                    u32 window;
                    u64 lo, hi;
                    if (split_for_sum(m, window, lo, hi)) {
                        atomicAdd(&s_acc[window], lo);
                        atomicAdd(&s_acc[window + 1], hi);
                    }
                }
            }
        }
        __syncthreads();
        block_exclusive_scan(s_cnt, TB, s_tmp);

        // words, in ascending order inside each bin
        for (int b = warp; b < TB; b += nwarp) {
            const float m = s_gmax[b];
            if (!(m > 0.f)) continue;
            u32 at = s_cnt[b];
            for (int j0 = 0; j0 < L; j0 += 32) {
                const int j = j0 + lane;
                bool sel = false;
                float g = 0.f;
                if (j < L) {
                    g = s_g[b * L + j];
                    const float h = __fadd_rn(g, s_d[b * L + j]);
                    sel = (g != 0.f) && (fabsf(h) >= m || (!a.literal && fabsf(g) == m));
                }
                const u32 mask = __ballot_sync(0xffffffffu, sel);
                if (sel) {
                    const u32 pos = at + __popc(mask & ((1u << lane) - 1u));
                    s_words[pos] = (Word)(((u32)j << 2) | (g < 0.f ? 3u : 1u));
                }
                at += __popc(mask);
            }
        }
        __syncthreads();

        for (int i = tid; i < elems; i += kGenericThreads) a.residue[base + i] = s_g[i];
        const u32 total = s_cnt[TB];
        Word *slot = reinterpret_cast<Word *>(a.packed + geo.slots_at + tile * geo.slot_bytes);
        for (u32 i = tid; i < total; i += kGenericThreads) slot[i] = s_words[i];
        if (tid == 0) tile_cnt[tile + 1] = total;
        __syncthreads();
    }

    if (tid < kWindows) {
        const u64 v = s_acc[tid];
        if (v) atomicAdd(reinterpret_cast<u64 *>(a.packed + geo.ctl_at) + tid, v);
    }
}

// ---------------------------------------------------------------------------------
// finalize: one CTA.  Exact sum -> scale; tile counts -> exclusive scan; header.
// ---------------------------------------------------------------------------------

// The nine windows hold the exact sum of the bin maxima in units of 2^-149.  Returns the
// double nearest to it (ties to even).
__device__ double windows_to_double(const u64 *win)
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

__global__ void __launch_bounds__(1024)
finalize(unsigned char *packed, Geometry geo, u32 flags, u64 *count_out)
{
    __shared__ u64 s_warp[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);

    // in-place exclusive scan of the tile counts held in tile_off[1 .. n_tiles]
    const u64 per = (geo.n_tiles + 1023) / 1024;
    const u64 lo = min((u64)tid * per, geo.n_tiles), hi = min(lo + per, geo.n_tiles);
    u64 sum = 0;
    for (u64 i = lo; i < hi; i++) sum += tile_off[i + 1];
    u64 inc = sum;
    for (int d = 1; d < 32; d <<= 1) {
        u64 t = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += t;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        u64 v = s_warp[lane], s = v;
        for (int d = 1; d < 32; d <<= 1) {
            u64 t = __shfl_up_sync(0xffffffffu, s, d);
            if (lane >= d) s += t;
        }
        s_warp[lane] = s - v;
        if (lane == 31) s_warp[32] = s;
    }
    __syncthreads();
    u64 run = s_warp[warp] + inc - sum;      // words before this thread's first tile
    // entry i+1 must become the count of words before tile i+1 = run + count(tile i)
    for (u64 i = lo; i < hi; i++) {
        const u64 c = tile_off[i + 1];
        run += c;
        tile_off[i + 1] = run;
    }
    const u64 n_sel = s_warp[32];

    if (tid == 0) {
        tile_off[0] = 0;
        const u64 *win = reinterpret_cast<const u64 *>(packed + geo.ctl_at);
        float scale = 0.f;
        if (geo.n_bins) {
            const double S = windows_to_double(win);
            scale = __double2float_rn(__ddiv_rn(S, (double)geo.n_bins));
        }
        const u64 bytes_used = geo.payload_at + align_up(n_sel * geo.w, 16);
        u32 *h32 = reinterpret_cast<u32 *>(packed);
        u64 *h64 = reinterpret_cast<u64 *>(packed);
        h32[0] = kMagic;
        h32[1] = 1u | (geo.w << 16) | ((flags & ADACOMP_FLAG_LITERAL) << 24);
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
    // zero padding behind the last word, and the alignment gaps of the directory sections
    const u64 pay_end = geo.payload_at + n_sel * geo.w;
    const u64 pad = align_up(pay_end, 16) - pay_end;
    if ((u64)tid < pad) packed[pay_end + tid] = 0;
    const u64 dir_end = geo.tile_off_at + 8 * (geo.n_tiles + 1);
    if ((u64)tid < geo.bin_cnt_at - dir_end) packed[dir_end + tid] = 0;
    const u64 cnt_end = geo.bin_cnt_at + geo.n_bins * geo.w;
    if ((u64)tid < geo.payload_at - cnt_end) packed[cnt_end + tid] = 0;
}

// ---------------------------------------------------------------------------------
// gather_fixup: per tile, copy the slot's words to the payload and finish the residue
// of the sent elements: residue = G - sign(G) * scale  (Algorithm 2, the "if" branch).
// ---------------------------------------------------------------------------------

template <typename Word>
__global__ void __launch_bounds__(kGatherThreads)
gather_fixup(float *residue, unsigned char *packed, Geometry geo)
{
    __shared__ u32 s_pre[kMaxTileBins + 1];
    __shared__ u32 s_tmp[33];
    const int tid = threadIdx.x;
    const int TB = (int)geo.tile_bins;
    const u64 *tile_off = reinterpret_cast<const u64 *>(packed + geo.tile_off_at);
    const Word *bin_cnt = reinterpret_cast<const Word *>(packed + geo.bin_cnt_at);
    Word *payload = reinterpret_cast<Word *>(packed + geo.payload_at);
    const float scale = __uint_as_float(reinterpret_cast<const u32 *>(packed)[12]);

    for (u64 tile = blockIdx.x; tile < geo.n_tiles; tile += gridDim.x) {
        const u64 off0 = tile_off[tile];
        const u32 cnt = (u32)(tile_off[tile + 1] - off0);
        if (cnt == 0) continue;
        const u64 bin0 = tile * (u64)TB;
        for (int b = tid; b < TB; b += kGatherThreads)
            s_pre[b] = bin0 + b < geo.n_bins ? (u32)bin_cnt[bin0 + b] : 0u;
        __syncthreads();
        block_exclusive_scan(s_pre, TB, s_tmp);
        const Word *slot = reinterpret_cast<const Word *>(packed + geo.slots_at + tile * geo.slot_bytes);
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

// ---------------------------------------------------------------------------------
// decode_sum: unpack() of k streams and their ordered sum, one output chunk per CTA pass.
// ---------------------------------------------------------------------------------

struct DecodeArgs {
    const unsigned char *stream[ADACOMP_MAX_STREAMS];
    float *dst;
    u32 k;
};

template <typename Word>
__device__ void decode_items(const DecodeArgs &a, const Geometry &geo, float *s_acc, u32 *s_pre,
                             u32 *s_tmp)
{
    const int tid = threadIdx.x;
    const int TB = (int)geo.tile_bins;
    const u32 chunks_per_tile = (geo.tile_elems + kDecodeChunk - 1) / kDecodeChunk;
    const u64 items = geo.n_tiles * chunks_per_tile;
    for (u64 item = blockIdx.x; item < items; item += gridDim.x) {
        const u64 tile = item / chunks_per_tile;
        const u32 c_lo = (u32)(item % chunks_per_tile) * kDecodeChunk;     // within the tile
        const u32 c_hi = min(c_lo + (u32)kDecodeChunk, geo.tile_elems);
        const u64 base = tile * (u64)geo.tile_elems;
        for (int i = tid; i < kDecodeChunk; i += kDecodeThreads) s_acc[i] = 0.f;
        __syncthreads();
        for (u32 l = 0; l < a.k; l++) {
            const unsigned char *s = a.stream[l];
            const u64 *tile_off = reinterpret_cast<const u64 *>(s + geo.tile_off_at);
            const u64 off0 = tile_off[tile];
            const u32 cnt = (u32)(tile_off[tile + 1] - off0);
            if (cnt == 0) continue;
            if (cnt > geo.tile_elems) { if (tid == 0) raise_status(ADACOMP_DEV_BAD_STREAM); continue; }
            const float scale = __uint_as_float(reinterpret_cast<const u32 *>(s)[12]);
            const Word *bin_cnt = reinterpret_cast<const Word *>(s + geo.bin_cnt_at);
            const Word *payload = reinterpret_cast<const Word *>(s + geo.payload_at);
            const u64 bin0 = tile * (u64)TB;
            int b_fixed = 0;
            if (TB > 1) {
                for (int b = tid; b < TB; b += kDecodeThreads)
                    s_pre[b] = bin0 + b < geo.n_bins ? (u32)bin_cnt[bin0 + b] : 0u;
                __syncthreads();
                block_exclusive_scan(s_pre, TB, s_tmp);
                if (s_pre[TB] != cnt) { if (tid == 0) raise_status(ADACOMP_DEV_BAD_STREAM); __syncthreads(); continue; }
            }
            for (u32 j = tid; j < cnt; j += kDecodeThreads) {
                const u32 word = payload[off0 + j];
                const u32 code = word & 3u;
                if (code == 0u) continue;
                if (code == 2u) { raise_status(ADACOMP_DEV_RESERVED_CODE); continue; }
                const int b = TB > 1 ? bin_of_word(s_pre, TB, j) : b_fixed;
                const u32 idx = word >> 2;
                const u32 at = (u32)b * geo.L_T + idx;          // within the tile
                if (idx >= geo.L_T || base + at >= geo.n) { raise_status(ADACOMP_DEV_BAD_STREAM); continue; }
                if (at < c_lo || at >= c_hi) continue;
                // one word per element per learner: no two threads meet on one address here
                const float v = s_acc[at - c_lo];
                s_acc[at - c_lo] = code == 3u ? __fsub_rn(v, scale) : __fadd_rn(v, scale);
            }
            __syncthreads();
        }
        const u64 out0 = base + c_lo;
        const u32 len = out0 < geo.n ? (u32)min((u64)(c_hi - c_lo), geo.n - out0) : 0u;
        if ((out0 & 3u) == 0) {
            float4 *o4 = reinterpret_cast<float4 *>(a.dst + out0);
            for (u32 i = tid; i < len / 4; i += kDecodeThreads)
                __stcs(o4 + i, reinterpret_cast<float4 *>(s_acc)[i]);
            for (u32 i = (len & ~3u) + tid; i < len; i += kDecodeThreads) a.dst[out0 + i] = s_acc[i];
        } else {
            for (u32 i = tid; i < len; i += kDecodeThreads) a.dst[out0 + i] = s_acc[i];
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kDecodeThreads)
decode_sum(DecodeArgs a)
{
    __shared__ __align__(16) float s_acc[kDecodeChunk];
    __shared__ u32 s_pre[kMaxTileBins + 1];
    __shared__ u32 s_tmp[33];
    __shared__ int s_bad;

    // every CTA reads and cross-checks the k headers itself: the decision is uniform
    const u32 *h0 = reinterpret_cast<const u32 *>(a.stream[0]);
    const u32 L_T = h0[2];
    const u64 n = reinterpret_cast<const u64 *>(a.stream[0])[2];
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    if (threadIdx.x < a.k) {
        const u32 *h = reinterpret_cast<const u32 *>(a.stream[threadIdx.x]);
        const u64 *h64 = reinterpret_cast<const u64 *>(h);
        bool ok = h[0] == kMagic && (h[1] & 0xffffu) == 1u && h[2] == L_T && h64[2] == n &&
                  L_T >= 1u && L_T <= ADACOMP_MAX_L_T;
        if (ok) {
            const Geometry g = make_geometry(n, L_T);
            ok = ((h[1] >> 16) & 0xffu) == g.w && h[3] == g.tile_bins && h64[3] == g.n_bins &&
                 h64[4] == g.n_tiles;
        }
        if (!ok) s_bad = 1;
    }
    __syncthreads();
    if (s_bad) {
        if (threadIdx.x == 0 && blockIdx.x == 0) raise_status(ADACOMP_DEV_HEADER_MISMATCH);
        return;
    }
    const Geometry geo = make_geometry(n, L_T);
    if (geo.w == 1u) decode_items<unsigned char>(a, geo, s_acc, s_pre, s_tmp);
    else decode_items<unsigned short>(a, geo, s_acc, s_pre, s_tmp);
}

__global__ void reset_status_kernel() { g_status = 0; }

// ---------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
};

DeviceInfo g_info[64];

int device_info(DeviceInfo &out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ADACOMP_ERR_CUDA;
    if (g_info[dev].sms == 0) {
        int sms = 0, optin = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return ADACOMP_ERR_CUDA;
        g_info[dev].smem_optin = optin;
        g_info[dev].sms = sms;
    }
    out = g_info[dev];
    return ADACOMP_OK;
}

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

template <typename Word>
int launch_generic(const PassArgs &args, const DeviceInfo &info, cudaStream_t st)
{
    const Geometry &geo = args.geo;
    const size_t smem = (size_t)align_up((u64)geo.tile_elems * (8 + sizeof(Word)), 16) +
                        (size_t)geo.tile_bins * 4 + ((size_t)geo.tile_bins + 1) * 4;
    if (smem > (size_t)info.smem_optin) return ADACOMP_ERR_SIZE;
    if (cudaFuncSetAttribute(tile_pass_generic<Word>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tile_pass_generic<Word>, kGenericThreads, smem);
    if (per_sm < 1) per_sm = 1;
    const u64 grid = geo.n_tiles < (u64)info.sms * per_sm ? geo.n_tiles : (u64)info.sms * per_sm;
    tile_pass_generic<Word><<<(unsigned)grid, kGenericThreads, smem, st>>>(args);
    return ADACOMP_OK;
}

int compress_impl(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                  uint64_t *count_out, void *stream, uint32_t flags, void *const *events = nullptr)
{
    if (!packed_out || !count_out || (n && (!grad || !residue))) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH)) return ADACOMP_ERR_FLAGS;
    if (misaligned(grad) || misaligned(residue) || misaligned(packed_out) ||
        (reinterpret_cast<uintptr_t>(count_out) & 7u))
        return ADACOMP_ERR_ALIGN;
    const Geometry geo = make_geometry(n, L_T);
    if (geo.n_bins >= (1ull << 31)) return ADACOMP_ERR_SIZE;

    DeviceInfo info;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *packed = static_cast<unsigned char *>(packed_out);

    if (cudaMemsetAsync(packed + geo.ctl_at, 0, kCtlBytes, st) != cudaSuccess) return ADACOMP_ERR_CUDA;
    auto mark = [&](int i) { if (events) cudaEventRecord(static_cast<cudaEvent_t>(events[i]), st); };

    mark(0);
    if (geo.n_tiles) {
        PassArgs args{grad, residue, packed, geo, flags & ADACOMP_FLAG_LITERAL};
        const bool fast = (L_T == 50u || L_T == 500u) && !(flags & ADACOMP_FLAG_GENERIC_PATH);
        if (fast) {
            int per_sm = 1;
            if (L_T == 50u)
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tile_pass_fast<2, unsigned char>, kFastThreads, 0);
            else
                cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, tile_pass_fast<20, unsigned short>, kFastThreads, 0);
            if (per_sm < 1) per_sm = 1;
            const u64 cap = (u64)info.sms * per_sm;
            const unsigned grid = (unsigned)(geo.n_tiles < cap ? geo.n_tiles : cap);
            if (L_T == 50u) tile_pass_fast<2, unsigned char><<<grid, kFastThreads, 0, st>>>(args);
            else tile_pass_fast<20, unsigned short><<<grid, kFastThreads, 0, st>>>(args);
        } else {
            rc = geo.w == 1u ? launch_generic<unsigned char>(args, info, st)
                             : launch_generic<unsigned short>(args, info, st);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    mark(1);
    finalize<<<1, 1024, 0, st>>>(packed, geo, flags, reinterpret_cast<u64 *>(count_out));
    mark(2);
    if (geo.n_tiles) {
        const u64 cap = (u64)info.sms * 8;
        const unsigned grid = (unsigned)(geo.n_tiles < cap ? geo.n_tiles : cap);
        if (geo.w == 1u) gather_fixup<unsigned char><<<grid, kGatherThreads, 0, st>>>(residue, packed, geo);
        else gather_fixup<unsigned short><<<grid, kGatherThreads, 0, st>>>(residue, packed, geo);
    }
    mark(3);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int decompress_impl(const void *const *packed, uint32_t k, float *dst, void *stream)
{
    if (!packed || !dst) return ADACOMP_ERR_NULL;
    if (k == 0 || k > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    DecodeArgs args;
    for (uint32_t l = 0; l < ADACOMP_MAX_STREAMS; l++) args.stream[l] = nullptr;
    for (uint32_t l = 0; l < k; l++) {
        if (!packed[l]) return ADACOMP_ERR_NULL;
        if (misaligned(packed[l])) return ADACOMP_ERR_ALIGN;
        args.stream[l] = static_cast<const unsigned char *>(packed[l]);
    }
    if (misaligned(dst)) return ADACOMP_ERR_ALIGN;
    args.dst = dst;
    args.k = k;
    DeviceInfo info;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum, kDecodeThreads, 0);
    if (per_sm < 1) per_sm = 1;
    decode_sum<<<(unsigned)(info.sms * per_sm), kDecodeThreads, 0, static_cast<cudaStream_t>(stream)>>>(args);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

}  // namespace

// ---------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------

extern "C" {

int adacomp_version(void) { return ADACOMP_VERSION; }

const char *adacomp_strerror(int code)
{
    switch (code) {
    case ADACOMP_OK: return "ok";
    case ADACOMP_ERR_NULL: return "a required pointer is NULL";
    case ADACOMP_ERR_L_T: return "L_T must be in 1..16384";
    case ADACOMP_ERR_ALIGN: return "a buffer is not 16-byte aligned";
    case ADACOMP_ERR_STREAMS: return "k_streams must be in 1..64";
    case ADACOMP_ERR_SIZE: return "tensor too large for this bin length";
    case ADACOMP_ERR_FLAGS: return "unknown flag bits";
    case ADACOMP_ERR_CUDA: return "a CUDA runtime call failed";
    default: return "unknown error code";
    }
}

size_t adacomp_packed_capacity(uint64_t n, uint32_t L_T)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return 0;
    return (size_t)make_geometry(n, L_T).capacity;
}

int adacomp_compress(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                     uint64_t *count_out, void *stream)
{
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0);
}

int adacomp_compress_ex(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                        uint64_t *count_out, void *stream, uint32_t flags)
{
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, flags);
}

int adacomp_decompress_accumulate(const void *const *packed, uint32_t k_streams, float *dst, void *stream)
{
    return decompress_impl(packed, k_streams, dst, stream);
}

int adacomp_compress_profile(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                             uint64_t *count_out, void *stream, uint32_t flags, void *const *events)
{
    if (!events) return ADACOMP_ERR_NULL;
    for (int i = 0; i < 4; i++)
        if (!events[i]) return ADACOMP_ERR_NULL;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, flags, events);
}

int adacomp_compress_host(const float *grad_host, float *grad_stage, float *residue, uint64_t n, uint32_t L_T,
                          void *packed_dev, uint64_t *count_dev, void *packed_host, uint64_t packed_host_cap,
                          uint64_t *count_host, void *stream)
{
    if (!count_host || !packed_host || (n && (!grad_host || !grad_stage))) return ADACOMP_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n && cudaMemcpyAsync(grad_stage, grad_host, n * sizeof(float), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    int rc = compress_impl(grad_stage, residue, n, L_T, packed_dev, count_dev, stream, 0);
    if (rc != ADACOMP_OK) return rc;
    if (cudaMemcpyAsync(count_host, count_dev, 2 * sizeof(uint64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    if (count_host[1] > packed_host_cap) return ADACOMP_ERR_SIZE;
    if (cudaMemcpyAsync(packed_host, packed_dev, count_host[1], cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    return ADACOMP_OK;
}

int adacomp_decompress_accumulate_host(const void *const *packed_host, const uint64_t *packed_bytes,
                                       void *const *packed_stage, uint32_t k_streams, float *dst_dev,
                                       float *dst_host, uint64_t n, void *stream)
{
    if (!packed_host || !packed_bytes || !packed_stage || !dst_dev || (n && !dst_host)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (uint32_t l = 0; l < k_streams; l++) {
        if (!packed_host[l] || !packed_stage[l]) return ADACOMP_ERR_NULL;
        if (cudaMemcpyAsync(packed_stage[l], packed_host[l], packed_bytes[l], cudaMemcpyHostToDevice, st) != cudaSuccess)
            return ADACOMP_ERR_CUDA;
    }
    int rc = decompress_impl(packed_stage, k_streams, dst_dev, stream);
    if (rc != ADACOMP_OK) return rc;
    if (n && cudaMemcpyAsync(dst_host, dst_dev, n * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int adacomp_compress_multi(const adacomp_layer_desc *layers, uint32_t n_layers, void *stream)
{
    if (n_layers && !layers) return ADACOMP_ERR_NULL;
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        if (!d.packed_out || !d.count_out || (d.n && (!d.grad || !d.residue))) return ADACOMP_ERR_NULL;
        if (d.L_T == 0 || d.L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
        if (d.flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH)) return ADACOMP_ERR_FLAGS;
        if (misaligned(d.grad) || misaligned(d.residue) || misaligned(d.packed_out)) return ADACOMP_ERR_ALIGN;
    }
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        int rc = compress_impl(d.grad, d.residue, d.n, d.L_T, d.packed_out, d.count_out, stream, d.flags);
        if (rc != ADACOMP_OK) return rc;
    }
    return ADACOMP_OK;
}

int adacomp_decompress_accumulate_multi(const void *const *packed, uint32_t k_streams, float *const *dst,
                                        uint32_t n_layers, void *stream)
{
    if (n_layers && (!packed || !dst)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    for (uint32_t t = 0; t < n_layers; t++) {
        int rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, dst[t], stream);
        if (rc != ADACOMP_OK) return rc;
    }
    return ADACOMP_OK;
}

int adacomp_device_status(uint32_t *host_out, void *stream)
{
    if (!host_out) return ADACOMP_ERR_NULL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ADACOMP_ERR_CUDA;
    u32 v = 0;
    if (cudaMemcpyFromSymbol(&v, g_status, sizeof(v)) != cudaSuccess) return ADACOMP_ERR_CUDA;
    *host_out = v;
    return ADACOMP_OK;
}

int adacomp_device_status_reset(void *stream)
{
    reset_status_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>();
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

}  // extern "C"
