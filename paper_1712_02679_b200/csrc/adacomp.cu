// libadacomp: AdaComp pack() / unpack()-and-sum for one B200 (sm_100a).
//
// pack() (Algorithm 2 of the paper) runs as three kernels on the caller's stream:
//   tile_pass     one read of dW and residue, one write of residue (= G everywhere);
//                 per-bin max |G|, selection, words compacted per tile into a scratch
//                 slot, per-bin counts, per-tile counts, exact partial sums of g_max
//   finalize      exact sum -> scale, scan of the tile-group counts, header, count_out
//   gather_fixup  moves each tile's words to their final place, writes the tile
//                 directory, and subtracts sign * scale from the residue of the sent
//                 elements only
// The layer-wide scale (Section 2.5: mean of the g_max vector) is needed by every
// sent element's residue but is known only after every bin has been seen; that is
// why the residue of sent elements is finished by the third kernel.
//
// unpack()-and-sum is one kernel: each CTA owns an output tile in shared memory,
// adds the k learners' words into it in learner order and stores it once.
//
// HBM-bandwidth bound; no tensor cores (nothing here is a contraction).  The fast
// tile pass (every L_T from 41 to 1000, the paper's 50 and 500 among them) is a persistent
// kernel fed by 1-D bulk copies (TMA) through a three-stage shared-memory ring guarded by
// mbarriers, and so is the decoder (every L_T from 41 up) with its ring of slots; every wait
// on a barrier is bounded and reports ADACOMP_DEV_TIMEOUT instead of spinning forever.

#include <cuda_runtime.h>
#include <stdint.h>

#include "adacomp.h"

namespace {

typedef unsigned long long u64;
typedef unsigned int u32;

constexpr u32 kMagic = 0x31434441u;
constexpr u32 kFlagFactor = 2u;       // header flag (set by the library): the stream was made with a scale-factor
constexpr u32 kHeaderBytes = 64;
constexpr u32 kCtlBytes = 256;       // control block at the start of the scratch area
constexpr int kWindows = 9;          // 32-bit windows of the exact g_max accumulator
constexpr int kGroupTiles = 32;      // tiles per group of the two-level count scan
constexpr int kSeg = 25;             // elements per thread on the fast path
constexpr int kTileSegs = 160;       // segments per tile on the fast path
constexpr int kFastTile = kSeg * kTileSegs;   // 4000 elements
constexpr int kFastThreads = 192;    // 5 compute warps + 1 service warp
constexpr int kStages = 3;
constexpr u32 kTileBytes = kFastTile * 4;     // 16000
constexpr u32 kMaskBytes = kTileSegs * 4;      // lazy mode: one 25-bit "sent" mask per segment
constexpr u32 kStageBytes = 2 * kTileBytes + kMaskBytes;   // dW + residue + previous step's masks
constexpr int kGenericThreads = 256;
constexpr int kDecodeChunk = 4096;   // output elements per decode work item
constexpr int kDecodeThreads = 128;  // decoding threads of a decode CTA (warps 0-3)
constexpr int kDecodeLaunch = 160;   // launched threads: warp 4 is the pipelined path's producer
constexpr int kGatherThreads = 128;
constexpr int kMaxTileBins = 4000;
constexpr int kSmallBins = 96;       // tiles with at most this many bins take the fast decode / gather
constexpr long long kWaitCycles = 4000000000ll;   // ~2 s: bound of every device-side wait

__device__ u32 g_status;             // sticky ADACOMP_DEV_* bits of this device

__host__ __device__ inline u64 align_up(u64 x, u64 a) { return (x + a - 1) / a * a; }

// Section offsets of a packed stream and of the scratch behind it.
struct Geometry {
    u32 w, L_T, tile_bins, tile_elems;
    u64 n, n_bins, n_tiles, n_groups;
    u64 tile_off_at, bin_cnt_at, payload_at;              // the stream, offsets in the packed buffer
    u64 group_at, tile_cnt_at, slots_at, slot_bytes;      // the scratch, offsets from its base
    u64 scratch_bytes;                                    // (the control block sits at offset 0)
    u64 scratch_at, capacity;     // where the scratch starts when it follows the stream in one buffer
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
    g.n_groups = (g.n_tiles + kGroupTiles - 1) / kGroupTiles;
    g.tile_off_at = kHeaderBytes;
    g.bin_cnt_at = align_up(g.tile_off_at + 8 * (g.n_tiles + 1), 16);
    g.payload_at = align_up(g.bin_cnt_at + g.n_bins * g.w, 16);
    g.group_at = kCtlBytes;                                    // u64[n_groups], zeroed per call
    g.tile_cnt_at = g.group_at + 8 * g.n_groups;               // u32[n_tiles]
    g.slots_at = align_up(g.tile_cnt_at + 4 * g.n_tiles, 256);
    g.slot_bytes = align_up((u64)g.tile_elems * g.w, 16);
    g.scratch_bytes = g.slots_at + g.n_tiles * g.slot_bytes;
    g.scratch_at = align_up(g.payload_at + align_up(n * g.w, 16), 256);
    g.capacity = g.scratch_at + g.scratch_bytes;
    return g;
}

// ---------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------

__device__ inline void raise_status(u32 bits) { atomicOr(&g_status, bits); }

// Element i of a gradient that is binary32, or bfloat16 widened exactly (sixteen zero bits appended).
__device__ inline float load_grad(const float *grad, u64 i, u32 bf16)
{
    return bf16 ? __uint_as_float((u32)reinterpret_cast<const unsigned short *>(grad)[i] << 16) : grad[i];
}

__device__ inline u32 warp_inclusive_scan(u32 v, int lane)
{
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const u32 t = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += t;
    }
    return v;
}

// Exclusive scan, in place, of a[0..count) in shared memory; a[count] receives the total.
// Called by every thread of the CTA; contains barriers.
// With `decoders` set it is called by the 128 decoding threads of a decode CTA only and meets at
// their named barrier.
__device__ inline void block_exclusive_scan(u32 *a, int count, u32 *warp_tmp /* >= 33 */, bool decoders = false)
{
    auto sync = [&]() {
        if (decoders) asm volatile("bar.sync 1, 128;" ::: "memory");
        else __syncthreads();
    };
    const int tid = threadIdx.x, nthr = decoders ? 128 : (int)blockDim.x;
    const int per = (count + nthr - 1) / nthr;
    const int lo = min(tid * per, count), hi = min(lo + per, count);
    u32 sum = 0;
    for (int i = lo; i < hi; i++) sum += a[i];
    const int lane = tid & 31, warp = tid >> 5, nwarp = (nthr + 31) >> 5;
    const u32 inc = warp_inclusive_scan(sum, lane);
    if (lane == 31) warp_tmp[warp] = inc;
    sync();
    if (warp == 0) {
        const u32 v = lane < nwarp ? warp_tmp[lane] : 0u;
        const u32 s = warp_inclusive_scan(v, lane);
        warp_tmp[lane] = s - v;
        if (lane == 31) warp_tmp[32] = s;
    }
    sync();
    u32 run = warp_tmp[warp] + inc - sum;
    for (int i = lo; i < hi; i++) {
        const u32 v = a[i];
        a[i] = run;
        run += v;
    }
    if (tid == 0) a[count] = warp_tmp[32];
    sync();
}

// Barrier of the 128 decoding threads of a decode CTA (its producer warp never joins).
__device__ inline void consumer_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Largest b in [0, bins) with prefix[b] <= j  (prefix is an exclusive scan, prefix[bins] > j).
__device__ inline int bin_of_word(const u32 *prefix, int bins, u32 j)
{
    int lo = 0, hi = bins;           // invariant: prefix[lo] <= j < prefix[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
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

// ---- mbarrier / bulk-copy (TMA) wrappers; no cluster multicast anywhere ----

__device__ inline u32 smem_addr(const void *p) { return (u32)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(u64 *bar, u32 arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
}

__device__ inline void mbar_arrive_expect_tx(u64 *bar, u32 bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}

__device__ inline bool mbar_try_wait(u64 *bar, u32 parity)
{
    u32 ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ inline void mbar_arrive(u64 *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Bounded wait: false if the phase did not complete within kWaitCycles.
__device__ inline bool mbar_wait(u64 *bar, u32 parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > kWaitCycles) return false;
    }
    return true;
}

__device__ inline void bulk_load(void *smem_dst, const void *gmem_src, u32 bytes, u64 *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
                     "r"(smem_addr(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

__device__ inline void bulk_store(void *gmem_dst, const void *smem_src, u32 bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
                 "r"(smem_addr(smem_src)), "r"(bytes)
                 : "memory");
}

__device__ inline void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ inline void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ inline void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ inline void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

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

struct TrueType { static constexpr bool value = true; };
struct FalseType { static constexpr bool value = false; };

struct PassArgs {
    const float *grad;
    float *residue;
    unsigned char *packed;      // the stream under construction
    unsigned char *scratch;     // control block, group counts, tile counts, word slots
    Geometry geo;
    u32 literal;
    unsigned char *lazy_state;  // lazy mode: header + per-segment masks of the elements sent last step
    float factor;               // 0: H = G + dW (Algorithm 2); else H = residue + factor * dW (Section 2.4's scale-factor)
    u32 grad_bf16;              // `grad` points to bfloat16 values (widened exactly on load)
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

struct FastSmem {
    static constexpr u32 kWordsAt = kStages * kStageBytes;            // 96000
    static constexpr u32 kInclAt = kWordsAt + 2 * kFastTile;          // + 8000 (16-bit words)
    static constexpr u32 kWtotAt = kInclAt + 4 * kTileSegs;
    static constexpr u32 kSegmaxAt = kWtotAt + 4 * 8;
    static constexpr u32 kBinmaxAt = kSegmaxAt + 4 * kTileSegs;
    static constexpr u32 kAccAt = kBinmaxAt + 4 * 4 * kSmallBins;     // (SPB = 0: two buffers each of bin maxima and counts) 8-byte aligned
    static constexpr u32 kBarAt = kAccAt + 8 * (kWindows + 1);
    static constexpr u32 kAbortAt = kBarAt + 8 * kStages;
    static constexpr u32 kBytes = kAbortAt + 16;
};
static_assert(FastSmem::kAccAt % 8 == 0, "accumulator must be 8-byte aligned");

// BF16: the gradient arrives as bfloat16 (8000-byte tiles, widened as they are read).
template <int SPB, typename Word, bool LAZY, bool BF16 = false>
__global__ void __launch_bounds__(kFastThreads, 2)
tile_pass_fast(PassArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    Word *s_words = reinterpret_cast<Word *>(smem + FastSmem::kWordsAt);
    u32 *s_incl = reinterpret_cast<u32 *>(smem + FastSmem::kInclAt);
    u32 *s_wtot = reinterpret_cast<u32 *>(smem + FastSmem::kWtotAt);
    float *s_segmax = reinterpret_cast<float *>(smem + FastSmem::kSegmaxAt);
    float *s_binmax = reinterpret_cast<float *>(smem + FastSmem::kBinmaxAt);
    u64 *s_acc = reinterpret_cast<u64 *>(smem + FastSmem::kAccAt);
    u64 *s_full = reinterpret_cast<u64 *>(smem + FastSmem::kBarAt);
    volatile u32 *s_abort = reinterpret_cast<volatile u32 *>(smem + FastSmem::kAbortAt);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const Geometry &geo = a.geo;
    constexpr bool ANY = SPB == 0;
    static_assert(!ANY || !BF16, "the any-L_T form takes fp32 gradients");
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

    if (tid < kWindows + 1) s_acc[tid] = 0;
    if (ANY)
        for (int b = tid; b < 4 * kSmallBins; b += kFastThreads) s_anymax[b] = 0;
    if (tid == 0) {
        *s_abort = 0;
        for (int s = 0; s < kStages; s++) mbar_init(&s_full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    u64 issued = 0;                     // service lane 0: loads issued for tiles [0, issued)
    auto issue_load = [&](u64 i) {
        const u64 tile = first + i * stride;
        if (i >= my_tiles || tile >= full_tiles) return;
        unsigned char *st = smem + (i % kStages) * kStageBytes;
        u64 *bar = &s_full[i % kStages];
        const u32 grad_bytes = BF16 ? kTileBytes / 2 : tile_bytes;
        mbar_arrive_expect_tx(bar, grad_bytes + tile_bytes + (LAZY ? kMaskBytes : 0u));
        bulk_load(st, reinterpret_cast<const unsigned char *>(a.grad) + tile * (u64)grad_bytes, grad_bytes, bar);
        bulk_load(st + kTileBytes, a.residue + tile * (u64)T, tile_bytes, bar);
        if (LAZY) bulk_load(st + 2 * kTileBytes, lazy_mask + tile * (u64)kTileSegs, kMaskBytes, bar);
        issued = i + 1;
    };
    if (service && lane == 0) {
        issue_load(0);
        issue_load(1);
    }

    u64 i = 0;
    for (; i < my_tiles; i++) {
        const u64 tile = first + i * stride;
        const u64 base = tile * (u64)T;
        float *s_d = reinterpret_cast<float *>(smem + (i % kStages) * kStageBytes);
        float *s_r = s_d + kFastTile;
        const u32 *s_prev = reinterpret_cast<const u32 *>(s_r + kFastTile);
        const bool whole = tile < full_tiles;
        const int elems = whole ? T : (int)(geo.n - base);
        u32 *const any_max = s_anymax + (i & 1) * kSmallBins, *const any_cnt = s_anycnt + (i & 1) * kSmallBins;

        if (whole) {
            if (!mbar_wait(&s_full[i % kStages], (u32)(i / kStages) & 1u)) {
                *s_abort = 1;                      // every thread that times out says so
                raise_status(ADACOMP_DEV_TIMEOUT);
            }
        } else {
            // the ragged last tile of the tensor: plain loads, zero fill past the end
            for (int e = tid; e < kFastTile; e += kFastThreads) {
                float d = 0.f, r = 0.f;
                if (e < elems) { d = load_grad(a.grad, base + e, BF16); r = a.residue[base + e]; }
                if (BF16) reinterpret_cast<unsigned short *>(s_d)[e] = (unsigned short)(__float_as_uint(d) >> 16);
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
            // bfloat16: the segment's 50 bytes start on a 4-byte boundary for even threads and two bytes
            // past one for odd threads; thirteen aligned 32-bit loads cover them either way, and a funnel
            // shift by 0 or 16 bits lines the pairs up (half as many shared-memory accesses as 25 16-bit loads)
            u32 pair[BF16 ? 13 : 1];
            if (BF16) {
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
                float d = BF16 ? __uint_as_float((j & 1) ? pair[j >> 1] & 0xffff0000u : pair[j >> 1] << 16) : pd[j];
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
                for (u64 j = i + 1; j < issued; j++) mbar_wait(&s_full[j % kStages], (u32)(j / kStages) & 1u);
                for (u64 j = i; j < my_tiles; j++) tile_cnt[first + j * stride] = 0;
            }
        }
        if (lane < kWindows) {
            const u64 v = s_acc[lane];
            if (v) atomicAdd(reinterpret_cast<u64 *>(a.scratch) + lane, v);
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
    u32 grad_bf16;
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
    const int quads = (T & 3) == 0 && !a.grad_bf16 ? elems >> 2 : 0;
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
        if (i < elems) { d = load_grad(a.grad, base + i, a.grad_bf16); r = a.residue[base + i]; }
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
    const int quads = (base & 3u) == 0 && !a.grad_bf16 ? elems >> 2 : 0;
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
            k = key_of(a.residue[base + i], load_grad(a.grad, base + i, a.grad_bf16), g);
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
    __shared__ u64 s_acc[kWindows + 1];
    const int tid = threadIdx.x;
    if (tid < kWindows + 1) s_acc[tid] = 0;
    __syncthreads();
    const TileIo io{a.grad, a.residue, a.packed, a.scratch, a.literal, a.factor, a.grad_bf16};
    for (u64 tile = blockIdx.x; tile < a.geo.n_tiles; tile += gridDim.x) {
        if (a.geo.tile_bins == 1u && sizeof(Word) == 2) generic_tile_one_bin<Word>(io, a.geo, tile, smem_raw, s_tmp, s_acc);
        else generic_tile<Word>(io, a.geo, tile, smem_raw, s_tmp, s_acc);
    }
    if (tid < kWindows) {
        const u64 v = s_acc[tid];
        if (v) atomicAdd(reinterpret_cast<u64 *>(a.scratch) + tid, v);
    }
}

// ---------------------------------------------------------------------------------
// finalize: one CTA.  Exact sum -> scale; group counts -> exclusive scan; header.
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

__device__ void finalize_body(unsigned char *packed, unsigned char *scratch, const Geometry &geo, u32 flags,
                              u64 *count_out, unsigned char *lazy_state)
{
    __shared__ u64 s_warp[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    u64 *group = reinterpret_cast<u64 *>(scratch + geo.group_at);

    // in-place exclusive scan of the per-group word counts
    const u64 per = (geo.n_groups + 1023) / 1024;
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
        group[i] = run;
        run += c;
    }
    const u64 n_sel = s_warp[32];

    if (tid == 0) {
        u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);
        tile_off[geo.n_tiles] = n_sel;
        const u64 *win = reinterpret_cast<const u64 *>(scratch);
        float scale = 0.f;
        if (geo.n_bins) {
            const double S = windows_to_double(win);
            scale = __double2float_rn(__ddiv_rn(S, (double)geo.n_bins));
        }
        const u64 bytes_used = geo.payload_at + align_up(n_sel * geo.w, 16);
        u32 *h32 = reinterpret_cast<u32 *>(packed);
        u64 *h64 = reinterpret_cast<u64 *>(packed);
        h32[0] = kMagic;
        h32[1] = 1u | (geo.w << 16) | ((flags & (ADACOMP_FLAG_LITERAL | kFlagFactor)) << 24);
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
}

__global__ void __launch_bounds__(1024)
finalize(unsigned char *packed, unsigned char *scratch, Geometry geo, u32 flags, u64 *count_out,
         unsigned char *lazy_state)
{
    finalize_body(packed, scratch, geo, flags, count_out, lazy_state);
}

// ---------------------------------------------------------------------------------
// gather_fixup: per tile, copy the slot's words to the payload, write the tile's
// directory entry and finish the residue of the sent elements:
// residue = G - sign(G) * scale  (Algorithm 2, the "if" branch).
// ---------------------------------------------------------------------------------

// Words before `tile`: its group's scanned offset plus the counts of the tiles before it
// in the group.  Warp-collective; also returns the tile's own count.
__device__ inline u64 tile_offset(const unsigned char *scratch, const Geometry &geo, u64 tile, int lane,
                                  u32 &count)
{
    const u32 *tile_cnt = reinterpret_cast<const u32 *>(scratch + geo.tile_cnt_at);
    const u64 *group = reinterpret_cast<const u64 *>(scratch + geo.group_at);
    const u64 g = tile / kGroupTiles;
    const int me = (int)(tile % kGroupTiles);
    const u64 t = g * kGroupTiles + lane;
    const u32 c = t < geo.n_tiles ? tile_cnt[t] : 0u;
    u32 before = lane < me ? c : 0u;
    for (int d = 16; d > 0; d >>= 1) before += __shfl_xor_sync(0xffffffffu, before, d);
    count = min(__shfl_sync(0xffffffffu, c, me), geo.tile_elems);
    return group[g] + before;
}

// One tile of at most 96 bins, handled by one warp.
template <typename Word, bool FIXUP>
__device__ void gather_tile_small(float *residue, unsigned char *packed, const unsigned char *scratch,
                                  const Geometry &geo, u64 tile, int lane, u32 *s_pre)
{
    const int TB = (int)geo.tile_bins;
    u64 *tile_off = reinterpret_cast<u64 *>(packed + geo.tile_off_at);
    const Word *bin_cnt = reinterpret_cast<const Word *>(packed + geo.bin_cnt_at);
    Word *payload = reinterpret_cast<Word *>(packed + geo.payload_at);
    const float scale = __uint_as_float(reinterpret_cast<const u32 *>(packed)[12]);
    u32 cnt;
    const u64 off0 = tile_offset(scratch, geo, tile, lane, cnt);
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
    for (u32 j0 = 0; j0 < cnt; j0 += 128) {
        // four words per lane per round: their residue loads overlap
        u32 word[4];
        u64 pos[4];
        float g[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
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
        for (int q = 0; q < 4; q++) {
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

// ---------------------------------------------------------------------------------
// Batched pack(): many small layers in four launches instead of four launches per layer.
// The layer table travels in the kernel parameters; a global tile index runs over the tiles
// of all layers, and every CTA (tile pass) or warp (gather) looks its tile's layer up.
// Layers of 42 <= L_T <= 1000 (tiles of at most 4000 elements and 96 bins) qualify.
// ---------------------------------------------------------------------------------

constexpr int kBatchMax = 184;                       // layers per batched launch (the table is 32392 of the 32764 bytes of kernel parameters)
constexpr u64 kBatchLayerMaxElems = 1ull << 22;      // decode: larger layers take the single-layer kernels
// pack(): layers up to this size share a batch's launches when the pipelined batch tile pass is there (a
// layer alone ramps its pipeline up and down over a few tiles per CTA and pays four launches and a finalize
// of its own: below 2^24 elements it runs at under half the speed it has inside a batch)
constexpr u64 kPackBatchMaxElems = 1ull << 25;
constexpr u32 kBatchSmemBytes = 4000 * 10 + 4 * kSmallBins + 4 * (kSmallBins + 1) + 16;

struct BatchLayer {
    const float *grad;
    float *residue;
    unsigned char *packed;
    u64 *count_out;
    Geometry geo;
    u32 tile_first;                                  // global index of the layer's first tile
    u32 pad;
    unsigned char *lazy;                             // lazy-scale mode: the layer's state (else null)
};

// The table comes in two sizes: kernel parameters are copied at every launch, and a launch with the
// full 27 KB table costs several microseconds more than one with the small table.
constexpr int kBatchSmall = 16;

template <int N>
struct BatchArgsT {
    u32 n_layers, total_tiles;
    BatchLayer layer[N];
};
typedef BatchArgsT<kBatchMax> BatchArgs;

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
        const TileIo io{L.grad, L.residue, L.packed, L.packed + L.geo.scratch_at, 0u, 0.f, 0u};
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
template <int N, bool LAZY>
__global__ void __launch_bounds__(kFastThreads, 2)
batch_tile_pass_fast(const __grid_constant__ BatchArgsT<N> b)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *s_words = smem + FastSmem::kWordsAt;
    u32 *s_incl = reinterpret_cast<u32 *>(smem + FastSmem::kInclAt);
    u32 *s_wtot = reinterpret_cast<u32 *>(smem + FastSmem::kWtotAt);
    u32 *s_anymax = reinterpret_cast<u32 *>(smem + FastSmem::kBinmaxAt);    // [2][kSmallBins] bits of the bin maxima, by tile parity
    u32 *s_anycnt = s_anymax + 2 * kSmallBins;                               // [2][kSmallBins] words per bin
    u64 *s_acc = reinterpret_cast<u64 *>(smem + FastSmem::kAccAt);
    u64 *s_full = reinterpret_cast<u64 *>(smem + FastSmem::kBarAt);
    volatile u32 *s_abort = reinterpret_cast<volatile u32 *>(smem + FastSmem::kAbortAt);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const u32 first = blockIdx.x, stride = gridDim.x;
    const u32 my_tiles = b.total_tiles > first ? (b.total_tiles - first + stride - 1) / stride : 0;
    const int n_layers = (int)b.n_layers;
    auto seek = [&](u32 gt, int &li) {      // (tiles only go up)
        while (li + 1 < n_layers && b.layer[li + 1].tile_first <= gt) li++;
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
        if ((u64)lt >= L.geo.n / T) return;             // a ragged last tile is read with plain loads
        unsigned char *st = smem + (i % kStages) * kStageBytes;
        u64 *bar = &s_full[i % kStages];
        mbar_arrive_expect_tx(bar, 8u * T + (LAZY ? kMaskBytes : 0u));
        bulk_load(st, L.grad + (u64)lt * T, 4u * T, bar);
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
            full_tiles = (u32)(geo.n / (u64)T);
            wbytes = geo.w;
            // the thread's elements [0, cut) lie in bin b0 of the tile, from place off0 of it on, the others
            // in bin b0 + 1; only the first `vcount` of them exist (tiles of less than 4000 elements)
            const int Lt = (int)geo.L_T, e0 = tid * kSeg;
            b0 = e0 / Lt;
            off0 = e0 - b0 * Lt;
            cut = min(kSeg, Lt - off0);
            vcount = max(0, min(kSeg, T - e0));
            aligned = T == kFastTile && Lt % kSeg == 0;     // (then cut = vcount = 25 in every thread)
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
        const u64 base = (u64)lt * (u64)T;
        float *s_d = reinterpret_cast<float *>(smem + (i % kStages) * kStageBytes);
        float *s_r = s_d + kFastTile;
        const bool whole = lt < full_tiles;
        const int elems = whole ? T : (int)(geo.n - base);
        u32 *const any_max = s_anymax + (i & 1) * kSmallBins, *const any_cnt = s_anycnt + (i & 1) * kSmallBins;

        if (whole) {
            const u32 stage = i % kStages;
            if (!mbar_wait(&s_full[stage], (phase >> stage) & 1u)) {
                *s_abort = 1;                      // every thread that times out says so
                raise_status(ADACOMP_DEV_TIMEOUT);
            }
            phase ^= 1u << stage;
        } else {
            // the ragged last tile of a layer: plain loads, zero fill past the end
            for (int e = tid; e < kFastTile; e += kFastThreads) {
                float d = 0.f, r = 0.f;
                if (e < elems) { d = L.grad[base + e]; r = L.residue[base + e]; }
                s_d[e] = d;
                s_r[e] = r;
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
            // 500, the tests on `vcount` and `cut` fold away)
            auto form = [&](auto lined_up) {
                constexpr bool AL = decltype(lined_up)::value;
                const int vc = AL ? kSeg : vcount, ct = AL ? kSeg : cut;
#pragma unroll
                for (int j = 0; j < kSeg; j++) {
                    float d = pd[j], r = pr[j];
                    if (j >= vc) d = r = 0.f;               // past the tile's end
                    if (LAZY) {
                        // r holds last step's G: finish "residue = G - sign(G) * scale" where it was sent
                        const float q = __uint_as_float(prev_scale_bits | (__float_as_uint(r) & 0x80000000u));
                        const float fixed = __fsub_rn(r, q);
                        r = (prev >> j & 1u) ? fixed : r;
                    }
                    g[j] = __fadd_rn(r, d);
                    const float h = __fadd_rn(g[j], d);
                    if (j >= ct) m1 = fmaxf(m1, fabsf(g[j]));
                    else m = fmaxf(m, fabsf(g[j]));
                    key[j] = fmaxf(fabsf(h), fabsf(g[j]));
                }
            };
            if (aligned) form(TrueType{});
            else form(FalseType{});
            // (non-negative floats order like their bits)
            if (m > 0.f && b0 < TB) atomicMax(&any_max[b0], __float_as_uint(m));
            if (m1 > 0.f && b0 + 1 < TB) atomicMax(&any_max[b0 + 1], __float_as_uint(m1));
        }
        __syncthreads();                                            // barrier A
        // the other parity's buffers are free: tile i - 1 is done with them, tile i + 1 starts after barrier D
        if (tid < kSmallBins) {
            s_anymax[((i & 1) ^ 1) * kSmallBins + tid] = 0;
            s_anycnt[((i & 1) ^ 1) * kSmallBins + tid] = 0;
        }
        if (!service) {
            gm = b0 < TB ? __uint_as_float(any_max[b0]) : 0.f;
            gm1 = b0 + 1 < TB ? __uint_as_float(any_max[b0 + 1]) : 0.f;
            // ---- selection (a zero bin has G == 0 everywhere and sends nothing) ----
            if (aligned) {
#pragma unroll
                for (int j = 0; j < kSeg; j++)
                    if (key[j] >= gm && g[j] != 0.f) selmask |= 1u << j;
            } else {
#pragma unroll
                for (int j = 0; j < kSeg; j++)
                    if (key[j] >= (j >= cut ? gm1 : gm) && g[j] != 0.f) selmask |= 1u << j;
            }
            cnt = __popc(selmask);
            const u32 c0 = __popc(selmask & ((1u << cut) - 1u));
            if (c0) atomicAdd(&any_cnt[b0], c0);
            if (cnt - c0) atomicAdd(&any_cnt[b0 + 1], cnt - c0);
            incl = warp_inclusive_scan(cnt, lane);
            s_incl[tid] = incl;
            if (lane == 31) s_wtot[warp] = incl;
        }
        __syncthreads();                                            // barrier B

        u32 total = 0;
        if (!service) {
            // ---- words into the staging area, G back into the residue stage ----
            u32 wpre = 0;
#pragma unroll
            for (int wv = 0; wv < 5; wv++)
                if (wv < warp) wpre += s_wtot[wv];
            float *pr = s_r + tid * kSeg;
#pragma unroll
            for (int j = 0; j < kSeg; j++) pr[j] = g[j];
            u32 at = wpre + incl - cnt;
            u32 mask = selmask;
            while (mask) {
                const int j = __ffs(mask) - 1;
                mask &= mask - 1;
                const u32 neg = __float_as_uint(pr[j]) >> 31;
                const u32 idx = j >= cut ? (u32)(j - cut) : (u32)(off0 + j);        // the element's place in its bin
                const u32 word = (idx << 2) | 1u | (neg << 1);
                if (wbytes == 1u) s_words[at] = (unsigned char)word;
                else reinterpret_cast<unsigned short *>(s_words)[at] = (unsigned short)word;
                at++;
            }
            if (LAZY) lazy_mask[(u64)lt * kTileSegs + tid] = selmask;
            if (tid < TB) {
                const u64 bin = (u64)lt * (u64)TB + tid;
                if (bin < geo.n_bins) {
                    unsigned char *bc = L.packed + geo.bin_cnt_at;
                    if (wbytes == 1u) bc[bin] = (unsigned char)any_cnt[tid];
                    else reinterpret_cast<unsigned short *>(bc)[bin] = (unsigned short)any_cnt[tid];
                }
            }
            fence_async_smem();          // the bulk store below reads what was just written
        } else {
            total = s_wtot[0] + s_wtot[1] + s_wtot[2] + s_wtot[3] + s_wtot[4];
            for (int bb = 0; bb < TB; bb += 32) {       // every lane takes part each round
                const int bq = bb + lane;
                const bool valid = bq < TB && (u64)lt * (u64)TB + bq < geo.n_bins;
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
                    bulk_store(L.residue + base, s_r, 4u * (u32)T);
                    bulk_commit();
                }
            } else {
                for (int e = lane; e < elems; e += 32) L.residue[base + e] = s_r[e];
            }
            uint4 *slot = reinterpret_cast<uint4 *>(scratch + geo.slots_at + (u64)lt * geo.slot_bytes);
            const int chunks = (int)((total * wbytes + 15) / 16);
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
    finalize_body(L.packed, L.packed + L.geo.scratch_at, L.geo, 0u, L.count_out, L.lazy);
}

// FIXUP: also finishes the sent elements' residues (eager mode; lazy-scale mode leaves G).
template <int N, bool FIXUP>
__global__ void __launch_bounds__(kGatherThreads)
batch_gather(const __grid_constant__ BatchArgsT<N> b)
{
    __shared__ u32 s_pre_all[kGatherThreads / 32][kSmallBins + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const u32 warps = gridDim.x * (kGatherThreads / 32);
    for (u32 gt = blockIdx.x * (kGatherThreads / 32) + warp; gt < b.total_tiles; gt += warps) {
        const BatchLayer &L = b.layer[batch_layer_of(b, gt)];
        const unsigned char *scratch = L.packed + L.geo.scratch_at;
        if (L.geo.w == 1u)
            gather_tile_small<unsigned char, FIXUP>(L.residue, L.packed, scratch, L.geo, gt - L.tile_first, lane, s_pre_all[warp]);
        else
            gather_tile_small<unsigned short, FIXUP>(L.residue, L.packed, scratch, L.geo, gt - L.tile_first, lane, s_pre_all[warp]);
    }
}

// ---------------------------------------------------------------------------------
// decode_sum: unpack() of k streams and their ordered sum.
// ---------------------------------------------------------------------------------

// What becomes of a finished tile of the ordered sum s: stored to dst (unpack() alone), or, with
// `weights` set, averageGradients() and updateWeights() of Algorithm 1 on the spot, every operation
// rounded to binary32 on its own, so that the dense gradient never reaches memory.  The paper
// names its optimizers ("SGD with momentum", Adam) and prints no formula:
//   SGD (adam == 0): the plain heavy-ball step
//       mean = s / k,  v' = (mu * v) + mean,  w' = w - (lr * v')
//   Adam (adam != 0): Kingma and Ba's Algorithm 1 in its "efficient" order; `momentum` is the first
//       moment m, `second` the second moment v, `mu` beta1, `lr` the bias-corrected step size
//       alpha * sqrt(1 - beta2^t) / (1 - beta1^t), which the caller computes
//       mean = s / k,  m' = (beta1 * m) + ((1 - beta1) * mean),  v' = (beta2 * v) + ((1 - beta2) * (mean * mean)),
//       w' = w - ((lr * m') / (sqrt(v') + eps))
struct Epilogue {
    float *weights, *momentum, *second;
    float lr, mu, beta2, eps, k;
    u32 adam;
    float inv_k;        // 1 / k where k is a power of two (the product with it is the correctly rounded quotient), else 0
};

// s / k without the division where the quotient is known without it: for k a power of two the product
// with 1 / k is the correctly rounded quotient; otherwise a zero sum, which is what most elements have,
// stays the same zero (and spares the division its slow path).
__device__ inline float mean_of(float s, const Epilogue &ep)
{
    if (ep.inv_k != 0.f) return __fmul_rn(s, ep.inv_k);
    return s == 0.f ? s : __fdiv_rn(s, ep.k);
}

__device__ inline void sgd_step(float s, float &w, float &v, const Epilogue &ep)
{
    const float mean = mean_of(s, ep);
    v = __fadd_rn(__fmul_rn(ep.mu, v), mean);
    w = __fsub_rn(w, __fmul_rn(ep.lr, v));
}

__device__ inline void adam_step(float s, float &w, float &m, float &v, const Epilogue &ep)
{
    const float mean = mean_of(s, ep);
    m = __fadd_rn(__fmul_rn(ep.mu, m), __fmul_rn(__fsub_rn(1.f, ep.mu), mean));
    v = __fadd_rn(__fmul_rn(ep.beta2, v), __fmul_rn(__fsub_rn(1.f, ep.beta2), __fmul_rn(mean, mean)));
    const float num = __fmul_rn(ep.lr, m), den = __fadd_rn(__fsqrt_rn(v), ep.eps);
    w = __fsub_rn(w, num == 0.f ? num : __fdiv_rn(num, den));      // (0 / den is that zero: den > 0 for eps > 0)
}

// Four elements at once.
__device__ inline void sgd_step4(float4 s, float4 &w, float4 &v, const Epilogue &ep)
{
    sgd_step(s.x, w.x, v.x, ep);
    sgd_step(s.y, w.y, v.y, ep);
    sgd_step(s.z, w.z, v.z, ep);
    sgd_step(s.w, w.w, v.w, ep);
}
__device__ inline void adam_step4(float4 s, float4 &w, float4 &m, float4 &v, const Epilogue &ep)
{
    adam_step(s.x, w.x, m.x, v.x, ep);
    adam_step(s.y, w.y, m.y, v.y, ep);
    adam_step(s.z, w.z, m.z, v.z, ep);
    adam_step(s.w, w.w, m.w, v.w, ep);
}

struct DecodeArgs {
    const unsigned char *stream[ADACOMP_MAX_STREAMS];
    Epilogue ep;
    float *dst;
    u32 k;
    u32 pairs;          // the kernel of pair_path() is launched too: its shapes are left to it
    u32 hint_L_T;       // 0: the caller did not say; else the streams must carry exactly this shape
    u64 hint_n;
};

// Work items of the decoder for a tensor: output tiles, split into chunks where a tile is larger.
__host__ __device__ inline u64 decode_items(u64 n, u32 L_T)
{
    const u32 tile_bins = L_T <= 1000u ? 4u * (1000u / L_T) : 1u;
    const u64 n_bins = (n + L_T - 1) / L_T;
    const u64 n_tiles = (n_bins + tile_bins - 1) / tile_bins;
    return n_tiles * (((u64)tile_bins * L_T + kDecodeChunk - 1) / kDecodeChunk);
}

constexpr int kWbufBytes = 8192;     // staged words of one round of learners (one learner's worst case fits)
constexpr int kRoundMax = 4;         // learners per round
constexpr int kGenericSegBins = 1024;   // generic decode: bins scanned per pass

// shared memory of the warp path (described with decode_warps below)
#ifndef ADACOMP_WARPS_PER_SM
#define ADACOMP_WARPS_PER_SM 6
#endif
constexpr int kWarpsPerSm = ADACOMP_WARPS_PER_SM;    // CTAs of the warp decoder per SM
constexpr int kSlots = 8;                       // tiles in flight per CTA at most
constexpr u32 kRingBytes = 19200;
constexpr u32 kSlotMax = kRingBytes / 2;        // a slot never takes more: two tiles are always in flight
// (five decoding warps: the kernel of the pairs of tiles, whose items are twice as large; what four CTAs per SM leave)
#ifndef ADACOMP_PAIR_RING
#define ADACOMP_PAIR_RING 21504
#endif
__host__ __device__ constexpr u32 ring_bytes(int nw) { return nw == 5 ? (u32)ADACOMP_PAIR_RING : kRingBytes; }

template <int NW>
struct WarpDecSmem {
    uint4 ring[ring_bytes(NW) / 16];
    u32 tmp[NW][32];                            // per decoding warp: output places of its non-empty bins
    unsigned short coff[ADACOMP_MAX_STREAMS];   // byte offset in a slot of learner l's bin counts (its words follow them)
    unsigned short wcap[ADACOMP_MAX_STREAMS];   // bytes of its word region
    unsigned char rfirst[ADACOMP_MAX_STREAMS];  // round r brings learners [rfirst[r], rfirst[r] + rcount[r]) of a tile
    unsigned char rcount[ADACOMP_MAX_STREAMS];
    u64 full[kSlots], empty[kSlots];            // mbarriers of the slots
    u64 wv_full[NW];                            // optimizer epilogue: a warp's share of the optimizer's arrays has landed
    u32 slot_bytes, n_slots, n_rounds, abort;
};

// A slot holds one round of one tile: the learners of the round, as many as fit a slot with their
// regions (all k of them when k is small).  It starts with {u32 staged, u32 bad, u32 item} (the first
// `staged` learners of the round are in the slot; failed directory checks; where items are 4096
// elements: the first one's place in its bin, the bins of the item << 16, the counts' offset in
// their room << 24), 4 bytes of padding, then u16 cnt[k8] and u16 head[k8], indexed by the learner's place in the round: its words in
// this tile and the byte offset of the first one in its word region.
constexpr u32 kSlotHead = 16;

struct DecodeSmem {
    float acc[kDecodeChunk];                    // the output tile
    union {
        struct {
            u32 pre[kGenericSegBins + 1];       // generic path: scanned bin counts of one stream
            u32 tmp[40];
        } g;
        struct {
            u32 tmp[40];
            uint4 wbuf[kWbufBytes / 16];        // staged path: the round's words
            u32 bin_pre[kRoundMax][33];         // staged by-word path: scanned bin counts per learner
            u64 off0[ADACOMP_MAX_STREAMS];      // first word of this tile in stream l
            u32 cnt[ADACOMP_MAX_STREAMS];       // words of this tile in stream l
        } f;
    };
    u64 n_sel[ADACOMP_MAX_STREAMS];             // words in stream l
    float scale[ADACOMP_MAX_STREAMS];
};

__device__ inline void store_tile(float *dst, u64 out0, u32 len, float *s_acc, const Epilogue &ep)
{
    const int tid = threadIdx.x;
    if (ep.weights) {
        for (u32 i = tid; i < len; i += kDecodeThreads) {
            float w = ep.weights[out0 + i], v = ep.momentum[out0 + i];
            if (ep.adam) {
                float v2 = ep.second[out0 + i];
                adam_step(s_acc[i], w, v, v2, ep);
                ep.second[out0 + i] = v2;
            } else {
                sgd_step(s_acc[i], w, v, ep);
            }
            ep.momentum[out0 + i] = v;
            ep.weights[out0 + i] = w;
            s_acc[i] = 0.f;
        }
        return;
    }
    if ((out0 & 3u) == 0) {
        float4 *o4 = reinterpret_cast<float4 *>(dst + out0);
        float4 *s4 = reinterpret_cast<float4 *>(s_acc);
        for (u32 i = tid; i < len / 4; i += kDecodeThreads) {
            __stcs(o4 + i, s4[i]);
            s4[i] = make_float4(0.f, 0.f, 0.f, 0.f);       // ready for the next tile
        }
        for (u32 i = (len & ~3u) + tid; i < len; i += kDecodeThreads) { dst[out0 + i] = s_acc[i]; s_acc[i] = 0.f; }
    } else {
        for (u32 i = tid; i < len; i += kDecodeThreads) { dst[out0 + i] = s_acc[i]; s_acc[i] = 0.f; }
    }
}

// Number of malformed fields in four packed bytes (Word = u8) or two packed halfwords (u16)
// of staged payload: the reserved ternary code 10, or an index >= L_T (field >= 4 * L_T).
// Returns non-zero status bits instead of a count.
template <typename Word>
__device__ inline u32 check_fields(u32 x, u32 L_T)
{
    u32 bad = 0;
    if (sizeof(Word) == 1) {
        const u32 t = (x & 0x03030303u) ^ 0x02020202u;                    // zero byte <=> code 10
        if ((t - 0x01010101u) & ~t & 0x80808080u) bad |= ADACOMP_DEV_RESERVED_CODE;
        const u32 T = 4u * L_T;                                           // L_T <= 64
        if (T < 256u) {
            const u32 low = x & 0x7f7f7f7fu;
            const u32 ge = T >= 128u ? ((low + (256u - T) * 0x01010101u) & x)
                                     : ((low + (128u - T) * 0x01010101u) | x);
            if (ge & 0x80808080u) bad |= ADACOMP_DEV_BAD_STREAM;
        }
    } else {
        const u32 t = (x & 0x00030003u) ^ 0x00020002u;
        if ((t - 0x00010001u) & ~t & 0x80008000u) bad |= ADACOMP_DEV_RESERVED_CODE;
        const u32 T = 4u * L_T;                                           // L_T <= 16384
        if (T < 65536u) {
            const u32 low = x & 0x7fff7fffu;
            const u32 ge = T >= 32768u ? ((low + (65536u - T) * 0x00010001u) & x)
                                       : ((low + (32768u - T) * 0x00010001u) | x);
            if (ge & 0x80008000u) bad |= ADACOMP_DEV_BAD_STREAM;
        }
    }
    return bad;
}

// Fast decode for tiles of at most 96 bins and 4096 elements (L_T = 42..1000).
//
// Per tile: (1) each learner's word range comes from its directory;
// (2) the words of a round of up to four learners are staged in shared memory with 16-byte
// loads, all in flight together, and checked as they pass (reserved code, index beyond the
// bin); (3) the words are added into the output tile in learner order:
//   BY_BIN  (32..96 bins): thread b owns bin b for every learner, so one thread adds all
//           contributions to an element, in learner order, with no barrier in between;
//   by word (2..31 bins): a learner's words are spread over the threads and a barrier
//           separates consecutive learners;
// (4) the tile is stored once with 128-bit streaming stores.
// A stream that fails a check raises a status bit; its words are still applied with the index
// clamped into the bin, so nothing is read or written out of bounds.
template <typename Word, bool BY_BIN>
__device__ void decode_item_staged(const unsigned char *const *streams, u32 k, const Geometry &geo, u64 tile,
                                   float *dst, const Epilogue &ep, DecodeSmem &sm, u32 &bad)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int TB = (int)geo.tile_bins;
    const u32 L_T = geo.L_T;
    u32 *s_wsum = sm.f.tmp;                    // BY_BIN: [4 warps][2 packed pairs of learners]
    const unsigned char *s_bytes = reinterpret_cast<const unsigned char *>(sm.f.wbuf);
    constexpr u32 kCap = kWbufBytes / 16;
    int top_probe = 1;                         // by word: highest power of two below the bin count
    while (top_probe * 2 < TB) top_probe *= 2;
    const u64 base = tile * (u64)geo.tile_elems;
    const u64 bin0 = tile * (u64)TB;

    if (tid < (int)k) {
        const unsigned char *s = streams[tid];
        const u64 n_sel = reinterpret_cast<const u64 *>(s)[5];
        const u64 *dir = reinterpret_cast<const u64 *>(s + geo.tile_off_at);
        const u64 o0 = dir[tile], o1 = dir[tile + 1];
        // a malformed directory must not send the copy below out of the stream
        const bool ok = o1 >= o0 && o1 - o0 <= geo.tile_elems && o1 <= n_sel;
        if (!ok) bad |= ADACOMP_DEV_BAD_STREAM;
        sm.scale[tid] = __uint_as_float(reinterpret_cast<const u32 *>(s)[12]);
        sm.f.off0[tid] = o0;
        sm.f.cnt[tid] = ok ? (u32)(o1 - o0) : 0u;
    }
    consumer_barrier();

    for (u32 g0 = 0; g0 < k; g0 += kRoundMax) {
        // ---- a group of up to four learners: one round if its words fit the staging
        //      buffer, else one round per learner (a single learner's tile always fits) ----
        const int R = (int)min((u32)kRoundMax, k - g0);
        u64 src[kRoundMax];
        u32 chunks[kRoundMax], headb[kRoundMax], cnts[kRoundMax];
        u32 total = 0;
#pragma unroll
        for (int q = 0; q < kRoundMax; q++) {
            src[q] = 0; chunks[q] = 0; headb[q] = 0; cnts[q] = 0;
            if (q < R) {
                const u64 p = (u64)(uintptr_t)(streams[g0 + q] + geo.payload_at) + sm.f.off0[g0 + q] * sizeof(Word);
                cnts[q] = sm.f.cnt[g0 + q];
                headb[q] = (u32)(p & 15u);
                src[q] = p & ~(u64)15u;
                chunks[q] = cnts[q] ? (headb[q] + cnts[q] * (u32)sizeof(Word) + 15u) / 16u : 0u;
                total += chunks[q];
            }
        }
        const bool fits = total <= kCap;
        const int nsub = fits ? 1 : R;
        for (int sub = 0; sub < nsub; sub++) {
            // learners of this round: q in [q_lo, q_hi); chunk offsets at[q] within the buffer
            const int q_lo = fits ? 0 : sub, q_hi = fits ? R : sub + 1;
            u32 at[kRoundMax + 1];
            at[0] = 0;
#pragma unroll
            for (int q = 0; q < kRoundMax; q++)
                at[q + 1] = at[q] + ((q >= q_lo && q < q_hi) ? chunks[q] : 0u);

            // ---- stage and check the words ----
            for (u32 c = tid; c < at[kRoundMax]; c += kDecodeThreads) {
                u64 from = src[0];
                u32 first = 0;
#pragma unroll
                for (int q = 1; q < kRoundMax; q++)
                    if (c >= at[q]) { from = src[q]; first = at[q]; }
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(from) + (c - first));
                bad |= check_fields<Word>(v.x, L_T) | check_fields<Word>(v.y, L_T) |
                       check_fields<Word>(v.z, L_T) | check_fields<Word>(v.w, L_T);
                sm.f.wbuf[c] = v;
            }

            if (BY_BIN) {
                // ---- bin counts -> word offsets: two learners per scan (16 bits each) ----
                const u64 bin = bin0 + tid;
                const bool live = tid < TB && bin < geo.n_bins;
                u32 c[kRoundMax];
#pragma unroll
                for (int q = 0; q < kRoundMax; q++) {
                    c[q] = 0;
                    if (q >= q_lo && q < q_hi && live)
                        c[q] = min((u32)reinterpret_cast<const Word *>(streams[g0 + q] + geo.bin_cnt_at)[bin], L_T);
                }
                u32 pair[2] = {c[0] | (c[1] << 16), c[2] | (c[3] << 16)};
                u32 excl[2];
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const u32 inc = warp_inclusive_scan(pair[h], lane);
                    excl[h] = inc - pair[h];
                    if (lane == 31) s_wsum[warp * 2 + h] = inc;
                }
                consumer_barrier();
                if (tid < TB) {
                    for (int wv = 0; wv < warp; wv++) {
                        excl[0] += s_wsum[wv * 2];
                        excl[1] += s_wsum[wv * 2 + 1];
                    }
                    const u32 pre[kRoundMax] = {excl[0] & 0xffffu, excl[0] >> 16, excl[1] & 0xffffu, excl[1] >> 16};
                    float *mine = sm.acc + tid * L_T;
#pragma unroll
                    for (int q = 0; q < kRoundMax; q++) {
                        if (c[q] == 0) continue;
                        if (pre[q] + c[q] > cnts[q]) { bad |= ADACOMP_DEV_BAD_STREAM; continue; }
                        const Word *p = reinterpret_cast<const Word *>(s_bytes + at[q] * 16u + headb[q]) + pre[q];
                        const u32 sbits = __float_as_uint(sm.scale[g0 + q]);
                        for (u32 i = 0; i < c[q]; i++) {
                            const u32 word = p[i];
                            const u32 e = min(word >> 2, L_T - 1u);
                            const float add = (word & 1u) ? __uint_as_float(sbits ^ ((word & 2u) << 30)) : 0.f;
                            mine[e] = __fadd_rn(mine[e], add);
                        }
                    }
                }
                consumer_barrier();
            } else {
                // warp wv scans the bin counts of learner wv of the round
                if (warp >= q_lo && warp < q_hi) {
                    u32 c = 0;
                    if (lane < TB && bin0 + lane < geo.n_bins)
                        c = reinterpret_cast<const Word *>(streams[g0 + warp] + geo.bin_cnt_at)[bin0 + lane];
                    const u32 inc = warp_inclusive_scan(c, lane);
                    sm.f.bin_pre[warp][lane] = inc - c;
                    if (lane == 31) sm.f.bin_pre[warp][32] = inc;
                }
                consumer_barrier();
#pragma unroll
                for (int q = 0; q < kRoundMax; q++) {
                    if (q < q_lo || q >= q_hi || cnts[q] == 0) continue;      // the same for every thread
                    if (sm.f.bin_pre[q][32] != cnts[q]) { bad |= ADACOMP_DEV_BAD_STREAM; continue; }
                    const Word *p = reinterpret_cast<const Word *>(s_bytes + at[q] * 16u + headb[q]);
                    const u32 sbits = __float_as_uint(sm.scale[g0 + q]);
                    const u32 *pre = sm.f.bin_pre[q];
                    for (u32 j = tid; j < cnts[q]; j += kDecodeThreads) {
                        const u32 word = p[j];
                        int b = 0;
                        for (int step = top_probe; step > 0; step >>= 1)
                            if (b + step < TB && pre[b + step] <= j) b += step;
                        const u32 e = (u32)b * L_T + min(word >> 2, L_T - 1u);
                        const float add = (word & 1u) ? __uint_as_float(sbits ^ ((word & 2u) << 30)) : 0.f;
                        sm.acc[e] = __fadd_rn(sm.acc[e], add);
                    }
                    consumer_barrier();
                }
                consumer_barrier();     // bin_pre and wbuf are rewritten by the next round
            }
        }
    }
    const u32 len = (u32)min((u64)geo.tile_elems, geo.n - base);
    store_tile(dst, base, len, sm.acc, ep);
    consumer_barrier();
}

// ---------------------------------------------------------------------------------
// decode, warp path: every L_T above 40.  A work item is a tile of 4..96 bins (L_T <= 1000) or,
// where a tile is one bin (L_T > 1000), 4096 consecutive output elements and the 1 to 6 bins
// they lie in.
//
// Warp 4 is a loader: for every item of this CTA, a lane per learner reads the learner's two
// directory entries (two steps ahead) and bulk-copies (TMA, no multicast) that learner's bin
// counts and words of the item into the learner's fixed region of a shared-memory slot; the
// slots form a ring of up to kSlots in flight.  (A bulk copy starts on a 16-byte boundary: counts
// and words are copied from the boundary at or below their first byte and found at the offset.)  Region sizes are set once per launch from the
// streams' word totals (1.5 times a tile's average plus slack).  When the k regions do not fit
// one slot together, a tile takes several rounds, each a slot of its own with the next learners
// in order.  A learner whose words of some tile do not fit its region is read by the decoding
// warps straight from global memory for that tile.  The loader does nothing else: it shares its
// SM's issue slots with some thirty busy warps, so its chain of dependent instructions per
// tile has to stay short.
//
// Warps 0-3 decode.  Each owns a quarter of the tile's bins and of the output tile and never
// touches the rest, so the four need no barrier among themselves: a warp waits for the slot,
// adds its words learner by learner (one __syncwarp() between learners keeps an element's
// contributions in learner order), gives the slot back, hands its quarter to one bulk copy
// (TMA store: the output does not pass through the warps' load/store path, which the adds keep
// busy) and zeroes it once the copy has read it.
// Tiles of 80 bins of 8-bit words (L_T = 48, 49, 50; tensors of 256 tiles and more) are taken in pairs by a
// kernel of its own with five decoding warps: an item is then 160 bins, 32 per warp (see pair_path()).
// Four schemes for the adds.  Where a warp's share of the item is a multiple of 4 and at most 32 bins of
// 8-bit words (the pairs; the 80- and 96-bin tiles in the kernels with an optimizer step): a lane per
// bin, see warp_add_lanes_all().  Items of 4096 elements (L_T > 1000): a warp owns a quarter of the
// elements whatever the bins are, reads the words of the bins its elements lie in and adds those
// that are its own.  Tiles of at most 64 bins (16-bit words among them): G lanes share a
// bin and take every G-th word of it.  Tiles of more bins (8-bit words, L_T <= 58): the warp works
// by word, lane j takes word j of the warp's run of words, 32 at a time; the bin of a word comes
// from the bin counts: the lanes that hold the warp's bins (at most 24) scan their counts, raise
// a flag bit at the position of each non-empty bin's first word, and a word's bin is the number
// of flags at or before it (a population count), mapped to the bin's place in the output tile by
// one shuffle.
// Loader and decoding warps meet only through the slots' full / empty mbarriers, and every wait
// on those is bounded.
// ---------------------------------------------------------------------------------

template <typename Word, bool SHARED>
__device__ inline u32 load_word(u64 addr)
{
    u32 v;
    if (SHARED) {
        if (sizeof(Word) == 1) asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"((u32)addr) : "memory");
        else asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"((u32)addr) : "memory");
    } else {
        if (sizeof(Word) == 1) asm volatile("ld.global.nc.u8 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
        else asm volatile("ld.global.nc.u16 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
    }
    return v;
}

// out[e] += v (fp32, round to nearest even, denormals kept) for a word that carries a value
// (bit 0 set) and an index inside its bin (word < 4 L_T); nothing is read or written otherwise.
__device__ inline void add_at_if_valid(u32 e, float v, u32 word, u32 LT4)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b32 t;\n\t.reg .f32 x;\n\t"
        "and.b32 t, %2, 1;\n\t"
        "setp.ne.u32 p, t, 0;\n\t"
        "setp.lt.and.u32 p, %2, %3, p;\n\t"
        "@p ld.shared.f32 x, [%0];\n\t"
        "@p add.rn.f32 x, x, %1;\n\t"
        "@p st.shared.f32 [%0], x;\n\t}"
        ::"r"(e), "f"(v), "r"(word), "r"(LT4)
        : "memory");
}

// A group of up to four learners, as the decoding warp holds it: lane q (q < 4) has learner q's
// addresses of its bin counts and first word of this tile, the words the directory gives it in
// this tile, and its scale's bits; the other lanes get them by shuffle.
template <typename Addr>
struct GroupSrc {
    Addr counts, words;
    u32 limit, sbits;
};
__device__ inline u32 bcast(u32 v, int q) { return __shfl_sync(0xffffffffu, v, q); }
__device__ inline u64 bcast(u64 v, int q)
{
    return ((u64)__shfl_sync(0xffffffffu, (u32)(v >> 32), q) << 32) | __shfl_sync(0xffffffffu, (u32)v, q);
}

// 1 << d for d < 32, else 0 (PTX shifts clamp at the register width).
__device__ inline u32 shl_clamped(u32 d)
{
    u32 r;
    asm("shl.b32 %0, 1, %1;" : "=r"(r) : "r"(d));
    return r;
}

// The warp's view of up to four learners' bin counts of one tile.  Two learners share a register
// (16 bits each: a tile has at most 4096 words), so one scan and one reduction serve two
// learners.  For learner q (field q & 1 of register q >> 1): `bef` = words of the tile in bins ahead
// of the warp's (the same in every lane); lane i holds in `mine` the count of the warp's bin i
// and in `ex` the words of the warp's bins ahead of it; `tot` = words of the warp's bins together.
struct WarpBins {
    u32 mine[2], ex[2], bef[2], tot[2];
};
__device__ inline u32 field(const u32 *x, int q) { return (x[q >> 1] >> (16 * (q & 1))) & 0xffffu; }

//   counts(q)  address of learner q's bin counts of this tile (bin 0 of the tile)
//   b0, nb     the warp's bins are [b0, b0 + nb) of the tile; `live` of the tile's bins exist
template <typename Word, bool SHARED, typename CountsFn>
__device__ inline void warp_bins(CountsFn counts, int R, int b0, int nb, u32 live, u32 L_T, int lane, WarpBins &wb)
{
    constexpr u32 full = 0xffffffffu;
    u32 bef[2] = {0u, 0u};
    wb.mine[0] = wb.mine[1] = 0u;
    const u32 mb = (u32)(b0 + lane);
    const bool have = lane < nb && mb < live;
#pragma unroll
    for (int q = 0; q < kRoundMax; q++) {
        if (q < R) {
            const auto at = counts(q);
            u32 cq = 0, bq = 0;
            if (have) cq = min(load_word<Word, SHARED>(at + mb * (u32)sizeof(Word)), L_T);
            if (SHARED && sizeof(Word) == 1 && ((((u32)at) | (u32)b0) & 3u) == 0u && (u32)b0 <= live) {
                // four 8-bit counts per load (the counts' run and the warp's first bin are 4-byte aligned);
                // a count beyond L_T (a malformed stream) is clamped like the others: bytes are compared pairwise
                if ((u32)lane < ((u32)b0 >> 2)) {
                    u32 x;
                    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"((u32)at + 4u * (u32)lane) : "memory");
                    x = __vminu4(x, L_T * 0x01010101u);
                    bq = __dp4a(x, 0x01010101u, 0u);
                }
            } else {
#pragma unroll
                for (int r = 0; r < 4; r++) {       // bins before b0: at most 128
                    const u32 b = (u32)lane + 32u * r;
                    if (b < (u32)b0 && b < live) bq += min(load_word<Word, SHARED>(at + b * (u32)sizeof(Word)), L_T);
                }
            }
            wb.mine[q >> 1] |= cq << (16 * (q & 1));
            bef[q >> 1] += bq << (16 * (q & 1));
        }
    }
#pragma unroll
    for (int h = 0; h < 2; h++) {
        wb.ex[h] = wb.bef[h] = wb.tot[h] = 0u;
        if (2 * h < R) {
            wb.bef[h] = b0 > 0 ? __reduce_add_sync(full, bef[h]) : 0u;
            const u32 incl = warp_inclusive_scan(wb.mine[h], lane);
            wb.ex[h] = incl - wb.mine[h];
            wb.tot[h] = __shfl_sync(full, incl, 31);
        }
    }
}

// One learner's words of one warp's bins, added into the warp's part of the output tile.
//   words    address of the first of them (word `before` of the learner's words of this tile)
//   W, c, excl  as WarpBins gives them for this learner
//   acc_at   shared-memory address of the first output element of the warp's first bin
//   tmp      32 words of scratch of this warp
// SHARED: `words` is a shared-memory address (a slot), else a global one.
// Returns the ADACOMP_DEV_* bits of what was wrong with the data.
template <typename Word, bool SHARED, typename Addr>
__device__ inline u32 warp_add_words(Addr words, u32 W, u32 c, u32 excl, int nb, u32 L_T, u32 sbits, u32 acc_at,
                                     u32 *tmp, int lane)
{
    constexpr u32 full = 0xffffffffu;
    if (W == 0) return 0;
    // ---- the output place of the r-th non-empty bin, held by lane r ----
    const u32 LT4 = L_T * 4u;
    u32 place = acc_at + (u32)lane * LT4;
    const u32 ne = __ballot_sync(full, c != 0u);
    if (ne & (ne + 1u)) {                           // (the non-empty bins are not the warp's first ones in a row)
        __syncwarp();
        if (c != 0u) tmp[__popc(ne & ((1u << lane) - 1u))] = place;
        __syncwarp();
        place = tmp[lane];
    }

    // ---- the words, 32 at a time: lane j takes word j0 + j ----
    const u32 le_mask = (2u << lane) - 1u;
    Addr wp = words + (Addr)((u32)lane * (u32)sizeof(Word));
    u32 d = c != 0u ? excl : 0x80000000u;           // distance from j0 to the first word of my bin (none: far away)
    u32 left = W - min(W, (u32)lane);               // words at or after mine
    int rbase = -1;
    u32 mx = 0, rsv = 0;
    for (u32 j0 = 0; j0 < W; j0 += 32u) {
        const u32 m = __reduce_or_sync(full, shl_clamped(d));         // first words of bins in this chunk
        d -= 32u;
        const int r = rbase + __popc(m & le_mask);
        rbase += __popc(m);
        const u32 bin_at = __shfl_sync(full, place, r);
        u32 word = 0;
        if (left != 0u) word = load_word<Word, SHARED>(wp);
        left -= min(left, 32u);
        wp += (Addr)(32u * (u32)sizeof(Word));
        mx = max(mx, word);
        rsv |= (word >> 1) & ~word;
        // 4 * idx is the element's byte offset in its bin
        add_at_if_valid(bin_at + (word & ~3u), __uint_as_float(sbits ^ ((word << 30) & 0x80000000u)), word, LT4);
    }
    u32 bad = 0;
    if (__any_sync(full, (rsv & 1u) != 0u)) bad |= ADACOMP_DEV_RESERVED_CODE;
    if (__any_sync(full, mx >= LT4)) bad |= ADACOMP_DEV_BAD_STREAM;
    return bad;
}

// Up to four learners (a group, in learner order) of one warp's bins of one tile, by word.
template <typename Word, bool SHARED, typename Addr>
__device__ inline u32 warp_add_group(const GroupSrc<Addr> &src, int R, int b0, int nb, u32 live, u32 L_T, u32 acc_at,
                                     u32 *tmp, int lane)
{
    WarpBins wb;
    warp_bins<Word, SHARED>([&](int q) { return bcast(src.counts, q); }, R, b0, nb, live, L_T, lane, wb);
    u32 bad = 0;
#pragma unroll
    for (int q = 0; q < kRoundMax; q++) {
        if (q >= R) break;
        const Addr words = bcast(src.words, q);
        const u32 limit = bcast(src.limit, q), sbits = bcast(src.sbits, q);
        const u32 before = field(wb.bef, q), W = field(wb.tot, q);
        if (before + W > limit) {
            bad |= ADACOMP_DEV_BAD_STREAM;          // counts and directory disagree: nothing is read
        } else {
            bad |= warp_add_words<Word, SHARED, Addr>(words + (Addr)(before * (u32)sizeof(Word)), W, field(wb.mine, q),
                                                      field(wb.ex, q), nb, L_T, sbits, acc_at, tmp, lane);
        }
        __syncwarp();                               // learner order, element by element
    }
    return bad;
}

// out[e] += v (as add_at_if_valid) when `go` is not zero; nothing is read or written otherwise.
__device__ inline void add_at_if(u32 e, float v, u32 go)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .f32 x;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "@p ld.shared.f32 x, [%0];\n\t"
        "@p add.rn.f32 x, x, %1;\n\t"
        "@p st.shared.f32 [%0], x;\n\t}"
        ::"r"(e), "f"(v), "r"(go)
        : "memory");
}

// Four 8-bit words of one bin (distinct indices; the no-op word 0 where there is none) added to the bin whose
// first element is at shared-memory address `bin_at`: byte b carries idx << 2 | code, the element is at
// bin_at + 4 idx = bin_at + (b & 0xfc), and the value is sb + (b << 30) as a bit pattern: sb is the scale's
// pattern minus 0x40000000, so code 01 gives +scale and code 11 -scale.  Loads first, stores last.
__device__ inline void add4_words(u32 bin_at, u32 w4, u32 sb)
{
    asm volatile(
        "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .f32 x0, x1, x2, x3;\n\t.reg .b32 t, a4, e0, e1, e2, e3, v0, v1, v2, v3;\n\t"
        "and.b32 t, %1, 0x00000001;\n\tsetp.ne.u32 p0, t, 0;\n\t"
        "and.b32 t, %1, 0x00000100;\n\tsetp.ne.u32 p1, t, 0;\n\t"
        "and.b32 t, %1, 0x00010000;\n\tsetp.ne.u32 p2, t, 0;\n\t"
        "and.b32 t, %1, 0x01000000;\n\tsetp.ne.u32 p3, t, 0;\n\t"
        "and.b32 a4, %1, 0xfcfcfcfc;\n\t"
        "prmt.b32 e0, a4, 0, 0x4440;\n\tadd.u32 e0, e0, %0;\n\t"
        "prmt.b32 e1, a4, 0, 0x4441;\n\tadd.u32 e1, e1, %0;\n\t"
        "prmt.b32 e2, a4, 0, 0x4442;\n\tadd.u32 e2, e2, %0;\n\t"
        "prmt.b32 e3, a4, 0, 0x4443;\n\tadd.u32 e3, e3, %0;\n\t"
        "mad.lo.u32 v0, %1, 0x40000000, %2;\n\t"
        "and.b32 t, %1, 0x00000300;\n\tmad.lo.u32 v1, t, 0x00400000, %2;\n\t"
        "and.b32 t, %1, 0x00030000;\n\tmad.lo.u32 v2, t, 0x00004000, %2;\n\t"
        "and.b32 t, %1, 0x03000000;\n\tmad.lo.u32 v3, t, 0x00000040, %2;\n\t"
        "@p0 ld.shared.f32 x0, [e0];\n\t"
        "@p1 ld.shared.f32 x1, [e1];\n\t"
        "@p2 ld.shared.f32 x2, [e2];\n\t"
        "@p3 ld.shared.f32 x3, [e3];\n\t"
        "{\n\t.reg .f32 f0, f1, f2, f3;\n\t"
        "mov.b32 f0, v0;\n\tmov.b32 f1, v1;\n\tmov.b32 f2, v2;\n\tmov.b32 f3, v3;\n\t"
        "@p0 add.rn.f32 x0, x0, f0;\n\t"
        "@p1 add.rn.f32 x1, x1, f1;\n\t"
        "@p2 add.rn.f32 x2, x2, f2;\n\t"
        "@p3 add.rn.f32 x3, x3, f3;\n\t}\n\t"
        "@p0 st.shared.f32 [e0], x0;\n\t"
        "@p1 st.shared.f32 [e1], x1;\n\t"
        "@p2 st.shared.f32 [e2], x2;\n\t"
        "@p3 st.shared.f32 [e3], x3;\n\t}"
        ::"r"(bin_at), "r"(w4), "r"(sb)
        : "memory");
}

// All the learners staged in a slot, a lane per bin, for the shapes whose bin counts line up with 32-bit
// loads: 8-bit counts whose run in the slot starts on a 16-byte boundary (the item's bins times one byte is a
// multiple of 16), nb a multiple of 4 and at most 32, and all nb bins of the warp inside the tensor.
// Lane t owns bin b0 + t of the item for every learner, so one thread adds all contributions to an
// element, in learner order, and no look-up from word to bin is needed.
// Per learner: lane i < nb / 4 loads the warp's counts 4 i .. 4 i + 3 as one word: a dot product gives
// their total, a scan over nb / 4 lanes the words ahead of each four, and one multiplication the running
// sums inside a four (bytes: a well-formed count is at most 64); the lanes below b0 / 4 sum the bins ahead of
// the warp's the same way.  Then every lane reads its bin's words four at a time (two aligned 32-bit
// loads and a funnel shift), turns the bytes past its count into the no-op word 0, skips (and reports) the
// malformed ones, and adds the others: four loads, four additions, four stores, the elements being distinct.
// Counts are not clamped to L_T: a count beyond it belongs to a stream that is flagged for its sums or
// whose words are skipped one by one, and every read it leads to stays inside the CTA's shared memory.
__device__ inline u32 warp_add_lanes_all(u32 sl_at, const unsigned short *coff, const unsigned short *m_cnt,
                                         const unsigned short *m_head, const float *s_scale, u32 l0, u32 staged,
                                         u32 count_bytes, int b0, int nb, u32 L_T, u32 acc_at, int lane)
{
    constexpr u32 full = 0xffffffffu;
    const u32 LT4 = L_T * 4u;
    const u32 mine_at = acc_at + (u32)lane * LT4;
    const u32 range_add = (256u - LT4) * 0x01010101u;       // (4 L_T is 164..256 here; 256: the term is 0 and no byte is out of range)
    const int nq = nb >> 2, src_lane = lane >> 2;
    const u32 sel = 0x4440u | ((u32)lane & 3u);             // byte (lane & 3) of a register, zero-extended
    const bool own = lane < nq, ahead = (u32)lane < ((u32)b0 >> 2);
    u32 bad = 0, rsv = 0, oor = 0;
#pragma unroll 1
    for (u32 j = 0; j < staged; j++) {
        const u32 l = l0 + j;
        const u32 counts = sl_at + coff[l];
        const u32 limit = m_cnt[j];
        const u32 words = counts + count_bytes + m_head[j];
        const u32 sb = __float_as_uint(s_scale[l]) - 0x40000000u;   // + (word << 30): +scale for code 01, -scale for code 11
        u32 x = 0, y = 0;
        if (own) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"(counts + (u32)(b0 + 4 * lane)) : "memory");
        if (ahead) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(y) : "r"(counts + 4u * (u32)lane) : "memory");
        const u32 t4 = __dp4a(x, 0x01010101u, 0u);
        const u32 before = b0 > 0 ? __reduce_add_sync(full, __dp4a(y, 0x01010101u, 0u)) : 0u;
        u32 v = t4;
#pragma unroll
        for (int d = 1; d < 8; d <<= 1) {
            const u32 t = __shfl_up_sync(full, v, d);
            if (lane >= d) v += t;
        }
        const u32 W = __shfl_sync(full, v, nq - 1);
        const u32 base = __shfl_sync(full, v - t4, src_lane);
        const u32 xs = __shfl_sync(full, x, src_lane);
        const u32 c = lane < nb ? __byte_perm(xs, 0u, sel) : 0u;
        if (before + W > limit) {
            bad |= ADACOMP_DEV_BAD_STREAM;          // counts and directory disagree: nothing is read
            continue;
        }
        u32 p = words + before + base + __byte_perm(xs * 0x01010100u, 0u, sel);     // my first word
        const u32 sh = (p & 3u) * 8u;
        p &= ~3u;
        const u32 groups = (__reduce_max_sync(full, c) + 3u) >> 2;
        int left8 = (int)(8u * c);                  // bits of my words still to come
        // (the next four words are on their way while these four are added)
        u32 x0, x1;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x0) : "r"(p) : "memory");
        asm volatile("ld.shared.u32 %0, [%1+4];" : "=r"(x1) : "r"(p) : "memory");
#pragma unroll 1
        for (u32 g = 0; g < groups; g++) {
            u32 past;
            u32 w4 = __funnelshift_r(x0, x1, sh);
            x0 = x1;
            p += 4u;
            asm volatile("ld.shared.u32 %0, [%1+4];" : "=r"(x1) : "r"(p) : "memory");
            asm("shl.b32 %0, %1, %2;" : "=r"(past) : "r"(full), "r"((u32)left8));     // (a shift by 32 or more gives 0)
            left8 = max(left8 - 32, 0);
            w4 &= ~past;                                                            // bytes past my count: the no-op word
            rsv |= (w4 >> 1) & ~w4;                                                 // bit 0 of a byte: reserved code 10
            const u32 ge = ((w4 & 0x7f7f7f7fu) + range_add) & w4 & 0x80808080u;     // bit 7 of a byte: index >= L_T
            if (ge) {
                oor |= ge;
                w4 &= ~((ge >> 7) * 0xffu);                                         // those are skipped
            }
            // the four elements are distinct (a bin's words carry distinct indices): loads first, stores last
            add4_words(mine_at, w4, sb);
        }
    }
    if (__any_sync(full, (rsv & 0x01010101u) != 0u)) bad |= ADACOMP_DEV_RESERVED_CODE;
    if (__any_sync(full, LT4 < 256u && oor != 0u)) bad |= ADACOMP_DEV_BAD_STREAM;
    return bad;
}

// Tiles of at most 64 bins: G = 32 / (a warp's bins), rounded down, lanes share a bin.  For a group of up to four learners (in learner order) every lane gets its bin's count and
// the words of the tile ahead of that bin from two warp scans over the tile's bin counts (lane j
// holds bins j and j + 32; two learners share a register, 16 bits each), then the bin's lanes
// take every G-th word of the bin.
//   bin      the lane's bin in the tile (>= TB: the lane has none), r its place among the bin's G lanes
//   mine_at  shared-memory address of the bin's first output element
template <typename Word, bool SHARED, typename Addr>
__device__ inline u32 warp_add_group_by_bin(const GroupSrc<Addr> &src, int R, int TB, u32 live, u32 L_T, int bin, int r,
                                            int G, u32 mine_at, int lane)
{
    constexpr u32 full = 0xffffffffu;
    const u32 LT4 = L_T * 4u;
    // ---- packed bin counts of the tile: lo = bin `lane`, hi = bin `lane + 32` ----
    u32 lo[2] = {0u, 0u}, hi[2] = {0u, 0u};
#pragma unroll
    for (int q = 0; q < kRoundMax; q++) {
        if (q < R) {
            const Addr counts = bcast(src.counts, q);
            if ((u32)lane < live) lo[q >> 1] |= min(load_word<Word, SHARED>(counts + (Addr)((u32)lane * (u32)sizeof(Word))), L_T) << (16 * (q & 1));
            if (TB > 32 && (u32)lane + 32u < live)
                hi[q >> 1] |= min(load_word<Word, SHARED>(counts + (Addr)(((u32)lane + 32u) * (u32)sizeof(Word))), L_T) << (16 * (q & 1));
        }
    }
    // ---- per learner pair: words ahead of my bin, words of my bin, words of the tile ----
    u32 ex[2] = {0u, 0u}, cm[2] = {0u, 0u}, tot[2] = {0u, 0u};
    const int bsrc = bin & 31;
#pragma unroll
    for (int h = 0; h < 2; h++) {
        if (2 * h < R) {
            const u32 il = warp_inclusive_scan(lo[h], lane);
            u32 t = __shfl_sync(full, il, 31);
            u32 e = __shfl_sync(full, il - lo[h], bsrc), c = __shfl_sync(full, lo[h], bsrc);
            if (TB > 32) {
                const u32 ih = warp_inclusive_scan(hi[h], lane) + t;
                const u32 e2 = __shfl_sync(full, ih - hi[h], bsrc), c2 = __shfl_sync(full, hi[h], bsrc);
                t = __shfl_sync(full, ih, 31);
                if (bin >= 32) {
                    e = e2;
                    c = c2;
                }
            }
            ex[h] = e;
            cm[h] = bin < TB ? c : 0u;
            tot[h] = t;
        }
    }
    // ---- the words ----
    u32 bad = 0, mx = 0, rsv = 0;
#pragma unroll
    for (int q = 0; q < kRoundMax; q++) {
        if (q >= R) break;
        const Addr words = bcast(src.words, q);
        const u32 limit = bcast(src.limit, q), sbits = bcast(src.sbits, q);
        if (field(tot, q) > limit) {
            bad |= ADACOMP_DEV_BAD_STREAM;          // counts and directory disagree: nothing is read
        } else {
            const u32 c = field(cm, q);
            Addr wp = words + (Addr)((field(ex, q) + (u32)r) * (u32)sizeof(Word));
            for (u32 j = (u32)r; j < c; j += (u32)G) {
                const u32 word = load_word<Word, SHARED>(wp);
                wp += (Addr)((u32)G * (u32)sizeof(Word));
                mx = max(mx, word);
                rsv |= (word >> 1) & ~word;
                add_at_if_valid(mine_at + (word & ~3u), __uint_as_float(sbits ^ ((word << 30) & 0x80000000u)), word, LT4);
            }
        }
        __syncwarp();                               // learner order, element by element
    }
    if (__any_sync(full, (rsv & 1u) != 0u)) bad |= ADACOMP_DEV_RESERVED_CODE;
    if (__any_sync(full, mx >= LT4)) bad |= ADACOMP_DEV_BAD_STREAM;
    return bad;
}

// L_T > 1000 (a tile is one bin): an item is 4096 consecutive output elements, which lie in `live` bins (at
// most 6), and the decoding warps split the elements between them whatever the bins are.  For a group of
// up to four learners (in learner order) the warp reads the words of the bins its own elements lie in (at
// most 3), bin by bin, and adds those that are its own: elements [lo, lo + len) counted from the first
// bin's first element, at shared-memory address acc_at onwards.
template <typename Word, bool SHARED, typename Addr>
__device__ inline u32 warp_add_group_flat(const GroupSrc<Addr> &src, int R, u32 live, u32 lo, u32 len, u32 L_T, u32 acc_at,
                                          int lane)
{
    constexpr u32 full = 0xffffffffu;
    constexpr u32 kBins = 6;
    const u32 LT4 = L_T * 4u;
    // the bins (of the item) of the warp's first and last element
    u32 wf = 0, wl = 0;
#pragma unroll
    for (u32 i = 1; i < kBins; i++) {
        wf += (u32)(lo >= i * L_T);
        wl += (u32)(lo + len > i * L_T);
    }
    // lane q looks at learner q's bin counts: P[t] words lie in the bins ahead of bin wf + t
    u32 P[4] = {0u, 0u, 0u, 0u};
    bool ok = true;
    if (lane < R) {
        u32 run = 0;
#pragma unroll
        for (u32 b = 0; b < kBins; b++) {
            const u32 c = b < live ? min(load_word<Word, SHARED>(src.counts + (Addr)(b * (u32)sizeof(Word))), L_T) : 0u;
#pragma unroll
            for (u32 t = 0; t < 4u; t++)
                if (b < wf + t) P[t] += c;
            run += c;
        }
        ok = run <= src.limit;
        if (!ok || len == 0u) P[0] = P[1] = P[2] = P[3] = 0u;
    }
    u32 bad = __any_sync(full, !ok) ? ADACOMP_DEV_BAD_STREAM : 0u;      // counts and directory disagree: nothing is read
    u32 mx = 0, rsv = 0;
#pragma unroll
    for (int q = 0; q < kRoundMax; q++) {
        if (q >= R) break;
        const Addr words = bcast(src.words, q);
        const u32 sbits = bcast(src.sbits, q);
        u32 j1 = bcast(P[0], q);
#pragma unroll
        for (u32 t = 0; t < 3u; t++) {
            const u32 j0 = j1;
            j1 = bcast(P[t + 1], q);
            if (wf + t > wl) continue;
            const u32 first = (wf + t) * L_T - lo;          // the bin's first element, counted from the warp's (wraps)
            const u32 base = acc_at + 4u * first;
            Addr wp = words + (Addr)((j0 + (u32)lane) * (u32)sizeof(Word));
            for (u32 j = j0 + (u32)lane; j < j1; j += 32u) {
                const u32 word = load_word<Word, SHARED>(wp);
                wp += (Addr)(32u * (u32)sizeof(Word));
                mx = max(mx, word);
                rsv |= (word >> 1) & ~word;
                add_at_if(base + (word & ~3u), __uint_as_float(sbits ^ ((word << 30) & 0x80000000u)),
                          (u32)((word & 1u) != 0u && first + (word >> 2) < len && word < LT4));
            }
        }
        __syncwarp();                               // learner order, element by element
    }
    if (__any_sync(full, (rsv & 1u) != 0u)) bad |= ADACOMP_DEV_RESERVED_CODE;
    if (__any_sync(full, mx >= LT4)) bad |= ADACOMP_DEV_BAD_STREAM;
    return bad;
}

// The same for learners read from global memory (rare).
template <typename Word>
__device__ u32 warp_add_group_by_bin_global(GroupSrc<u64> src, int R, int TB, u32 live, u32 L_T, int bin, int r,
                                                         int G, u32 mine_at, int lane)
{
    return warp_add_group_by_bin<Word, false, u64>(src, R, TB, live, L_T, bin, r, G, mine_at, lane);
}
template <typename Word>
__device__ u32 warp_add_group_global(GroupSrc<u64> src, int R, int b0, int nb, u32 live, u32 L_T, u32 acc_at,
                                                  u32 *tmp, int lane)
{
    return warp_add_group<Word, false, u64>(src, R, b0, nb, live, L_T, acc_at, tmp, lane);
}

template <typename Word>
__device__ u32 warp_add_group_flat_global(GroupSrc<u64> src, int R, u32 live, u32 lo, u32 len, u32 L_T,
                                                       u32 acc_at, int lane)
{
    return warp_add_group_flat<Word, false, u64>(src, R, live, lo, len, L_T, acc_at, lane);
}

// How the warp path cuts a tensor into work items.  L_T <= 1000: an item is a tile.  L_T > 1000 (a tile is one
// bin of up to 16384 elements): item v is the output elements [4096 v, 4096 v + 4096), whatever bins they lie in;
// it needs the words of every bin it touches, at most `max_bins` of them.
struct WarpItems {
    u64 n_items;
    u32 max_bins;   // bins an item needs the counts of
};
// M (tiles of more than one bin only): an item is M consecutive tiles of the stream, decoded as one tile of
// M * tile_bins bins (their bin counts and their words are contiguous in the stream).
__host__ __device__ inline WarpItems warp_items(const Geometry &g, u32 M = 1u)
{
    WarpItems w;
    if (g.tile_bins == 1u) {
        w.n_items = (g.n + (u64)kDecodeChunk - 1) / (u64)kDecodeChunk;
        w.max_bins = ((u32)kDecodeChunk - 2u) / g.L_T + 2u;
    } else {
        w.n_items = (g.n_tiles + M - 1u) / M;
        w.max_bins = M * g.tile_bins;
    }
    return w;
}

// Tiles of 80 bins of 8-bit words (L_T = 48, 49, 50) go in pairs: 160 bins split between five decoding
// warps give every lane of a warp a bin, and a warp's run of words per learner is long enough to
// spread the per-learner set-up (counts to offsets, flags) over six 32-word steps instead of four.
#ifndef ADACOMP_PAIR_MIN_TILES
#define ADACOMP_PAIR_MIN_TILES 256
#endif
constexpr long long kPairMinTiles = ADACOMP_PAIR_MIN_TILES;

// Items whose adds run a lane per bin (see warp_add_lanes_all): more than 64 bins of 8-bit words, split between
// nw warps into shares of a multiple of 4 and at most 32 bins, the item's run of counts a multiple of 16 bytes.
__host__ __device__ inline bool lanes_shape(u32 item_bins, u32 nw, u32 word_bytes)
{
    const u32 nb = item_bins / nw;
    return word_bytes == 1u && item_bins > 64u && item_bins % nw == 0u && (nb & 3u) == 0u && nb <= 32u && (item_bins & 15u) == 0u;
}
__host__ __device__ inline bool pair_path(const Geometry &g)
{
    // (small tensors keep single tiles: more items to spread over the SMs)
    return g.w == 1u && g.tile_bins == 80u && g.tile_elems <= (u32)kDecodeChunk && g.n_tiles >= (u64)kPairMinTiles;
}

// A CTA's work items in turn: it takes every stride-th.  Where items are tiles, `tile` is all there is to
// one.  Where they are 4096 output elements (L_T > 1000), `tile` is the bin (= tile) of the item's first
// element and `at` that element's place in the bin.  (Stepped, not divided: a 64-bit division per item and
// warp costs more than a small item.)
// (32 bits do: the warp path takes tensors of less than 2^40 elements)
struct ItemAt {
    u32 v, tile, at;
};
struct ItemStep {
    u32 items, tiles, at, L_T;
};
__device__ inline void next_item(ItemAt &p, const ItemStep &st)
{
    p.v += st.items;
    p.tile += st.tiles;
    p.at += st.at;
    if (p.at >= st.L_T) {
        p.at -= st.L_T;
        p.tile++;
    }
}
// Bins that `len` (> 0) elements touch, the first of them element `at` of its bin.
__device__ inline u32 bins_touched(u32 at, u32 len, u32 L_T)
{
    u32 last = at + len - 1u, bins = 1u;
    while (last >= L_T) {
        last -= L_T;
        bins++;
    }
    return bins;
}

// Room of one learner's bin counts of a tile in a slot.  The counts are bulk-copied from the
// 16-byte boundary at or below their first byte, so a run that is not a multiple of 16 bytes
// starts up to 15 bytes into its room.
template <typename Word>
__device__ inline u32 count_room(int TB)
{
    const u32 run = (u32)TB * (u32)sizeof(Word);
    return run % 16u == 0 ? run : (u32)align_up(run + 15u, 16);
}

// Lays the slots out (see WarpDecSmem), then decodes.
template <typename Word, bool MULTI, int OPT, int NW, bool ONE, int M>
__device__ void decode_warps(const DecodeArgs &a, const Geometry &geo, float *s_acc, WarpDecSmem<NW> &ws,
                             const float *s_scale, const u64 *s_nsel, float *s_wv);

//   s_wv   (OPT != 0) shared memory for a tile of weights, a tile of momentum and (Adam) a tile of second moments
template <typename Word, int OPT, int NW, bool ONE, int M>
__device__ void decode_warps_any(const DecodeArgs &a, const Geometry &geo, float *s_acc, WarpDecSmem<NW> &ws,
                                 const float *s_scale, const u64 *s_nsel, float *s_wv)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const WarpItems wi = warp_items(geo, (u32)M);
    const int TB = (int)wi.max_bins;
    const u32 count_bytes = count_room<Word>(TB);
    const u32 k8 = (a.k + 7u) & ~7u;
    const u32 meta_bytes = kSlotHead + 4u * k8;                    // slot header + cnt[k8] + head[k8]
    if (tid == 0) {
        for (int s = 0; s < kSlots; s++) {
            mbar_init(&ws.full[s], 32);         // every lane of the loader arrives, with or without bytes to expect
            mbar_init(&ws.empty[s], NW);        // every decoding warp arrives
        }
        for (int w = 0; w < NW; w++) mbar_init(&ws.wv_full[w], 1);
        ws.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < M * kDecodeChunk; i += blockDim.x) s_acc[i] = 0.f;
    if (warp == NW) {
        // the learners' regions: counts, then room for 1.5 times a tile's average words + slack
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const u32 l = (u32)lane + 32u * h;
            if (l < a.k) {
                // (an item of 4096 elements brings the words of the bins at its ends whole: L_T more elements, on average)
                const u64 per = s_nsel[l] / wi.n_items, avg = ONE ? per + per * geo.L_T / (u64)kDecodeChunk : per;
                const u64 cap = min(ONE ? (u64)wi.max_bins * geo.L_T : (u64)M * geo.tile_elems, avg + avg / 2 + 64);
                // (a learner alone always fits a slot; tiles of more than 4096 elements can have more words than that)
                ws.wcap[l] = (unsigned short)min(align_up(cap * sizeof(Word) + 16, 16), (u64)((kSlotMax - meta_bytes - count_bytes) & ~15u));
            }
        }
        __syncwarp();
        if (lane == 0) {
            // rounds: learners in order, as many per round as fit a slot (any one learner fits)
            u32 r = 0, used = meta_bytes, most = 0, r0 = 0;
            for (u32 l = 0; l < a.k; l++) {
                const u32 need = count_bytes + ws.wcap[l];
                if (used + need > kSlotMax && l > r0) {
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
            ws.rcount[r] = (unsigned char)(a.k - r0);
            ws.n_rounds = r + 1u;
            ws.slot_bytes = most;
            ws.n_slots = min((u32)kSlots, ring_bytes(NW) / most);
        }
    }
    __syncthreads();
    if (ws.n_rounds > 1u) decode_warps<Word, true, OPT, NW, ONE, M>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
    else decode_warps<Word, false, OPT, NW, ONE, M>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
}

// MULTI: a tile takes several rounds (the learners' regions do not fit one slot together).
// OPT: 0 the finished share goes to a.dst; 1 (SGD) / 2 (Adam) it feeds the optimizer step of a.ep instead.
// NW: decoding warps (warp NW is the loader); each owns 1/NW of the tile's bins ("quarter" below, whatever NW is).
// ONE: tiles of one bin (L_T > 1000): an item is 4096 output elements (see WarpItems) and each warp owns 1/NW of them.
// M: tiles of the stream per item (see warp_items); an item is decoded as one tile of M * tile_bins bins.
template <typename Word, bool MULTI, int OPT, int NW, bool ONE, int M>
__device__ void decode_warps(const DecodeArgs &a, const Geometry &geo, float *s_acc, WarpDecSmem<NW> &ws,
                             const float *s_scale, const u64 *s_nsel, float *s_wv)
{
    static_assert(M == 1 || !ONE, "items of several tiles are for tiles of more than one bin");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const WarpItems wi = warp_items(geo, (u32)M);
    const int TB = (int)wi.max_bins;                               // bins of an item (ONE: at most)
    const u32 L_T = geo.L_T;
    const u32 item_len = (u32)M * geo.tile_elems;                  // (!ONE) output elements of an item
    const u32 count_bytes = count_room<Word>(TB);                  // room of a learner's bin counts in a slot
    const u64 first = blockIdx.x, stride = gridDim.x, n_items = wi.n_items;
    const u64 my_tiles = n_items > first ? (n_items - first + stride - 1) / stride : 0;     // items of this CTA
    const u32 k8 = (a.k + 7u) & ~7u;
    unsigned char *const ring = reinterpret_cast<unsigned char *>(ws.ring);
    constexpr u32 full_mask = 0xffffffffu;

    const u32 NR = MULTI ? ws.n_rounds : 1u, slot_bytes = ws.slot_bytes, S = ws.n_slots;

    if (warp == NW) {
        // ================================ loader warp ================================
        // An item is one round of one tile; lane j (and j + 32) looks after the j-th learner of the
        // round.  The learners' directory entries are read two items ahead.
        // With them travels (ONE) the item's first bin and {place of the item's first element in that bin,
        // bins of the item << 16, offset of the counts in their room << 24}: the loader steps through the
        // bins once, for the item two ahead.
        u64 da0[2] = {0, 0}, da1[2] = {0, 0}, db0[2] = {0, 0}, db1[2] = {0, 0};
        u32 ta = 0, ia = 0, tb = 0, ib = 0;
        const u32 last_item = (u32)(n_items - 1), last_len = (u32)(geo.n - (n_items - 1) * (u64)kDecodeChunk);   // (ONE)
        auto load_dir = [&](u64 tile, const ItemAt &p, u32 r, bool valid, u64 *d0, u64 *d1, u32 &t, u32 &info) {
            u32 tiles = 1u;             // tiles of the item (ONE: each a bin)
            if (!ONE && M > 1 && valid) {
                tile *= (u64)M;         // the item's first tile
                tiles = (u32)min((u64)M, geo.n_tiles - tile);
            }
            if (ONE && valid) {
                tiles = bins_touched(p.at, p.v == last_item ? last_len : (u32)kDecodeChunk, L_T);
                t = p.tile;
                info = p.at | (tiles << 16) | (((p.tile * (u32)sizeof(Word)) & 15u) << 24);
                tile = p.tile;
            }
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const u32 j = (u32)lane + 32u * h;
                if (valid && j < (MULTI ? (u32)ws.rcount[r] : a.k)) {
                    const u64 *dir = reinterpret_cast<const u64 *>(a.stream[(MULTI ? (u32)ws.rfirst[r] : 0u) + j] + geo.tile_off_at);
                    d0[h] = dir[tile];
                    d1[h] = dir[tile + tiles];
                }
            }
        };
        // (no division in the loops: slot, use count and the look-ahead position step along)
        // the item two ahead: its tile (ONE: its place, stepped in elements: the stride as whole bins and a rest) and round
        u64 ptile = first, pit = 0;
        const ItemStep item_step = {(u32)stride, (u32)(stride * (u64)kDecodeChunk / L_T), (u32)(stride * (u64)kDecodeChunk % L_T), L_T};
        ItemAt pa = {(u32)first, (u32)(first * (u64)kDecodeChunk / L_T), (u32)(first * (u64)kDecodeChunk % L_T)};
        u32 pr = 0;
        auto step_ahead = [&]() {
            if (++pr == NR) {
                pr = 0;
                if (ONE) next_item(pa, item_step);
                else ptile += stride;
                pit++;
            }
        };
        load_dir(ptile, pa, pr, pit < my_tiles, da0, da1, ta, ia);
        step_ahead();
        load_dir(ptile, pa, pr, pit < my_tiles, db0, db1, tb, ib);
        step_ahead();
        u32 my_coff[2] = {0, 0}, my_wcap[2] = {0, 0};       // one round: the lane's learners stay the same
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const u32 l = (u32)lane + 32u * h;
            if (!MULTI && l < a.k) {
                my_coff[h] = ws.coff[l];
                my_wcap[h] = ws.wcap[l];
            }
        }
        u64 issued = 0;                 // copies were started for items [0, issued)
        u32 s = 0, use = 0;             // the item's slot; how many times the slot was used before
        u64 tile = first;
        bool failed = false;
        for (u64 it = 0; it < my_tiles && !failed; it++, tile += stride) {
            for (u32 r = 0; r < NR; r++, s = s + 1u == S ? 0u : s + 1u, use += s == 0u) {
                const u64 bin0 = ONE ? (u64)ta : tile * (u64)TB;
                const u32 live = ONE ? (ia >> 16) & 0xffu : (u32)min((u64)TB, geo.n_bins - bin0);
                const u32 item_elems = ONE ? live * L_T : item_len;            // more words than that are an error
                // the item's bin counts start `clead` bytes behind a 16-byte boundary: the copy starts at the boundary
                const u32 clead = ONE ? ia >> 24 : (u32)(bin0 * sizeof(Word)) & 15u;
                const u32 cbytes = (u32)align_up(clead + live * (u32)sizeof(Word), 16);
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
                const u32 l0 = MULTI ? ws.rfirst[r] : 0u, nl = MULTI ? ws.rcount[r] : a.k;
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
                        ok = da1[h] >= da0[h] && da1[h] - da0[h] <= item_elems && da1[h] <= s_nsel[l];
                        const u32 cnt = ok ? (u32)(da1[h] - da0[h]) : 0u;
                        src[h] = (u64)(uintptr_t)(a.stream[l] + geo.payload_at) + da0[h] * sizeof(Word);
                        const u32 head = (u32)(src[h] & 15u);
                        wbytes[h] = cnt ? (u32)align_up(head + cnt * sizeof(Word), 16) : 0u;
                        fit = wbytes[h] <= (MULTI ? (u32)ws.wcap[l] : my_wcap[h]);
                        coff[h] = MULTI ? (u32)ws.coff[l] : my_coff[h];
                        m_cnt[j] = (unsigned short)cnt;
                        m_head[j] = (unsigned short)head;
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
                    if (ONE) reinterpret_cast<u32 *>(sl)[2] = ia;
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
                        bulk_load(sl + coff[h], a.stream[l0 + j] + geo.bin_cnt_at + (bin0 * sizeof(Word) - clead), cbytes, &ws.full[s]);
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
                }
                ta = tb;
                ia = ib;
                load_dir(ptile, pa, pr, pit < my_tiles, db0, db1, tb, ib);
                step_ahead();
            }
        }
        if (*reinterpret_cast<volatile u32 *>(&ws.abort)) {
            // after a timeout the copies already started must land (or time out in turn) before
            // this CTA's shared memory is given back
            for (u64 j = issued > S ? issued - S : 0; j < issued; j++) mbar_wait(&ws.full[j % S], (u32)(j / S) & 1u);    // (rare)
        }
        return;
    }

    // =============================== decoding warps ===============================
    const int nb = ONE ? 1 : TB / NW;               // bins of a warp (the launcher picks NW to divide tile_bins)
    const int b0 = warp * nb;
    const u32 quarter = ONE ? (u32)kDecodeChunk / NW : (u32)nb * L_T;   // output elements of a warp
    const u32 acc_at = smem_addr(s_acc) + (u32)warp * quarter * 4u;
    float *const my_acc = s_acc + (u32)warp * quarter;
    u32 *const tmp = ws.tmp[warp];
    const bool vec_store = (quarter & 3u) == 0 && (ONE || (geo.tile_elems & 3u) == 0);
    // tiles of at most 64 bins: G lanes share a bin
    const bool by_bin = M == 1 && (sizeof(Word) == 2 || TB <= 64);     // (16-bit words: L_T >= 65, at most 60 bins)
    const int G = nb <= 32 ? 32 / nb : 1;           // (need not be a power of two: 5 bins take 6 lanes each)
    // tiles of more than 64 bins of 8-bit words whose counts line up with 32-bit loads: a lane per bin
    // (not in the plain decoder of single tiles: at its 64 registers the lane-per-bin loop spills and is slower than by word)
    const bool lanes_ok = (M == 2 || OPT != 0) && lanes_shape((u32)TB, (u32)NW, sizeof(Word));
    const int my_local = lane / G, my_r = lane % G;
    const int my_bin = my_local < nb ? b0 + my_local : TB;
    const u32 mine_at = smem_addr(s_acc) + (u32)my_bin * L_T * 4u;
    u32 bad = 0;
    u32 s = 0, use = 0;                             // the item's slot; how many times the slot was used before
    u64 v = first;                                  // the item
    bool failed = false;
    // (OPT != 0) the warp's quarters of the staged weights, momentum and second moments
    float *const wq = s_wv + (u32)warp * quarter, *const vq = s_wv + kDecodeChunk + (u32)warp * quarter;
    float *const uq = s_wv + 2 * kDecodeChunk + (u32)warp * quarter;
    u32 wv_use = 0;                                 // fetches of the quarters so far
    for (u64 it = 0; it < my_tiles; it++, v += stride) {
        // (ONE: the loader, which steps through the bins anyway, leaves these in the slot's header)
        u32 live = ONE ? 0u : (u32)min((u64)TB, geo.n_bins - v * (u64)TB);      // bins of the item
        u32 clead = ONE ? 0u : (u32)(v * (u64)TB * sizeof(Word)) & 15u;          // where the counts start in their room (see the loader)
        u32 lo = 0;                                 // (ONE) the warp's first element, counted from the first bin's
        const u64 out0 = v * (u64)(ONE ? (u32)kDecodeChunk : item_len) + (u64)warp * quarter;
        const u32 len = out0 < geo.n ? (u32)min((u64)quarter, geo.n - out0) : 0u;
        const bool whole = vec_store && len == quarter;
        if (OPT != 0 && whole && lane == 0) {
            // the warp's quarters of the optimizer's arrays travel while the words are added
            bulk_wait_read_all();                   // the previous tile's copies out have read the buffers
            mbar_arrive_expect_tx(&ws.wv_full[warp], (OPT == 2 ? 3u : 2u) * quarter * 4u);
            bulk_load(wq, a.ep.weights + out0, quarter * 4u, &ws.wv_full[warp]);
            bulk_load(vq, a.ep.momentum + out0, quarter * 4u, &ws.wv_full[warp]);
            if (OPT == 2) bulk_load(uq, a.ep.second + out0, quarter * 4u, &ws.wv_full[warp]);
        }
        for (u32 r = 0; r < NR; r++, s = s + 1u == S ? 0u : s + 1u, use += s == 0u) {
            if (!mbar_wait(&ws.full[s], use & 1u)) {
                ws.abort = 1;
                bad |= ADACOMP_DEV_TIMEOUT;
                failed = true;
                break;
            }
            const unsigned char *sl = ring + s * slot_bytes;
            const u32 l0 = MULTI ? ws.rfirst[r] : 0u, nl = MULTI ? ws.rcount[r] : a.k;
            const u32 staged = min(reinterpret_cast<const u32 *>(sl)[0], nl);
            if (warp == 0) bad |= reinterpret_cast<const u32 *>(sl)[1];
            if (ONE) {
                const u32 info = reinterpret_cast<const u32 *>(sl)[2];
                lo = (info & 0xffffu) + (u32)warp * quarter;
                live = (info >> 16) & 0xffu;
                clead = info >> 24;
            }
            const unsigned short *m_cnt = reinterpret_cast<const unsigned short *>(sl + kSlotHead), *m_head = m_cnt + k8;
            const u32 sl_at = smem_addr(sl);

            // ---- the round's learners whose words wait in the slot ----
            if (lanes_ok && (u32)(b0 + nb) <= live) {
                bad |= warp_add_lanes_all(sl_at, ws.coff, m_cnt, m_head, s_scale, l0, staged, count_bytes, b0, nb, L_T, acc_at, lane);
                __syncwarp();
            } else
            // (the other shapes: four learners at a time)
            for (u32 g0 = 0; g0 < staged; g0 += kRoundMax) {
                const int R = (int)min((u32)kRoundMax, staged - g0);
                GroupSrc<u32> src = {0u, 0u, 0u, 0u};
                if (lane < R) {
                    const u32 j = g0 + (u32)lane, l = l0 + j;
                    src.counts = sl_at + ws.coff[l] + clead;
                    src.words = sl_at + ws.coff[l] + count_bytes + m_head[j];
                    src.limit = m_cnt[j];
                    src.sbits = __float_as_uint(s_scale[l]);
                }
                if (ONE) bad |= warp_add_group_flat<Word, true, u32>(src, R, live, lo, len, L_T, acc_at, lane);
                else if (by_bin) bad |= warp_add_group_by_bin<Word, true, u32>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else bad |= warp_add_group<Word, true, u32>(src, R, b0, nb, live, L_T, acc_at, tmp, lane);
            }
            if (lane == 0) mbar_arrive(&ws.empty[s]);   // (the group's last __syncwarp orders the warp's reads before it)

            // ---- the round's others: read from global memory ----
            for (u32 g0 = staged; g0 < nl; g0 += kRoundMax) {
                const int R = (int)min((u32)kRoundMax, nl - g0);
                GroupSrc<u64> src = {0ull, 0ull, 0u, 0u};
                bool ok = true;
                if (lane < R) {
                    const u32 l = l0 + g0 + (u32)lane;
                    const unsigned char *st = a.stream[l];
                    const u64 *dir = reinterpret_cast<const u64 *>(st + geo.tile_off_at);
                    // (ONE: the first tile, that is bin, of the item, by division on this rare path)
                    const u64 tile = ONE ? (v * (u64)kDecodeChunk) / L_T : v * (u64)M, bin0 = ONE ? tile : v * (u64)TB;
                    const u64 w0 = dir[tile], w1 = dir[tile + (ONE ? live : (u32)min((u64)M, geo.n_tiles - tile))];
                    ok = w1 >= w0 && w1 - w0 <= (ONE ? live * L_T : item_len) && w1 <= s_nsel[l];
                    src.counts = (u64)__cvta_generic_to_global(st + geo.bin_cnt_at) + bin0 * sizeof(Word);
                    src.words = (u64)__cvta_generic_to_global(st + geo.payload_at) + (ok ? w0 : 0) * sizeof(Word);
                    src.limit = ok ? (u32)(w1 - w0) : 0u;
                    src.sbits = __float_as_uint(s_scale[l]);
                }
                if (__any_sync(full_mask, !ok)) bad |= ADACOMP_DEV_BAD_STREAM;
                if (ONE) bad |= warp_add_group_flat_global<Word>(src, R, live, lo, len, L_T, acc_at, lane);
                else if (by_bin) bad |= warp_add_group_by_bin_global<Word>(src, R, TB, live, L_T, my_bin, my_r, G, mine_at, lane);
                else bad |= warp_add_group_global<Word>(src, R, b0, nb, live, L_T, acc_at, tmp, lane);
            }
        }
        if (failed) break;

        // ---- store the warp's quarter of the tile (and leave it zeroed for the next one) ----
        if (OPT != 0) {
            // averageGradients() + updateWeights() on the warp's quarter, in shared memory; two bulk
            // copies take the new weights and momentum back
            if (whole) {
                if (!mbar_wait(&ws.wv_full[warp], wv_use & 1u)) {
                    ws.abort = 1;
                    bad |= ADACOMP_DEV_TIMEOUT;
                    break;
                }
                wv_use++;
                float4 *w4 = reinterpret_cast<float4 *>(wq), *v4 = reinterpret_cast<float4 *>(vq);
                float4 *s4 = reinterpret_cast<float4 *>(my_acc);
                const int n4 = (int)(quarter >> 2);
                float4 *u4 = reinterpret_cast<float4 *>(uq);
                for (int at = lane; at < n4; at += 32) {
                    float4 w = w4[at], v = v4[at];
                    if (OPT == 2) {
                        float4 u = u4[at];
                        adam_step4(s4[at], w, v, u, a.ep);
                        u4[at] = u;
                    } else {
                        sgd_step4(s4[at], w, v, a.ep);
                    }
                    s4[at] = make_float4(0.f, 0.f, 0.f, 0.f);
                    v4[at] = v;
                    w4[at] = w;
                }
                fence_async_smem();                 // this lane's results, for the copy engine
                __syncwarp();
                if (lane == 0) {
                    bulk_store(a.ep.weights + out0, wq, quarter * 4u);
                    bulk_store(a.ep.momentum + out0, vq, quarter * 4u);
                    if (OPT == 2) bulk_store(a.ep.second + out0, uq, quarter * 4u);
                    bulk_commit();
                }
            } else {
                for (u32 i = lane; i < quarter; i += 32) {
                    if (i < len) {
                        float w = a.ep.weights[out0 + i], v = a.ep.momentum[out0 + i];
                        if (OPT == 2) {
                            float u = a.ep.second[out0 + i];
                            adam_step(my_acc[i], w, v, u, a.ep);
                            a.ep.second[out0 + i] = u;
                        } else {
                            sgd_step(my_acc[i], w, v, a.ep);
                        }
                        a.ep.momentum[out0 + i] = v;
                        a.ep.weights[out0 + i] = w;
                    }
                    my_acc[i] = 0.f;
                }
            }
        } else if (whole) {
            // one bulk copy (TMA) takes the quarter from shared memory: the warp's own stores stay
            // out of the way of everybody's shared-memory traffic
            fence_async_smem();                     // this lane's adds, for the copy engine
            __syncwarp();
            if (lane == 0) {
                bulk_store(a.dst + out0, my_acc, quarter * 4u);
                bulk_commit();
                bulk_wait_read_all();               // shared memory has been read: it can be zeroed
            }
            __syncwarp();
            float4 *s4 = reinterpret_cast<float4 *>(my_acc);
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
            if (quarter == 1000u) {
#pragma unroll
                for (int i = 0; i < 8; i++)
                    if (i < 7 || lane < 26) s4[lane + 32 * i] = zero;
            } else {
                for (int at = lane; at < (int)(quarter >> 2); at += 32) s4[at] = zero;
            }
        } else {
            for (u32 i = lane; i < quarter; i += 32) {
                if (i < len) a.dst[out0 + i] = my_acc[i];
                my_acc[i] = 0.f;
            }
        }
        __syncwarp();                               // zeroed before the next tile's adds
    }
    if (lane == 0) bulk_wait_all();                // the last copies leave shared memory before the CTA ends
    if (bad) raise_status(bad);
}

// Any tile shape (also tiles larger than one output chunk).
template <typename Word>
__device__ void decode_generic(const DecodeArgs &a, const Geometry &geo, DecodeSmem &sm)
{
    const int tid = threadIdx.x;
    const int TB = (int)geo.tile_bins;
    float *s_acc = sm.acc;
    u32 *s_pre = sm.g.pre;
    const u32 chunks_per_tile = (geo.tile_elems + kDecodeChunk - 1) / kDecodeChunk;
    const u64 items = geo.n_tiles * chunks_per_tile;
    for (int i = tid; i < kDecodeChunk; i += kDecodeThreads) s_acc[i] = 0.f;
    consumer_barrier();
    for (u64 item = blockIdx.x; item < items; item += gridDim.x) {
        const u64 tile = item / chunks_per_tile;
        const u32 c_lo = (u32)(item % chunks_per_tile) * kDecodeChunk;     // within the tile
        const u32 c_hi = min(c_lo + (u32)kDecodeChunk, geo.tile_elems);
        const u64 base = tile * (u64)geo.tile_elems;
        for (u32 l = 0; l < a.k; l++) {
            const unsigned char *s = a.stream[l];
            const u64 *tile_off = reinterpret_cast<const u64 *>(s + geo.tile_off_at);
            const u64 off0 = tile_off[tile];
            const u32 cnt = (u32)(tile_off[tile + 1] - off0);
            if (cnt == 0) continue;
            if (cnt > geo.tile_elems || off0 + cnt > reinterpret_cast<const u64 *>(s)[5]) {
                if (tid == 0) raise_status(ADACOMP_DEV_BAD_STREAM);
                continue;
            }
            const float scale = __uint_as_float(reinterpret_cast<const u32 *>(s)[12]);
            const Word *bin_cnt = reinterpret_cast<const Word *>(s + geo.bin_cnt_at);
            const Word *payload = reinterpret_cast<const Word *>(s + geo.payload_at);
            const u64 bin0 = tile * (u64)TB;
            // the tile's bins are scanned kGenericSegBins at a time; `done` words precede the pass
            u32 done = 0;
            for (int seg = 0; seg < TB; seg += kGenericSegBins) {
                const int bins = min(kGenericSegBins, TB - seg);
                u32 words = cnt;                               // one bin per tile: all words are its
                if (TB > 1) {
                    for (int b = tid; b < bins; b += kDecodeThreads)
                        s_pre[b] = bin0 + seg + b < geo.n_bins ? (u32)bin_cnt[bin0 + seg + b] : 0u;
                    consumer_barrier();
                    block_exclusive_scan(s_pre, bins, sm.g.tmp, true);
                    words = s_pre[bins];
                }
                if (done + words > cnt) {                       // counts and directory disagree
                    if (tid == 0) raise_status(ADACOMP_DEV_BAD_STREAM);
                    consumer_barrier();
                    break;
                }
                for (u32 j = tid; j < words; j += kDecodeThreads) {
                    const u32 word = payload[off0 + done + j];
                    const u32 code = word & 3u;
                    if (code == 0u) continue;
                    if (code == 2u) { raise_status(ADACOMP_DEV_RESERVED_CODE); continue; }
                    const int b = seg + (TB > 1 ? bin_of_word(s_pre, bins, j) : 0);
                    const u32 idx = word >> 2;
                    const u32 at = (u32)b * geo.L_T + idx;          // within the tile
                    if (idx >= geo.L_T || base + at >= geo.n) { raise_status(ADACOMP_DEV_BAD_STREAM); continue; }
                    if (at < c_lo || at >= c_hi) continue;
                    // one word per element per learner: no two threads meet on one address here
                    const float v = s_acc[at - c_lo];
                    s_acc[at - c_lo] = code == 3u ? __fsub_rn(v, scale) : __fadd_rn(v, scale);
                }
                done += words;
                consumer_barrier();
            }
        }
        const u64 out0 = base + c_lo;
        const u32 len = out0 < geo.n ? (u32)min((u64)(c_hi - c_lo), geo.n - out0) : 0u;
        store_tile(a.dst, out0, len, s_acc, a.ep);
        consumer_barrier();
    }
}

// Tiles the warp path takes: 4..96 bins, a multiple of 4, at most 4096 elements (L_T = 41..1000); and the
// tiles of one bin (L_T > 1000).
__host__ __device__ inline bool warp_path(const Geometry &g)
{
    if (g.tile_bins == 1u) return g.L_T > 1000u && g.n < (1ull << 40);
    return g.tile_bins >= 4u && g.tile_bins <= (u32)kSmallBins && g.tile_bins % 4u == 0 && g.tile_elems <= (u32)kDecodeChunk;
}

// Every CTA of a decode kernel reads and cross-checks the k headers itself: the decision is
// uniform.  Returns false when this CTA has nothing to do (bad headers, raised by CTA 0; or a
// CTA beyond the tensor's last work item); else the shape in L_T and n, and the streams' scales
// and word totals in shared memory (behind a barrier).
__device__ inline bool decode_headers(const DecodeArgs &a, int *s_bad, float *s_scale, u64 *s_nsel, u32 &L_T, u64 &n)
{
    const u32 *h0 = reinterpret_cast<const u32 *>(a.stream[0]);
    L_T = h0[2];
    n = reinterpret_cast<const u64 *>(a.stream[0])[2];
    // (CTA 0 stays to report bad headers)
    if (blockIdx.x > 0 && L_T >= 1u && L_T <= ADACOMP_MAX_L_T && blockIdx.x >= decode_items(n, L_T)) return false;
    if (threadIdx.x == 0) *s_bad = a.hint_L_T != 0 && (a.hint_L_T != L_T || a.hint_n != n);
    __syncthreads();
    if (threadIdx.x < a.k) {
        const u32 *h = reinterpret_cast<const u32 *>(a.stream[threadIdx.x]);
        const u64 *h64 = reinterpret_cast<const u64 *>(h);
        bool ok = h[0] == kMagic && (h[1] & 0xffffu) == 1u && h[2] == L_T && h64[2] == n &&
                  L_T >= 1u && L_T <= ADACOMP_MAX_L_T;
        if (ok) {
            const Geometry g = make_geometry(n, L_T);
            ok = ((h[1] >> 16) & 0xffu) == g.w && h[3] == g.tile_bins && h64[3] == g.n_bins &&
                 h64[4] == g.n_tiles && h64[5] <= n;
        }
        if (!ok) *s_bad = 1;
        s_scale[threadIdx.x] = __uint_as_float(h[12]);
        s_nsel[threadIdx.x] = h64[5];
    }
    __syncthreads();
    if (*s_bad) {
        if (threadIdx.x == 0 && blockIdx.x == 0) raise_status(ADACOMP_DEV_HEADER_MISMATCH);
        return false;
    }
    return true;
}

// The decoder is three kernels, so that each gets the registers its path needs: decode_sum_warps
// takes the shapes of warp_path() (its ONE form the tiles of one bin, its other form the rest) and
// returns at once for any other, decode_sum the reverse.  A caller that knows the shape launches
// the one that works; one that does not launches all three.
// dynamic shared memory of decode_sum_warps<OPT>: a tile per array of the optimizer
constexpr u32 opt_smem_bytes(int opt) { return opt == 0 ? 0u : (opt == 2 ? 3u : 2u) * kDecodeChunk * 4u; }
constexpr u32 kPairSmemBytes = 2u * kDecodeChunk * 4u;     // dynamic shared memory of the M = 2 kernel: its output tile

// NW decoding warps and the loader warp: 4 for plain decoding; with an optimizer step, whose staged tiles
// leave room for fewer CTAs per SM, 8 where they divide the tile's bins (more warps to hide the adds' latency).
// ONE: the kernel of the tiles of one bin (L_T > 1000): a kernel of its own, so that its registers are
// allotted apart from the other shapes'.
// (The one-bin form runs four CTAs per SM: with 96 registers it keeps everything in registers, and its few
// words per item leave it less to hide than the other shapes have; measured 3 % faster than six CTAs of 64.)
// M = 2 (plain decoding only): the pairs of 80-bin tiles of pair_path(), five decoding warps, four CTAs per SM; the
// output tile of 2 x 4096 elements is dynamic shared memory.
template <int OPT, int NW, bool ONE = false, int M = 1>
__global__ void __launch_bounds__((NW + 1) * 32, M == 2 ? 4 : OPT == 0 ? (ONE ? 4 : kWarpsPerSm) : OPT == 1 ? 3 : 2)
decode_sum_warps(DecodeArgs a)
{
    static_assert(!ONE || NW == 4, "tiles of one bin are split between four warps");
    static_assert(M == 1 || (M == 2 && OPT == 0 && !ONE && NW == 5), "pairs of tiles: plain decoding, five warps");
    __shared__ __align__(16) float s_acc_static[M == 1 ? kDecodeChunk : 4];
    __shared__ __align__(16) WarpDecSmem<NW> ws;
    __shared__ u64 s_nsel[ADACOMP_MAX_STREAMS];
    __shared__ float s_scale[ADACOMP_MAX_STREAMS];
    __shared__ int s_bad;
    u32 L_T;
    u64 n;
    if (!decode_headers(a, &s_bad, s_scale, s_nsel, L_T, n)) return;
    const Geometry geo = make_geometry(n, L_T);
    // (the launcher picks NW from the shape it was given: a divisor of the tile's bins; 4 for tiles of one bin)
    if (!warp_path(geo) || ONE != (geo.tile_bins == 1u) || (!ONE && (M * geo.tile_bins) % (u32)NW != 0)) return;
    // plain decoding: the shapes of pair_path() belong to the M = 2 kernel, all others to the M = 1 kernels
    if (OPT == 0 && !ONE && (M == 2) != (a.pairs != 0u && pair_path(geo))) return;
    // (the rounds are laid out inside; the first thing decode_warps does after that is uniform)
    extern __shared__ __align__(16) float s_dyn[];     // (OPT != 0) the optimizer's staged tiles; (M == 2) the output tile
    float *const s_wv = OPT ? s_dyn : nullptr;
    float *const s_acc = M == 1 ? s_acc_static : s_dyn;
    if constexpr (ONE) {
        decode_warps_any<unsigned short, OPT, NW, true, 1>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
    } else if constexpr (M == 2) {
        decode_warps_any<unsigned char, OPT, NW, false, 2>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
    } else {
        if (geo.w == 1u) decode_warps_any<unsigned char, OPT, NW, false, 1>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
        else decode_warps_any<unsigned short, OPT, NW, false, 1>(a, geo, s_acc, ws, s_scale, s_nsel, s_wv);
    }
}

__global__ void __launch_bounds__(kDecodeThreads, 6)
decode_sum(DecodeArgs a)
{
    __shared__ __align__(16) DecodeSmem sm;
    __shared__ int s_bad;
    u32 L_T;
    u64 n;
    if (!decode_headers(a, &s_bad, sm.scale, sm.n_sel, L_T, n)) return;
    const Geometry geo = make_geometry(n, L_T);
    if (warp_path(geo)) return;
    // (what is left: tiles of 100 bins and more, L_T <= 40; and tensors beyond the warp path's 2^40 elements)
    if (geo.w == 1u) decode_generic<unsigned char>(a, geo, sm);
    else decode_generic<unsigned short>(a, geo, sm);
}

// ---------------------------------------------------------------------------------
// Batched decode-sum: many small layers in one launch.  The layer table (shapes, output and
// stream pointers) travels in the kernel parameters; every CTA builds the same tile index over
// all layers in shared memory and takes (layer, tile) items from it.  Layers of
// 42 <= L_T <= 1000 qualify (tiles of at most 4096 elements and 2..96 bins).
// ---------------------------------------------------------------------------------

constexpr int kDecBatchLayers = 192;
constexpr int kDecBatchPtrs = 2900;

struct DecodeBatchArgs {
    u32 n_layers, k;
    u64 n[kDecBatchLayers];
    u32 L_T[kDecBatchLayers];
    float *dst[kDecBatchLayers];                     // the layer's output; with `sgd` its weights
    float *aux[kDecBatchLayers];                     // with `opt`: its momentum (Adam: first moments)
    float *aux2[kDecBatchLayers];                    // Adam: its second moments
    float lr, mu, beta2, eps;
    u32 opt;                                         // 1 SGD, 2 Adam: the optimizer step takes the place of the store (see Epilogue)
    const unsigned char *stream[kDecBatchPtrs];      // [layer * k + learner]
};

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
            if (at_li != 0xffffffffu) {
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

__global__ void reset_status_kernel() { g_status = 0; }

__global__ void lazy_init_kernel(unsigned char *state, u64 n, u32 L_T)
{
    LazyHeader *lh = reinterpret_cast<LazyHeader *>(state);
    lh->magic = kLazyMagic;
    lh->L_T = L_T;
    lh->n = n;
    lh->scale = 0.f;
    lh->steps = 0;
}

// residue_flush: finish "residue = G - sign(G) * scale" for the elements the last lazy step sent,
// and clear their marks.  One thread per 25-element segment.
__global__ void __launch_bounds__(256)
lazy_flush_kernel(float *residue, unsigned char *state, u64 n, u32 L_T, u32 tile_elems)
{
    const LazyHeader *lh = reinterpret_cast<const LazyHeader *>(state);
    if (lh->magic != kLazyMagic || lh->n != n || lh->L_T != L_T) {
        if (threadIdx.x == 0 && blockIdx.x == 0) raise_status(ADACOMP_DEV_HEADER_MISMATCH);
        return;
    }
    const u32 sbits = __float_as_uint(lh->scale) & 0x7fffffffu;
    u32 *mask = reinterpret_cast<u32 *>(state + kLazyHeaderBytes);
    // segment s of tile t starts at element t * tile_elems + 25 s (tiles of 4000 elements: 25 (160 t + s))
    const u64 segs = (n + tile_elems - 1) / tile_elems * (u64)kTileSegs;
    for (u64 sgm = (u64)blockIdx.x * blockDim.x + threadIdx.x; sgm < segs; sgm += (u64)gridDim.x * blockDim.x) {
        u32 m = mask[sgm];
        if (m == 0) continue;
        mask[sgm] = 0;
        const u64 first = sgm / kTileSegs * tile_elems + sgm % kTileSegs * kSeg;
        while (m) {
            const int j = __ffs(m) - 1;
            m &= m - 1;
            const u64 i = first + j;
            if (i < n) {
                const float r = residue[i];
                residue[i] = __fsub_rn(r, __uint_as_float(sbits | (__float_as_uint(r) & 0x80000000u)));
            }
        }
    }
}

// ---------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------

// The batched warp decoder's ring of slots (dynamic shared memory).  Deeper rings for more learners were
// measured: they cost a CTA per SM and the decode of a list is bound by the warps' fixed work per learner and
// tile, so more warps beat more tiles in flight (8 learners: 0.20 ms with this ring, 0.21 ms with twice it).
constexpr u32 kBatchRingBytes = 19200u;

// The fast tile pass takes L_T = 25 * SPB for the divisors SPB of 40 but 1 (tiles of exactly 4000 elements):
// 50, 100, 125, 200, 250, 500 and 1000.
__host__ __device__ inline bool fast_L_T(u32 L_T)
{
    return L_T == 50u || L_T == 100u || L_T == 125u || L_T == 200u || L_T == 250u || L_T == 500u || L_T == 1000u;
}
// Calls f(kernel) for the fast tile pass of L_T (LAZY, BF16 as given); false when there is none.
template <bool LAZY, bool BF16, typename F>
bool with_fast_kernel(u32 L_T, F f)
{
    switch (L_T) {
    case 50u: f(tile_pass_fast<2, unsigned char, LAZY, BF16>); return true;
    case 100u: f(tile_pass_fast<4, unsigned short, LAZY, BF16>); return true;
    case 125u: f(tile_pass_fast<5, unsigned short, LAZY, BF16>); return true;
    case 200u: f(tile_pass_fast<8, unsigned short, LAZY, BF16>); return true;
    case 250u: f(tile_pass_fast<10, unsigned short, LAZY, BF16>); return true;
    case 500u: f(tile_pass_fast<20, unsigned short, LAZY, BF16>); return true;
    case 1000u: f(tile_pass_fast<40, unsigned short, LAZY, BF16>); return true;
    default: return false;
    }
}
constexpr u32 kFastL_T[] = {50u, 100u, 125u, 200u, 250u, 500u, 1000u};
// Every other L_T from 41 to 1000 (tiles of at most 96 bins, bins longer than a thread's 25 elements) takes
// the same kernel in its any-bin form (fp32 gradient), and so do the one-bin tiles of at most 4000 elements
// that start on 16-byte boundaries (L_T up to 4000, a multiple of 4).
__host__ __device__ inline bool any_fast_L_T(u32 L_T)
{
    return (L_T >= 41u && L_T <= 1000u && !fast_L_T(L_T)) || (L_T > 1000u && L_T <= (u32)kFastTile && L_T % 4u == 0);
}
template <bool LAZY, typename F>
void with_any_fast_kernel(u32 L_T, F f)
{
    if (L_T <= 64u) f(tile_pass_fast<0, unsigned char, LAZY, false>);
    else f(tile_pass_fast<0, unsigned short, LAZY, false>);
}

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    int decode_per_sm = 0;
    int decode_warps_per_sm = 0, decode_one_per_sm = 0;
    int decode_pair_per_sm = 0;         // 0: the kernel of pair_path() cannot be launched on this device
    int decode_opt_per_sm[2][2] = {{0, 0}, {0, 0}};     // [SGD, Adam][4, 8 decoding warps]; 0: unavailable on this device
    int batch_per_sm = 0;
    bool batch_fast_ready = false;      // the pipelined batch tile pass can be launched       // 0: batched pack() unavailable on this device
    int dec_batch_per_sm = 0;   // 0: batched decode unavailable on this device
    int dec_batch_warps_per_sm[3] = {0, 0, 0};      // CTAs of the batched warp decoder per SM, by optimizer form
    bool fast_ready = false;
};

DeviceInfo g_info[64];

int device_info(DeviceInfo *&out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ADACOMP_ERR_CUDA;
    DeviceInfo &d = g_info[dev];
    if (d.sms == 0) {
        int sms = 0, optin = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return ADACOMP_ERR_CUDA;
        d.smem_optin = optin;
        int per_sm = 1;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum, kDecodeThreads, 0);
        d.decode_per_sm = per_sm < 1 ? 1 : per_sm;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum_warps<0, 4>, kDecodeLaunch, 0);
        d.decode_warps_per_sm = per_sm < 1 ? 1 : per_sm;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum_warps<0, 4, true>, kDecodeLaunch, 0);
        d.decode_one_per_sm = per_sm < 1 ? 1 : per_sm;
        auto opt_ready = [&](auto kernel, int threads, u32 smem) -> int {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
            int per = 0;
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, kernel, threads, smem);
            return per;
        };
        d.decode_pair_per_sm = opt_ready(decode_sum_warps<0, 5, false, 2>, 6 * 32, kPairSmemBytes);
        d.decode_opt_per_sm[0][0] = opt_ready(decode_sum_warps<1, 4>, 5 * 32, opt_smem_bytes(1));
        d.decode_opt_per_sm[0][1] = opt_ready(decode_sum_warps<1, 8>, 9 * 32, opt_smem_bytes(1));
        d.decode_opt_per_sm[1][0] = opt_ready(decode_sum_warps<2, 4>, 5 * 32, opt_smem_bytes(2));
        d.decode_opt_per_sm[1][1] = opt_ready(decode_sum_warps<2, 8>, 9 * 32, opt_smem_bytes(2));
        // (the kernels of the one-bin tiles: same shared memory and launch bounds as their four-warp siblings)
        if (!opt_ready(decode_sum_warps<1, 4, true>, 5 * 32, opt_smem_bytes(1))) d.decode_opt_per_sm[0][0] = 0;
        if (!opt_ready(decode_sum_warps<2, 4, true>, 5 * 32, opt_smem_bytes(2))) d.decode_opt_per_sm[1][0] = 0;
        const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
        const int bytes = (int)FastSmem::kBytes;
        bool ready = true;
        auto allow = [&](auto kernel) { ready = ready && cudaFuncSetAttribute(kernel, at, bytes) == cudaSuccess; };
        for (u32 L_T : kFastL_T) {
            with_fast_kernel<false, false>(L_T, allow);
            with_fast_kernel<true, false>(L_T, allow);
            with_fast_kernel<false, true>(L_T, allow);
        }
        with_any_fast_kernel<false>(41u, allow);
        with_any_fast_kernel<false>(65u, allow);
        with_any_fast_kernel<true>(41u, allow);
        with_any_fast_kernel<true>(65u, allow);
        d.fast_ready = ready;
        if (cudaFuncSetAttribute(batch_tile_pass<kBatchMax>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kBatchSmemBytes) == cudaSuccess &&
            cudaFuncSetAttribute(batch_tile_pass<kBatchSmall>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kBatchSmemBytes) == cudaSuccess) {
            int per = 0;
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, batch_tile_pass<kBatchMax>, kGenericThreads,
                                                          kBatchSmemBytes);
            d.batch_per_sm = per;
        }
        d.batch_fast_ready = d.fast_ready &&
                             cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, false>, at, bytes) == cudaSuccess &&
                             cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, false>, at, bytes) == cudaSuccess &&
                             cudaFuncSetAttribute(batch_tile_pass_fast<kBatchMax, true>, at, bytes) == cudaSuccess &&
                             cudaFuncSetAttribute(batch_tile_pass_fast<kBatchSmall, true>, at, bytes) == cudaSuccess;
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
        d.sms = sms;
    }
    out = &d;
    return ADACOMP_OK;
}

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

template <typename Word>
int launch_generic(const PassArgs &args, const DeviceInfo &info, cudaStream_t st)
{
    const Geometry &geo = args.geo;
    const size_t units = geo.tile_bins < 8u ? 8u : geo.tile_bins;      // generic_tile: a bin or a part of one per warp
    const size_t smem = geo.tile_bins == 1u && sizeof(Word) == 2
                            ? (size_t)align_up((u64)geo.tile_elems * (4 + sizeof(Word)), 16)      // generic_tile_one_bin
                            : (size_t)align_up((u64)geo.tile_elems * (8 + sizeof(Word)), 16) + units * 4 + (units + 1) * 4;
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

// `own_scratch` (optional): the scratch to use in place of the one behind the stream in packed_out.
int compress_impl(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                  uint64_t *count_out, void *stream, uint32_t flags, void *const *events = nullptr,
                  void *lazy_state = nullptr, float factor = 0.f, bool grad_bf16 = false,
                  unsigned char *own_scratch = nullptr)
{
    if (!packed_out || !count_out || (n && (!grad || !residue))) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH)) return ADACOMP_ERR_FLAGS;
    if (factor != 0.f && !(factor > 0.f && factor <= 1e30f)) return ADACOMP_ERR_FLAGS;
    if (misaligned(grad) || misaligned(residue) || misaligned(packed_out) ||
        (reinterpret_cast<uintptr_t>(count_out) & 7u))
        return ADACOMP_ERR_ALIGN;
    const Geometry geo = make_geometry(n, L_T);
    if (geo.n_bins >= (1ull << 31)) return ADACOMP_ERR_SIZE;
    unsigned char *lazy = static_cast<unsigned char *>(lazy_state);
    if (lazy) {
        if (!(fast_L_T(L_T) || any_fast_L_T(L_T)) || flags != 0 || factor != 0.f || grad_bf16) return ADACOMP_ERR_UNSUPPORTED;
        if (misaligned(lazy)) return ADACOMP_ERR_ALIGN;
    }

    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    if (lazy && !info->fast_ready) return ADACOMP_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned char *packed = static_cast<unsigned char *>(packed_out);
    unsigned char *scratch = own_scratch ? own_scratch : packed + geo.scratch_at;

    // the exact-sum windows and the group counts start from zero (a scratch that is reused keeps the last
    // call's contents: tile counts and word slots are fully rewritten before they are read)
    if (cudaMemsetAsync(scratch, 0, kCtlBytes + 8 * geo.n_groups, st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    auto mark = [&](int i) { if (events) cudaEventRecord(static_cast<cudaEvent_t>(events[i]), st); };

    mark(0);
    if (geo.n_tiles) {
        PassArgs args{grad, residue, packed, scratch, geo, flags & ADACOMP_FLAG_LITERAL, lazy, factor, grad_bf16 ? 1u : 0u};
        const bool fast = fast_L_T(L_T) && flags == 0 && info->fast_ready;
        // (one-bin tiles fill the pipelined kernel's 4000-element stages only in part: below 2800 elements the
        // warp-per-part kernel is faster, measured; lazy-scale mode exists in the pipelined kernel only)
        const bool any_fast = any_fast_L_T(L_T) && flags == 0 && !grad_bf16 && info->fast_ready &&
                              (lazy || L_T <= 1000u || L_T >= 2800u);
        if (fast || any_fast) {
            const u64 cap = (u64)info->sms * 2;
            const unsigned grid = (unsigned)(geo.n_tiles < cap ? geo.n_tiles : cap);
            auto launch = [&](auto kernel) { kernel<<<grid, kFastThreads, FastSmem::kBytes, st>>>(args); };
            if (any_fast && lazy) with_any_fast_kernel<true>(L_T, launch);
            else if (any_fast) with_any_fast_kernel<false>(L_T, launch);
            else if (lazy) with_fast_kernel<true, false>(L_T, launch);
            else if (grad_bf16) with_fast_kernel<false, true>(L_T, launch);
            else with_fast_kernel<false, false>(L_T, launch);
        } else {
            rc = geo.w == 1u ? launch_generic<unsigned char>(args, *info, st)
                             : launch_generic<unsigned short>(args, *info, st);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    mark(1);
    finalize<<<1, 1024, 0, st>>>(packed, scratch, geo, flags | (factor != 0.f ? kFlagFactor : 0u), reinterpret_cast<u64 *>(count_out), lazy);
    mark(2);
    if (geo.n_tiles) {
        if (geo.tile_bins <= (u32)kSmallBins) {
            const u64 want = (geo.n_tiles + 3) / 4, cap = (u64)info->sms * 16;
            const unsigned grid = (unsigned)(want < cap ? want : cap);
            if (lazy) {     // the residue keeps G; only the words move
                if (geo.w == 1u) gather_fixup_small<unsigned char, false><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
                else gather_fixup_small<unsigned short, false><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
            } else {
                if (geo.w == 1u) gather_fixup_small<unsigned char, true><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
                else gather_fixup_small<unsigned short, true><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
            }
        } else {
            const u64 cap = (u64)info->sms * 8;
            const unsigned grid = (unsigned)(geo.n_tiles < cap ? geo.n_tiles : cap);
            if (geo.w == 1u) gather_fixup<unsigned char><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
            else gather_fixup<unsigned short><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo);
        }
    }
    mark(3);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

// `ep` (optional): the optimizer step that takes the place of the store to dst (dst is null then).
int decompress_impl(const void *const *packed, uint32_t k, float *dst, void *stream, uint64_t hint_n = 0,
                    uint32_t hint_L_T = 0, const Epilogue *ep = nullptr)
{
    if (!packed || (!dst && !ep)) return ADACOMP_ERR_NULL;
    if (k == 0 || k > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    DecodeArgs args;
    for (uint32_t l = 0; l < ADACOMP_MAX_STREAMS; l++) args.stream[l] = nullptr;
    for (uint32_t l = 0; l < k; l++) {
        if (!packed[l]) return ADACOMP_ERR_NULL;
        if (misaligned(packed[l])) return ADACOMP_ERR_ALIGN;
        args.stream[l] = static_cast<const unsigned char *>(packed[l]);
    }
    if (dst && misaligned(dst)) return ADACOMP_ERR_ALIGN;
    args.ep = Epilogue{nullptr, nullptr, nullptr, 0.f, 0.f, 0.f, 0.f, (float)k, 0u, 0.f};
    if (ep) {
        if (!ep->weights || !ep->momentum || (ep->adam && !ep->second)) return ADACOMP_ERR_NULL;
        if (misaligned(ep->weights) || misaligned(ep->momentum) || (ep->adam && misaligned(ep->second)))
            return ADACOMP_ERR_ALIGN;
        args.ep = *ep;
        args.ep.k = (float)k;
        args.ep.inv_k = (k & (k - 1u)) == 0u ? 1.0f / (float)k : 0.f;
    }
    args.dst = dst;
    args.k = k;
    args.hint_n = hint_n;
    args.hint_L_T = hint_L_T;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    args.pairs = !ep && info->decode_pair_per_sm > 0 ? 1u : 0u;
    u64 grid = (u64)info->sms * info->decode_per_sm, grid_w = (u64)info->sms * info->decode_warps_per_sm;
    u64 grid_one = (u64)info->sms * info->decode_one_per_sm;
    bool warps = true, others = true;   // the shape is on the device: every kernel goes, all but one return at once
    if (hint_L_T) {                     // the shape is known on the host: one kernel, no more CTAs than work items
        const Geometry hg = make_geometry(hint_n, hint_L_T);
        warps = warp_path(hg);
        others = !warps;
        const u64 items = warps ? warp_items(hg).n_items : decode_items(hint_n, hint_L_T);
        grid = items < grid ? (items ? items : 1) : grid;
        grid_w = items < grid_w ? (items ? items : 1) : grid_w;
        grid_one = items < grid_one ? (items ? items : 1) : grid_one;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (warps && ep) {
        // (the optimizer entry points always pass the shape)
        // (eight warps where they divide the tile's bins, unless four can work a lane per bin)
        const Geometry og = make_geometry(hint_n, hint_L_T ? hint_L_T : 1u);
        const bool eight = hint_L_T && og.tile_bins % 8u == 0 && !lanes_shape(og.tile_bins, 4u, og.w);
        const int per = info->decode_opt_per_sm[ep->adam ? 1 : 0][eight ? 1 : 0];
        if (!per) return ADACOMP_ERR_CUDA;
        u64 grid_s = (u64)info->sms * per;
        if (hint_L_T) {
            const u64 items = warp_items(make_geometry(hint_n, hint_L_T)).n_items;
            grid_s = items < grid_s ? (items ? items : 1) : grid_s;
        }
        const unsigned g = (unsigned)grid_s;
        const bool one = hint_L_T > 1000u;
        if (ep->adam && eight) decode_sum_warps<2, 8><<<g, 9 * 32, opt_smem_bytes(2), st>>>(args);
        else if (ep->adam && one) decode_sum_warps<2, 4, true><<<g, 5 * 32, opt_smem_bytes(2), st>>>(args);
        else if (ep->adam) decode_sum_warps<2, 4><<<g, 5 * 32, opt_smem_bytes(2), st>>>(args);
        else if (eight) decode_sum_warps<1, 8><<<g, 9 * 32, opt_smem_bytes(1), st>>>(args);
        else if (one) decode_sum_warps<1, 4, true><<<g, 5 * 32, opt_smem_bytes(1), st>>>(args);
        else decode_sum_warps<1, 4><<<g, 5 * 32, opt_smem_bytes(1), st>>>(args);
    } else if (warps) {
        // (without the shape all three go and two of them return at once; the pairs of 80-bin tiles have a
        // kernel of their own, see pair_path())
        const bool pairs_ok = info->decode_pair_per_sm > 0;
        const bool pair = pairs_ok && hint_L_T && pair_path(make_geometry(hint_n, hint_L_T));
        if (pairs_ok && (!hint_L_T || pair)) {
            u64 grid_p = (u64)info->sms * info->decode_pair_per_sm;
            if (hint_L_T) {
                const u64 items = warp_items(make_geometry(hint_n, hint_L_T), 2u).n_items;
                grid_p = items < grid_p ? (items ? items : 1) : grid_p;
            }
            decode_sum_warps<0, 5, false, 2><<<(unsigned)grid_p, 6 * 32, kPairSmemBytes, st>>>(args);
        }
        if (!hint_L_T || (hint_L_T <= 1000u && !pair)) decode_sum_warps<0, 4><<<(unsigned)grid_w, kDecodeLaunch, 0, st>>>(args);
        if (!hint_L_T || hint_L_T > 1000u) decode_sum_warps<0, 4, true><<<(unsigned)grid_one, kDecodeLaunch, 0, st>>>(args);
    }
    if (others) decode_sum<<<(unsigned)grid, kDecodeThreads, 0, st>>>(args);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
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
            if (lazy) batch_tile_pass_fast<N, true><<<grid, kFastThreads, FastSmem::kBytes, st>>>(b);
            else batch_tile_pass_fast<N, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(b);
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
int launch_batch(const BatchArgs &b, const DeviceInfo &info, cudaStream_t st, bool lazy = false)
{
    if (b.n_layers == 0) return ADACOMP_OK;
    if (b.n_layers == 1) {      // a batch of one gains nothing over the single-layer kernels
        const BatchLayer &L = b.layer[0];
        return compress_impl(L.grad, L.residue, L.geo.n, L.geo.L_T, L.packed, reinterpret_cast<uint64_t *>(L.count_out),
                             st, 0, nullptr, L.lazy);
    }
    if (b.n_layers <= (u32)kBatchSmall) {
        BatchArgsT<kBatchSmall> small;
        small.n_layers = b.n_layers;
        small.total_tiles = b.total_tiles;
        for (u32 i = 0; i < b.n_layers; i++) small.layer[i] = b.layer[i];
        return launch_batch_sized(small, info, st, lazy);
    }
    return launch_batch_sized(b, info, st, lazy);
}

inline bool batchable(const adacomp_layer_desc &d, const DeviceInfo &info)
{
    return d.flags == 0 && d.L_T >= 42u && d.L_T <= 1000u && d.n < (info.batch_fast_ready ? kPackBatchMaxElems : kBatchLayerMaxElems);
}

// ---------------------------------------------------------------------------------
// pack() with the library's own scratch: for callers that cannot allocate device memory
// ---------------------------------------------------------------------------------

// Built-in scratch of adacomp_compress_static.  It is part of the loaded module: every
// GPU that loads the library holds these bytes until the process exits.  All calls on a
// device share it and it keeps the previous call's contents.
static __device__ __align__(256) unsigned char g_static_scratch[ADACOMP_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch per device, looked up on the first call there.  In
// host code the array's name is only a handle for the runtime, never a device address.
unsigned char *g_static_scratch_addr[64];

int compress_static_impl(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                         uint64_t *count_out, void *stream)
{
    if (!packed_out || !count_out || (n && (!grad || !residue))) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (misaligned(grad) || misaligned(residue) || misaligned(packed_out) ||
        (reinterpret_cast<uintptr_t>(count_out) & 7u))
        return ADACOMP_ERR_ALIGN;
    const Geometry geo = make_geometry(n, L_T);
    if (geo.n_bins >= (1ull << 31)) return ADACOMP_ERR_SIZE;
    if (geo.scratch_bytes > (u64)ADACOMP_STATIC_SCRATCH_BYTES) return ADACOMP_ERR_STATIC_SCRATCH;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ADACOMP_ERR_CUDA;
    if (!g_static_scratch_addr[dev]) {
        // set-up, once per device, with that device current (two host threads that meet here store the same
        // address: the look-up is idempotent, so no lock guards it)
        unsigned char *ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_scratch) != cudaSuccess || !ptr)
            return ADACOMP_ERR_CUDA;
        g_static_scratch_addr[dev] = ptr;
    }
    // the same kernels, in the same order, as adacomp_compress: only the scratch is elsewhere
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, nullptr, 0.f, false,
                         g_static_scratch_addr[dev]);
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
    case ADACOMP_ERR_UNSUPPORTED: return "lazy mode supports L_T = 41..1000 (and multiples of 4 up to 4000) without flags only";
    case ADACOMP_ERR_STATIC_SCRATCH:
        return "tensor needs more scratch than the library's built-in array holds; use adacomp_compress";
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

int adacomp_compress_static(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                            uint64_t *count_out, void *stream)
{
    return compress_static_impl(grad, residue, n, L_T, packed_out, count_out, stream);
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

int adacomp_decompress_accumulate_ex(const void *const *packed, uint32_t k_streams, float *dst, uint64_t n,
                                     uint32_t L_T, void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    return decompress_impl(packed, k_streams, dst, stream, n, L_T);
}

// Decode-sum of a list of layers whose shapes the caller knows.  `opt` (optional; its pointers unused):
// `dst` then holds the layers' weights, `aux` their momentum (Adam: first moments), `aux2` (Adam) their
// second moments, and every layer gets the optimizer step instead of a store.
int decompress_multi_impl(const void *const *packed, uint32_t k_streams, float *const *dst, float *const *aux,
                          float *const *aux2, const uint64_t *n, const uint32_t *L_T, uint32_t n_layers, void *stream,
                          const Epilogue *opt)
{
    if (opt && n_layers && (!aux || (opt->adam && !aux2))) return ADACOMP_ERR_NULL;
    if (n_layers && (!packed || !dst || !n || !L_T)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    for (uint32_t t = 0; t < n_layers; t++) {
        if (L_T[t] == 0 || L_T[t] > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
        if (!dst[t] || (opt && !aux[t]) || (opt && opt->adam && !aux2[t])) return ADACOMP_ERR_NULL;
        if (misaligned(dst[t]) || (opt && misaligned(aux[t])) || (opt && opt->adam && misaligned(aux2[t])))
            return ADACOMP_ERR_ALIGN;
        for (uint32_t l = 0; l < k_streams; l++) {
            if (!packed[(size_t)t * k_streams + l]) return ADACOMP_ERR_NULL;
            if (misaligned(packed[(size_t)t * k_streams + l])) return ADACOMP_ERR_ALIGN;
        }
    }
    if (n_layers == 0) return ADACOMP_OK;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // small layers of the paper's bin lengths share launches; the rest are decoded one by one
    static thread_local DecodeBatchArgs batch;
    batch.n_layers = 0;
    batch.k = k_streams;
    batch.opt = !opt ? 0u : opt->adam ? 2u : 1u;
    batch.lr = opt ? opt->lr : 0.f;
    batch.mu = opt ? opt->mu : 0.f;
    batch.beta2 = opt ? opt->beta2 : 0.f;
    batch.eps = opt ? opt->eps : 0.f;
    u64 batch_tiles = 0;
    // (the batched warp decoder, and with it layers of up to 2^25 elements for plain decode-sum; with an
    // optimizer step larger layers keep the single-tensor kernels, which stage the optimizer's arrays by bulk copies)
    const int opt_form = !opt ? 0 : opt->adam ? 2 : 1;
    const bool warps_batch = info->dec_batch_warps_per_sm[opt_form] > 0;
    const u64 batch_max_elems = warps_batch && !opt ? kPackBatchMaxElems : kBatchLayerMaxElems;
    auto flush = [&]() -> int {
        if (batch.n_layers == 0) return ADACOMP_OK;
        if (warps_batch) {
            const u32 ring = kBatchRingBytes;
            const u64 cap = (u64)info->sms * info->dec_batch_warps_per_sm[batch.opt];
            const unsigned grid = (unsigned)(batch_tiles < cap ? (batch_tiles ? batch_tiles : 1) : cap);
            if (batch.opt == 2u) decode_batch_warps<2><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
            else if (batch.opt == 1u) decode_batch_warps<1><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
            else decode_batch_warps<0><<<grid, kDecodeLaunch, ring, st>>>(batch, ring);
        } else {
            const u64 cap = (u64)info->sms * info->dec_batch_per_sm;
            const unsigned grid = (unsigned)(batch_tiles < cap ? (batch_tiles ? batch_tiles : 1) : cap);
            decode_batch<<<grid, kDecodeThreads, sizeof(DecodeBatchSmem), st>>>(batch);
        }
        batch.n_layers = 0;
        batch_tiles = 0;
        return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
    };
    const uint32_t per_batch = (uint32_t)kDecBatchPtrs / k_streams < (uint32_t)kDecBatchLayers
                                   ? (uint32_t)kDecBatchPtrs / k_streams : (uint32_t)kDecBatchLayers;
    for (uint32_t t = 0; t < n_layers; t++) {
        const bool small = info->dec_batch_per_sm > 0 && L_T[t] >= 42u && L_T[t] <= 1000u &&
                           n[t] < batch_max_elems && n_layers > 1;
        if (small) {
            const u32 i = batch.n_layers++;
            batch.n[i] = n[t];
            batch.L_T[i] = L_T[t];
            batch.dst[i] = dst[t];
            batch.aux[i] = opt ? aux[t] : nullptr;
            batch.aux2[i] = opt && opt->adam ? aux2[t] : nullptr;
            for (uint32_t l = 0; l < k_streams; l++)
                batch.stream[(size_t)i * k_streams + l] = static_cast<const unsigned char *>(packed[(size_t)t * k_streams + l]);
            batch_tiles += decode_items(n[t], L_T[t]);
            if (batch.n_layers == per_batch) {
                rc = flush();
                if (rc != ADACOMP_OK) return rc;
            }
        } else if (opt) {
            Epilogue ep = *opt;
            ep.weights = dst[t];
            ep.momentum = aux[t];
            ep.second = opt->adam ? aux2[t] : nullptr;
            rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, nullptr, stream, n[t], L_T[t], &ep);
            if (rc != ADACOMP_OK) return rc;
        } else {
            rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, dst[t], stream, n[t], L_T[t]);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    return flush();
}

int adacomp_decompress_accumulate_multi_ex(const void *const *packed, uint32_t k_streams, float *const *dst,
                                           const uint64_t *n, const uint32_t *L_T, uint32_t n_layers, void *stream)
{
    return decompress_multi_impl(packed, k_streams, dst, nullptr, nullptr, n, L_T, n_layers, stream, nullptr);
}

int adacomp_decompress_average_sgd_multi(const void *const *packed, uint32_t k_streams, float *const *weights,
                                         float *const *momentum, const uint64_t *n, const uint32_t *L_T,
                                         uint32_t n_layers, float lr, float mu, void *stream)
{
    const Epilogue opt = {nullptr, nullptr, nullptr, lr, mu, 0.f, 0.f, 0.f, 0u, 0.f};
    return decompress_multi_impl(packed, k_streams, weights, momentum, nullptr, n, L_T, n_layers, stream, &opt);
}

int adacomp_decompress_average_adam_multi(const void *const *packed, uint32_t k_streams, float *const *weights,
                                          float *const *m, float *const *v, const uint64_t *n, const uint32_t *L_T,
                                          uint32_t n_layers, float step_size, float beta1, float beta2, float eps,
                                          void *stream)
{
    const Epilogue opt = {nullptr, nullptr, nullptr, step_size, beta1, beta2, eps, 0.f, 1u, 0.f};
    return decompress_multi_impl(packed, k_streams, weights, m, v, n, L_T, n_layers, stream, &opt);
}

int adacomp_compress_profile(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                             uint64_t *count_out, void *stream, uint32_t flags, void *const *events,
                             void *lazy_state)
{
    if (!events) return ADACOMP_ERR_NULL;
    for (int i = 0; i < 4; i++)
        if (!events[i]) return ADACOMP_ERR_NULL;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, flags, events, lazy_state);
}

size_t adacomp_lazy_state_bytes(uint64_t n, uint32_t L_T)
{
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return 0;
    return (size_t)lazy_state_bytes(make_geometry(n, L_T));
}

int adacomp_lazy_state_init(void *state, uint64_t n, uint32_t L_T, void *stream)
{
    if (!state) return ADACOMP_ERR_NULL;
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return ADACOMP_ERR_UNSUPPORTED;
    if (misaligned(state)) return ADACOMP_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(state, 0, lazy_state_bytes(make_geometry(n, L_T)), st) != cudaSuccess) return ADACOMP_ERR_CUDA;
    lazy_init_kernel<<<1, 1, 0, st>>>(static_cast<unsigned char *>(state), n, L_T);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int adacomp_compress_lazy(const float *grad, float *residue, void *state, uint64_t n, uint32_t L_T,
                          void *packed_out, uint64_t *count_out, void *stream)
{
    if (!state) return ADACOMP_ERR_NULL;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, state);
}

int adacomp_residue_flush(float *residue, void *state, uint64_t n, uint32_t L_T, void *stream)
{
    if (!state || (n && !residue)) return ADACOMP_ERR_NULL;
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return ADACOMP_ERR_UNSUPPORTED;
    if (misaligned(residue) || misaligned(state)) return ADACOMP_ERR_ALIGN;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    const u64 segs = (n + kSeg - 1) / kSeg;
    const u64 want = (segs + 255) / 256, cap = (u64)info->sms * 8;
    const unsigned grid = (unsigned)(want < 1 ? 1 : (want < cap ? want : cap));
    lazy_flush_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(residue, static_cast<unsigned char *>(state), n, L_T,
                                                                          make_geometry(n, L_T).tile_elems);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int adacomp_compress_host(const float *grad_host, float *grad_stage, float *residue, uint64_t n, uint32_t L_T,
                          void *packed_dev, uint64_t *count_dev, void *packed_host, uint64_t packed_host_cap,
                          uint64_t *count_host, void *stream)
{
    if (!count_host || !packed_host || (n && (!grad_host || !grad_stage))) return ADACOMP_ERR_NULL;
    // every check pack() makes on the host comes before the first copy: an error code means nothing was enqueued
    if (!packed_dev || !count_dev || (n && !residue)) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (misaligned(grad_stage) || misaligned(residue) || misaligned(packed_dev) ||
        (reinterpret_cast<uintptr_t>(count_dev) & 7u))
        return ADACOMP_ERR_ALIGN;
    if ((n + L_T - 1) / L_T >= (1ull << 31)) return ADACOMP_ERR_SIZE;
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

// `states` (optional): lazy-scale mode, states[t] the state of layer t.
static int compress_multi_impl(const adacomp_layer_desc *layers, void *const *states, uint32_t n_layers, void *stream)
{
    if (n_layers && !layers) return ADACOMP_ERR_NULL;
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        if (!d.packed_out || !d.count_out || (d.n && (!d.grad || !d.residue))) return ADACOMP_ERR_NULL;
        if (d.L_T == 0 || d.L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
        if (d.flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH)) return ADACOMP_ERR_FLAGS;
        if (misaligned(d.grad) || misaligned(d.residue) || misaligned(d.packed_out) ||
            (reinterpret_cast<uintptr_t>(d.count_out) & 7u))
            return ADACOMP_ERR_ALIGN;
        if ((d.n + d.L_T - 1) / d.L_T >= (1ull << 31)) return ADACOMP_ERR_SIZE;
        if (states) {
            if (!states[t]) return ADACOMP_ERR_NULL;
            if (misaligned(states[t])) return ADACOMP_ERR_ALIGN;
            if (d.flags != 0 || !(fast_L_T(d.L_T) || any_fast_L_T(d.L_T))) return ADACOMP_ERR_UNSUPPORTED;
        }
    }
    if (n_layers == 0) return ADACOMP_OK;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // small layers share four launches per batch; the rest go through the single-layer path
    static thread_local BatchArgs batch;
    batch.n_layers = 0;
    batch.total_tiles = 0;
    auto batched = [&](const adacomp_layer_desc &d) {
        return info->batch_per_sm > 0 && batchable(d, *info) && (!states || info->batch_fast_ready);
    };
    // (more layers than a table holds: batches of equal size, so that none is left with a layer or two)
    uint32_t to_batch = 0;
    for (uint32_t t = 0; t < n_layers; t++) to_batch += batched(layers[t]) ? 1u : 0u;
    const uint32_t n_batches = (to_batch + (uint32_t)kBatchMax - 1) / (uint32_t)kBatchMax;
    const uint32_t per_batch = n_batches ? (to_batch + n_batches - 1) / n_batches : (uint32_t)kBatchMax;
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        if (batched(d)) {
            BatchLayer &L = batch.layer[batch.n_layers++];
            L.grad = d.grad;
            L.residue = d.residue;
            L.packed = static_cast<unsigned char *>(d.packed_out);
            L.count_out = reinterpret_cast<u64 *>(d.count_out);
            L.geo = make_geometry(d.n, d.L_T);
            L.tile_first = batch.total_tiles;
            L.pad = 0;
            L.lazy = states ? static_cast<unsigned char *>(states[t]) : nullptr;
            batch.total_tiles += (u32)L.geo.n_tiles;
            if (batch.n_layers == per_batch) {
                rc = launch_batch(batch, *info, st, states != nullptr);
                if (rc != ADACOMP_OK) return rc;
                batch.n_layers = 0;
                batch.total_tiles = 0;
            }
        } else {
            rc = compress_impl(d.grad, d.residue, d.n, d.L_T, d.packed_out, d.count_out, stream, d.flags, nullptr,
                               states ? states[t] : nullptr);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    return launch_batch(batch, *info, st, states != nullptr);
}

int adacomp_compress_multi(const adacomp_layer_desc *layers, uint32_t n_layers, void *stream)
{
    return compress_multi_impl(layers, nullptr, n_layers, stream);
}

int adacomp_compress_multi_lazy(const adacomp_layer_desc *layers, void *const *states, uint32_t n_layers, void *stream)
{
    if (n_layers && !states) return ADACOMP_ERR_NULL;
    return compress_multi_impl(layers, states, n_layers, stream);
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

int adacomp_compress_bf16(const void *grad_bf16, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                          uint64_t *count_out, void *stream)
{
    return compress_impl(static_cast<const float *>(grad_bf16), residue, n, L_T, packed_out, count_out, stream, 0, nullptr,
                         nullptr, 0.f, true);
}

int adacomp_compress_scaled(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                            uint64_t *count_out, void *stream, float factor)
{
    if (!(factor > 0.f && factor <= 1e30f)) return ADACOMP_ERR_FLAGS;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, nullptr, factor);
}

int adacomp_decompress_average_sgd(const void *const *packed, uint32_t k_streams, float *weights, float *momentum,
                                   uint64_t n, uint32_t L_T, float lr, float mu, void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    const Epilogue ep = {weights, momentum, nullptr, lr, mu, 0.f, 0.f, 0.f, 0u, 0.f};
    return decompress_impl(packed, k_streams, nullptr, stream, n, L_T, &ep);
}

int adacomp_decompress_average_adam(const void *const *packed, uint32_t k_streams, float *weights, float *m, float *v,
                                    uint64_t n, uint32_t L_T, float step_size, float beta1, float beta2, float eps,
                                    void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    const Epilogue ep = {weights, m, v, step_size, beta1, beta2, eps, 0.f, 1u, 0.f};
    return decompress_impl(packed, k_streams, nullptr, stream, n, L_T, &ep);
}

int adacomp_set_device(int device)
{
    return cudaSetDevice(device) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
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
