// unpack() and the ordered sum: everything the single-tensor and the batched decoders share.
#pragma once

#include "common.cuh"

namespace adacomp_impl {

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
    long long wait_limit;   // cycles a wait for a slot may take (kWaitCycles unless a test shortened it)
    u32 withhold;           // testing aid: CTA 0's loader starts no copies for its item number `withhold` (0: none)
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
                if (use > 0 && !mbar_wait(&ws.empty[s], (use - 1u) & 1u, a.wait_limit)) {
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
                // (testing aid) bytes are expected and never sent: the decoding warps' wait for this slot runs out
                const bool hold = a.withhold != 0u && blockIdx.x == 0 && it == (u64)a.withhold;
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const u32 j = (u32)lane + 32u * h;
                    if (j < staged && !hold) {
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
            for (u64 j = issued > S ? issued - S : 0; j < issued; j++) mbar_wait(&ws.full[j % S], (u32)(j / S) & 1u, a.wait_limit);    // (rare)
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
            if (!mbar_wait(&ws.full[s], use & 1u, a.wait_limit)) {
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
                if (!mbar_wait(&ws.wv_full[warp], wv_use & 1u, a.wait_limit)) {
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


}  // namespace adacomp_impl
