// Stream version 2, the form for the wire: the bins are told apart by a first-of-bin flag in the words instead of
// a count per bin (the paper's rate figures, Section "Experiment Results", count the words alone), and a bin that
// sends nothing is one marker word.  The decoders read version 1; these kernels re-encode a packed stream either way,
// so that exchange() can send version 2 and decode what it receives:
//   word (version 1) = (index << 2) | code,  code 01 = +scale, 11 = -scale
//   word (version 2) = (index << 2) | (first_of_bin << 1) | negative;  marker = (L_T << 2) | 2
// Version 2 words are 8 bits wide for L_T <= 63 (the marker's index must fit 6 bits) and 16 bits above; there is
// no count section, the directory holds version-2 word offsets, and bytes 52..55 of the header hold the number of
// bins that send nothing.  Each direction is three small kernels: per tile, how many markers it has (into the
// output's directory); one CTA turns those into the output's word offsets and writes the header; per tile, the
// words.  A warp per tile throughout; nothing here waits on anything.
#include "internal.h"

namespace adacomp_impl {

constexpr int kWireThreads = 128;

struct WireGeo {
    Geometry g;         // the version-1 geometry of (n, L_T)
    u32 w2;             // bytes of a version-2 word
    u64 pay2;           // offset of the version-2 payload
};

__host__ __device__ inline WireGeo wire_geometry(u64 n, u32 L_T)
{
    WireGeo q;
    q.g = make_geometry(n, L_T);
    q.w2 = L_T <= 63u ? 1u : 2u;
    q.pay2 = align_up(kHeaderBytes + 8 * (q.g.n_tiles + 1), 16);
    return q;
}

__device__ inline u32 load_w(const unsigned char *p, u64 i, u32 w)
{
    return w == 1u ? (u32)p[i] : (u32)reinterpret_cast<const unsigned short *>(p)[i];
}
__device__ inline void store_w(unsigned char *p, u64 i, u32 w, u32 v)
{
    if (w == 1u) p[i] = (unsigned char)v;
    else reinterpret_cast<unsigned short *>(p)[i] = (unsigned short)v;
}

// The header must be the one of a stream of this shape and version; else the conversion does nothing but say so.
__device__ inline bool wire_header_ok(const unsigned char *in, const WireGeo &q, u32 version)
{
    const u32 *h = reinterpret_cast<const u32 *>(in);
    const u64 *h64 = reinterpret_cast<const u64 *>(in);
    const u32 w = version == 1u ? q.g.w : q.w2;
    return h[0] == kMagic && (h[1] & 0xffffu) == version && ((h[1] >> 16) & 0xffu) == w && h[2] == q.g.L_T &&
           h64[2] == q.g.n && h64[3] == q.g.n_bins && h64[4] == q.g.n_tiles && h64[5] <= q.g.n;
}

// ---- version 1 -> version 2 ----

// (1) bins of each tile that send nothing, left in the output's directory for the scan
__global__ void __launch_bounds__(kWireThreads)
to_v2_count(const unsigned char *in, unsigned char *out, WireGeo q)
{
    if (!wire_header_ok(in, q, 1u)) return;
    const int lane = threadIdx.x & 31;
    const u64 warp = ((u64)blockIdx.x * kWireThreads + threadIdx.x) >> 5, warps = ((u64)gridDim.x * kWireThreads) >> 5;
    const unsigned char *cnt = in + q.g.bin_cnt_at;
    u64 *dir2 = reinterpret_cast<u64 *>(out + kHeaderBytes);
    for (u64 t = warp; t < q.g.n_tiles; t += warps) {
        const u64 b0 = t * q.g.tile_bins, b1 = min(b0 + q.g.tile_bins, q.g.n_bins);
        u32 empty = 0;
        for (u64 b = b0 + lane; b < b1; b += 32) empty += load_w(cnt, b, q.g.w) == 0u;
        empty = __reduce_add_sync(0xffffffffu, empty);
        if (lane == 0) dir2[t] = empty;
    }
}

// (2) one CTA: marker counts -> word offsets of the output (in place), header, counts for the caller, padding.
// `to_v2`: the output is version 2 (offsets grow by the markers ahead), else version 1 (they shrink).
__global__ void __launch_bounds__(1024)
wire_scan(const unsigned char *in, unsigned char *out, WireGeo q, u64 *count_out, u32 to_v2)
{
    __shared__ u64 s_warp[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (!wire_header_ok(in, q, to_v2 ? 1u : 2u)) {
        if (tid == 0) {
            raise_status(ADACOMP_DEV_HEADER_MISMATCH);
            if (count_out) count_out[0] = count_out[1] = 0;
        }
        return;
    }
    const u64 n_tiles = q.g.n_tiles;
    const u64 *dir_in = reinterpret_cast<const u64 *>(in + kHeaderBytes);
    u64 *dir_out = reinterpret_cast<u64 *>(out + kHeaderBytes);
    const u64 per = (n_tiles + 1023) / 1024;
    const u64 lo = min((u64)tid * per, n_tiles), hi = min(lo + per, n_tiles);
    u64 sum = 0;
    for (u64 i = lo; i < hi; i++) sum += dir_out[i];
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
    u64 run = s_warp[warp] + inc - sum;          // markers ahead of tile lo
    for (u64 i = lo; i < hi; i++) {
        const u64 m = dir_out[i];
        dir_out[i] = to_v2 ? dir_in[i] + run : dir_in[i] - run;
        run += m;
    }
    const u64 markers = s_warp[32];
    const u32 *h32 = reinterpret_cast<const u32 *>(in);
    const u64 *h64 = reinterpret_cast<const u64 *>(in);
    const u64 n_sel = h64[5];
    const u64 words_out = to_v2 ? n_sel + markers : n_sel;
    const u32 w_out = to_v2 ? q.w2 : q.g.w;
    const u64 pay_out = to_v2 ? q.pay2 : q.g.payload_at;
    const u64 bytes_used = pay_out + align_up(words_out * w_out, 16);
    if (tid == 0) {
        dir_out[n_tiles] = words_out;
        u32 *o32 = reinterpret_cast<u32 *>(out);
        u64 *o64 = reinterpret_cast<u64 *>(out);
        o32[0] = kMagic;
        o32[1] = (to_v2 ? 2u : 1u) | (w_out << 16) | (h32[1] & 0xff000000u);
        o32[2] = h32[2];
        o32[3] = h32[3];
        o64[2] = h64[2];
        o64[3] = h64[3];
        o64[4] = h64[4];
        o64[5] = n_sel;
        o32[12] = h32[12];
        o32[13] = to_v2 ? (u32)markers : 0u;
        o64[7] = bytes_used;
        if (count_out) {
            count_out[0] = words_out;
            count_out[1] = bytes_used;
        }
        // (a version-2 stream that says it has other markers than its words show is malformed)
        if (!to_v2 && markers != (u64)h32[13]) raise_status(ADACOMP_DEV_BAD_STREAM);
    }
    // zero padding behind the last word and in the alignment gaps of the sections
    const u64 pay_end = pay_out + words_out * w_out;
    const u64 pad = align_up(pay_end, 16) - pay_end;
    if ((u64)tid < pad) out[pay_end + tid] = 0;
    const u64 dir_end = kHeaderBytes + 8 * (n_tiles + 1);
    const u64 gap = (to_v2 ? q.pay2 : q.g.bin_cnt_at) - dir_end;
    if ((u64)tid < gap) out[dir_end + tid] = 0;
    if (!to_v2) {
        const u64 cnt_end = q.g.bin_cnt_at + q.g.n_bins * q.g.w;
        if ((u64)tid < q.g.payload_at - cnt_end) out[cnt_end + tid] = 0;
    }
}

// (3) the words of each tile: lane b of a chunk of 32 bins scans the counts; the chunk's words are then taken 32
// at a time, lane j finding its word's bin among the 32 running sums.
__global__ void __launch_bounds__(kWireThreads)
to_v2_words(const unsigned char *in, unsigned char *out, WireGeo q)
{
    if (!wire_header_ok(in, q, 1u)) return;
    constexpr u32 full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const u64 warp = ((u64)blockIdx.x * kWireThreads + threadIdx.x) >> 5, warps = ((u64)gridDim.x * kWireThreads) >> 5;
    const unsigned char *cnt = in + q.g.bin_cnt_at, *pay1 = in + q.g.payload_at;
    const u64 *dir1 = reinterpret_cast<const u64 *>(in + kHeaderBytes);
    const u64 *dir2 = reinterpret_cast<const u64 *>(out + kHeaderBytes);
    unsigned char *pay2 = out + q.pay2;
    const u64 n_sel = reinterpret_cast<const u64 *>(in)[5];
    u32 bad = 0;
    for (u64 t = warp; t < q.g.n_tiles; t += warps) {
        const u64 b0 = t * q.g.tile_bins, b1 = min(b0 + q.g.tile_bins, q.g.n_bins);
        u64 base1 = dir1[t], base2 = dir2[t];
        const u64 end1 = min(dir1[t + 1], n_sel);
        for (u64 bb = b0; bb < b1; bb += 32) {
            const u64 bin = bb + lane;
            const bool exists = bin < b1;
            const u32 c = exists ? load_w(cnt, bin, q.g.w) : 0u;
            const u32 marker = exists && c == 0u ? 1u : 0u;
            u32 i1 = c, i2 = c + marker;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const u32 a1 = __shfl_up_sync(full, i1, d), a2 = __shfl_up_sync(full, i2, d);
                if (lane >= d) { i1 += a1; i2 += a2; }
            }
            const u32 tot1 = __shfl_sync(full, i1, 31), tot2 = __shfl_sync(full, i2, 31);
            const u32 ex1 = i1 - c, ex2 = i2 - c - marker;
            if (base1 + tot1 > end1) {              // counts and directory disagree: nothing more of this tile is read
                bad |= ADACOMP_DEV_BAD_STREAM;
                break;
            }
            if (base2 + tot2 > q.g.n) {             // more words than elements: a malformed directory
                bad |= ADACOMP_DEV_BAD_STREAM;
                break;
            }
            if (marker) store_w(pay2, base2 + ex2, q.w2, (q.g.L_T << 2) | 2u);
            for (u32 j0 = 0; j0 < tot1; j0 += 32) {
                const u32 j = j0 + lane;
                // the bin of word j: the first lane whose inclusive sum exceeds j
                int lo = 0;
#pragma unroll
                for (int step = 16; step > 0; step >>= 1) {
                    const u32 probe = __shfl_sync(full, i1, lo + step - 1);
                    if (probe <= j) lo += step;
                }
                const u32 qe1 = __shfl_sync(full, ex1, lo), qe2 = __shfl_sync(full, ex2, lo);
                const u32 qm = __shfl_sync(full, marker, lo);
                if (j < tot1) {
                    const u32 word1 = load_w(pay1, base1 + j, q.g.w);
                    if ((word1 & 1u) == 0u) bad |= (word1 & 2u) ? ADACOMP_DEV_RESERVED_CODE : ADACOMP_DEV_BAD_STREAM;
                    const u32 word2 = (word1 & ~3u) | (j == qe1 ? 2u : 0u) | ((word1 & 3u) == 3u ? 1u : 0u);
                    store_w(pay2, base2 + qe2 + qm + (j - qe1), q.w2, word2);
                }
            }
            base1 += tot1;
            base2 += tot2;
        }
    }
    if (bad) raise_status(bad);
}

// ---- version 2 -> version 1 ----

// (1) marker words of each tile, left in the output's directory for the scan
__global__ void __launch_bounds__(kWireThreads)
from_v2_count(const unsigned char *in, unsigned char *out, WireGeo q)
{
    if (!wire_header_ok(in, q, 2u)) return;
    const int lane = threadIdx.x & 31;
    const u64 warp = ((u64)blockIdx.x * kWireThreads + threadIdx.x) >> 5, warps = ((u64)gridDim.x * kWireThreads) >> 5;
    const u64 *dir2 = reinterpret_cast<const u64 *>(in + kHeaderBytes);
    const unsigned char *pay2 = in + q.pay2;
    u64 *dir1 = reinterpret_cast<u64 *>(out + kHeaderBytes);
    const u64 total = reinterpret_cast<const u64 *>(in)[5] + reinterpret_cast<const u32 *>(in)[13];
    for (u64 t = warp; t < q.g.n_tiles; t += warps) {
        const u64 w0 = min(dir2[t], total), w1 = min(dir2[t + 1], total);
        u32 markers = 0;
        for (u64 j = w0 + lane; j < w1; j += 32) markers += (load_w(pay2, j, q.w2) >> 2) == q.g.L_T;
        markers = __reduce_add_sync(0xffffffffu, markers);
        if (lane == 0) dir1[t] = markers;
    }
}

// (3) the words and the bin counts of each tile.  Every bin owns exactly one flagged word (its first one, or its
// marker), so the r-th flag of a tile opens the tile's r-th bin and a bin's count is the distance to the next
// flag (less its marker).
__global__ void __launch_bounds__(kWireThreads)
from_v2_words(const unsigned char *in, unsigned char *out, WireGeo q)
{
    if (!wire_header_ok(in, q, 2u)) return;
    constexpr u32 full = 0xffffffffu;
    const int lane = threadIdx.x & 31;
    const u64 warp = ((u64)blockIdx.x * kWireThreads + threadIdx.x) >> 5, warps = ((u64)gridDim.x * kWireThreads) >> 5;
    const u64 *dir2 = reinterpret_cast<const u64 *>(in + kHeaderBytes);
    const u64 *dir1 = reinterpret_cast<const u64 *>(out + kHeaderBytes);
    const unsigned char *pay2 = in + q.pay2;
    unsigned char *cnt = out + q.g.bin_cnt_at, *pay1 = out + q.g.payload_at;
    const u64 total = reinterpret_cast<const u64 *>(in)[5] + reinterpret_cast<const u32 *>(in)[13];
    const u32 le_mask = (2u << lane) - 1u;
    u32 bad = 0;
    for (u64 t = warp; t < q.g.n_tiles; t += warps) {
        const u64 b0 = t * q.g.tile_bins, b1 = min(b0 + q.g.tile_bins, q.g.n_bins);
        const u64 w0 = min(dir2[t], total), w1 = min(max(dir2[t + 1], w0), total);
        u64 at1 = dir1[t];                      // version-1 words written so far
        u64 bins_open = 0;                      // bins of this tile opened so far
        u64 open_at = 0;                        // where the bin that is open started (its flagged word)
        u32 open_marker = 0;
        for (u64 j0 = w0; j0 < w1; j0 += 32) {
            const u64 j = j0 + lane;
            const bool valid = j < w1;
            const u32 word = valid ? load_w(pay2, j, q.w2) : 0u;
            const bool first = valid && (word & 2u);
            const bool marker = valid && (word >> 2) == q.g.L_T;
            const u32 F = __ballot_sync(full, first), M = __ballot_sync(full, marker);
            const u32 V = __ballot_sync(full, valid);
            // the bin that was open when this chunk began ends at the chunk's first flag
            if (F != 0u && bins_open > 0 && lane == 0) {
                const u64 count = j0 + (u32)(__ffs(F) - 1) - open_at - open_marker;
                const u64 bin = b0 + bins_open - 1;
                if (bin < b1 && count <= q.g.L_T) store_w(cnt, bin, q.g.w, (u32)count);
                else bad |= ADACOMP_DEV_BAD_STREAM;
            }
            if (first) {
                const u64 bin = b0 + bins_open + (u32)__popc(F & le_mask) - 1;
                const u32 later = F & ~le_mask;
                if (later) {                    // the next flag is in this chunk: the bin's count is known
                    const u32 count = (u32)(__ffs(later) - 1) - (u32)lane - (marker ? 1u : 0u);
                    if (bin < b1) store_w(cnt, bin, q.g.w, count);
                    else bad |= ADACOMP_DEV_BAD_STREAM;
                }
            }
            if (valid && !marker) {
                if (bins_open == 0 && (F & le_mask) == 0u) {
                    bad |= ADACOMP_DEV_BAD_STREAM;          // a word before the tile's first flag
                } else {
                    if ((word >> 2) > q.g.L_T) bad |= ADACOMP_DEV_BAD_STREAM;
                    const u32 before = (u32)__popc(V & ~M & (le_mask >> 1));   // words (not markers) ahead of mine in the chunk
                    if (at1 + before < q.g.n) store_w(pay1, at1 + before, q.g.w, (word & ~3u) | ((word & 1u) ? 3u : 1u));
                    else bad |= ADACOMP_DEV_BAD_STREAM;
                }
            } else if (marker && !first) {
                bad |= ADACOMP_DEV_BAD_STREAM;
            }
            at1 += (u32)__popc(V & ~M);
            if (F != 0u) {
                const int last = 31 - __clz(F);
                open_at = j0 + (u32)last;
                open_marker = (M >> last) & 1u;
                bins_open += (u32)__popc(F);
            }
        }
        // the tile's last bin ends with the tile; bins of the tile that no flag opened are malformed
        if (lane == 0) {
            if (bins_open > 0) {
                const u64 count = w1 - open_at - open_marker, bin = b0 + bins_open - 1;
                if (bin < b1 && count <= q.g.L_T) store_w(cnt, bin, q.g.w, (u32)count);
                else bad |= ADACOMP_DEV_BAD_STREAM;
            }
            if (bins_open != b1 - b0) bad |= ADACOMP_DEV_BAD_STREAM;
        }
        __syncwarp();
    }
    if (bad) raise_status(bad);
}

int stream_convert(const void *in, void *out, uint64_t out_capacity, uint64_t *count_out, uint64_t n, uint32_t L_T,
                   bool to_v2, void *stream)
{
    if (!in || !out) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T >= ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;        // (L_T = 16384 has no version-2 form)
    if (misaligned(in) || misaligned(out) || (reinterpret_cast<uintptr_t>(count_out) & 7u)) return ADACOMP_ERR_ALIGN;
    const WireGeo q = wire_geometry(n, L_T);
    if (q.g.n_bins >= (1ull << 31)) return ADACOMP_ERR_SIZE;
    const u64 need = to_v2 ? q.pay2 + align_up(n * q.w2, 16) : q.g.payload_at + align_up(n * q.g.w, 16);
    if (out_capacity < need) return ADACOMP_ERR_SIZE;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const u64 want = (q.g.n_tiles + 3) / 4, cap = (u64)info->sms * 16;
    const unsigned grid = (unsigned)(want < 1 ? 1 : (want < cap ? want : cap));
    const unsigned char *src = static_cast<const unsigned char *>(in);
    unsigned char *dst = static_cast<unsigned char *>(out);
    if (to_v2) to_v2_count<<<grid, kWireThreads, 0, st>>>(src, dst, q);
    else from_v2_count<<<grid, kWireThreads, 0, st>>>(src, dst, q);
    wire_scan<<<1, 1024, 0, st>>>(src, dst, q, reinterpret_cast<u64 *>(count_out), to_v2 ? 1u : 0u);
    if (to_v2) to_v2_words<<<grid, kWireThreads, 0, st>>>(src, dst, q);
    else from_v2_words<<<grid, kWireThreads, 0, st>>>(src, dst, q);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

ADACOMP_STATUS_HOOKS(wire)

}  // namespace adacomp_impl
