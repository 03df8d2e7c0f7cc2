// Shared by every translation unit of libadacomp: types, constants, the stream's geometry, small device
// helpers, and the mbarrier / bulk-copy (TMA) wrappers (no cluster multicast anywhere).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "adacomp.h"

namespace adacomp_impl {

typedef unsigned long long u64;
typedef unsigned int u32;

constexpr u32 kMagic = 0x31434441u;
constexpr u32 kFlagFactor = 2u;       // header flag (set by the library): the stream was made with a scale-factor
constexpr u32 kFlagQuant = 4u;        // header flag (set by the library): the scale is the mean |G| of the sent elements
constexpr u32 kCtlSentSumAt = 128;    // control block: the nine windows of the exact sum of the sent |G| (second quantiser)
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

// Sticky ADACOMP_DEV_* bits of this device.  Every translation unit of the library is whole-program device code
// with its own copy of this word (no relocatable device code: it costs the kernels registers); the ABI's status
// call reads them all and ORs them together, see ADACOMP_STATUS_HOOKS below and abi.cu.
static __device__ u32 g_status;

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
__device__ inline float load_grad(const float *grad, u64 i, u32 grad_type)
{
    if (grad_type == ADACOMP_GRAD_BF16) return __uint_as_float((u32)reinterpret_cast<const unsigned short *>(grad)[i] << 16);
    if (grad_type == ADACOMP_GRAD_F16) return __half2float(__ushort_as_half(reinterpret_cast<const unsigned short *>(grad)[i]));
    return grad[i];
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

// The same into an accumulator that several warps of the CTA share (shared-memory atomics).
__device__ inline void warp_accumulate_shared(u64 *acc, float v, bool valid)
{
    const u32 full = 0xffffffffu;
    u32 window = 0;
    u64 lo = 0, hi = 0;
    valid = valid && split_for_sum(v, window, lo, hi);
    const u32 vm = __ballot_sync(full, valid);
    if (vm == 0) return;
    const u32 w0 = __shfl_sync(full, window, __ffs(vm) - 1);
    if (__all_sync(full, !valid || window == w0)) {
        if (!valid) { lo = 0; hi = 0; }
        for (int d = 16; d > 0; d >>= 1) {
            lo += __shfl_down_sync(full, lo, d);
            hi += __shfl_down_sync(full, hi, d);
        }
        if ((threadIdx.x & 31) == 0) { atomicAdd(&acc[w0], lo); atomicAdd(&acc[w0 + 1], hi); }
    } else if (valid) {
        atomicAdd(&acc[window], lo);
        atomicAdd(&acc[window + 1], hi);
    }
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

// Bounded wait: false if the phase did not complete within `limit` cycles.
__device__ inline bool mbar_wait(u64 *bar, u32 parity, long long limit = kWaitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (clock64() - t0 > limit) return false;
    }
    return true;
}

// What adacomp_debug_waits sets (a testing aid, see include/adacomp.h): the bound of the waits of the single-layer
// tile pass and of the single-tensor warp decoder, and which of CTA 0's loads its copy engine is to leave out
// (0: none) so that a wait runs out without anything being wrong with the device.
struct DebugWaits {
    long long limit;
    u32 withhold_pack, withhold_decode;
};

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

struct TrueType { static constexpr bool value = true; };
struct FalseType { static constexpr bool value = false; };

// One per .cu file that holds kernels: how abi.cu reads and clears that file's status word.
#define ADACOMP_STATUS_HOOKS(unit)                                                                        \
    __global__ void status_reset_kernel_##unit() { g_status = 0; }                                        \
    bool status_read_##unit(u32 *bits)                                                                     \
    {                                                                                                      \
        u32 v = 0;                                                                                         \
        if (cudaMemcpyFromSymbol(&v, g_status, sizeof(v)) != cudaSuccess) return false;                   \
        *bits |= v;                                                                                        \
        return true;                                                                                       \
    }                                                                                                      \
    void status_reset_##unit(cudaStream_t st) { status_reset_kernel_##unit<<<1, 1, 0, st>>>(); }
#define ADACOMP_STATUS_DECLARE(unit)                                                                      \
    bool status_read_##unit(u32 *bits);                                                                    \
    void status_reset_##unit(cudaStream_t st);

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

}  // namespace adacomp_impl
