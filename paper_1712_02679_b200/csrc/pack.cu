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


// This file: the single-layer pack() launcher, its generic, finalize and gather kernels, the lazy-scale
// state's upkeep and the entry point with the library's own scratch.
#include "internal.h"

namespace adacomp_impl {

__global__ void __launch_bounds__(1024)
finalize(unsigned char *packed, unsigned char *scratch, Geometry geo, u32 flags, u64 *count_out,
         unsigned char *lazy_state)
{
    finalize_body(packed, scratch, geo, flags, count_out, lazy_state);
}


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


void init_pack_info(DeviceInfo &d)
{
    d.fast_ready = fast_tile_pass_a(nullptr, 0, nullptr) && fast_tile_pass_b(nullptr, 0, nullptr) &&
                   fast_tile_pass_c(nullptr, 0, nullptr) && fast_tile_pass_d(nullptr, 0, nullptr);
}

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
                  uint64_t *count_out, void *stream, uint32_t flags, void *const *events, void *lazy_state,
                  float factor, uint32_t grad_type, unsigned char *own_scratch, uint32_t quantiser)
{
    if (!packed_out || !count_out || (n && (!grad || !residue))) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH | ADACOMP_FLAG_STREAMING)) return ADACOMP_ERR_FLAGS;
    const bool streaming = (flags & ADACOMP_FLAG_STREAMING) != 0;       // (the flag chooses among kernels that give the same bytes)
    flags &= ~ADACOMP_FLAG_STREAMING;
    if (factor != 0.f && !(factor > 0.f && factor <= 1e30f)) return ADACOMP_ERR_FLAGS;
    if (grad_type > ADACOMP_GRAD_F16 || quantiser > ADACOMP_QUANT_SENT_MEAN) return ADACOMP_ERR_FLAGS;
    if (misaligned(grad) || misaligned(residue) || misaligned(packed_out) ||
        (reinterpret_cast<uintptr_t>(count_out) & 7u))
        return ADACOMP_ERR_ALIGN;
    const Geometry geo = make_geometry(n, L_T);
    if (geo.n_bins >= (1ull << 31)) return ADACOMP_ERR_SIZE;
    unsigned char *lazy = static_cast<unsigned char *>(lazy_state);
    if (lazy) {
        if (!(fast_L_T(L_T) || any_fast_L_T(L_T)) || flags != 0) return ADACOMP_ERR_UNSUPPORTED;
        // (16-bit gradients: the any-bin form needs tiles of them to start on 16-byte boundaries)
        if (grad_type != ADACOMP_GRAD_F32 && !fast_L_T(L_T) && geo.tile_elems % 8u != 0) return ADACOMP_ERR_UNSUPPORTED;
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
    // a layer whose tiles all fit in the shared memory of the CTAs that are resident together: one kernel, the
    // residue visited once (pack_onchip.cu)
    if (!lazy && !streaming && flags == 0 && fast_L_T(L_T) && grad_type == ADACOMP_GRAD_F32 && quantiser == 0 && geo.n_tiles != 0 &&
        geo.n_tiles <= onchip_tile_capacity(*info) && debug_waits().withhold_pack == 0) {
        PassArgs args{grad, residue, packed, scratch, geo, 0u, nullptr, factor, grad_type, quantiser, debug_waits().limit, 0u};
        rc = launch_pack_onchip(args, reinterpret_cast<u64 *>(count_out), factor != 0.f ? kFlagFactor : 0u, *info, st);
        mark(1);
        mark(2);
        mark(3);
        return rc;
    }
    if (geo.n_tiles) {
        PassArgs args{grad, residue, packed, scratch, geo, flags & ADACOMP_FLAG_LITERAL, lazy, factor, grad_type,
                      quantiser, debug_waits().limit, debug_waits().withhold_pack};
        const bool fast = fast_L_T(L_T) && flags == 0 && info->fast_ready;
        // (one-bin tiles fill the pipelined kernel's 4000-element stages only in part: below 2800 elements the
        // warp-per-part kernel is faster, measured; lazy-scale mode exists in the pipelined kernel only)
        const bool any_fast = any_fast_L_T(L_T) && flags == 0 && info->fast_ready &&
                              (grad_type == ADACOMP_GRAD_F32 || geo.tile_elems % 8u == 0) &&
                              (lazy || L_T <= 1000u || L_T >= 2800u);
        if (fast || any_fast) {
            const u64 cap = (u64)info->sms * 2;
            const unsigned grid = (unsigned)(geo.n_tiles < cap ? geo.n_tiles : cap);
            if (!(fast_tile_pass_a(&args, grid, st) || fast_tile_pass_b(&args, grid, st) ||
                  fast_tile_pass_c(&args, grid, st) || fast_tile_pass_d(&args, grid, st)))
                return ADACOMP_ERR_UNSUPPORTED;
        } else {
            rc = geo.w == 1u ? launch_generic<unsigned char>(args, *info, st)
                             : launch_generic<unsigned short>(args, *info, st);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    mark(1);
    const u32 header_flags = flags | (factor != 0.f ? kFlagFactor : 0u) | (quantiser ? kFlagQuant : 0u);
    // (layers of at most kFoldGroups groups of tiles: the gather does finalize's work itself, a launch fewer)
    const bool fold = geo.n_tiles != 0 && geo.tile_bins <= (u32)kSmallBins && geo.n_groups <= (u64)kFoldGroups;
    if (!fold) finalize<<<1, 1024, 0, st>>>(packed, scratch, geo, header_flags, reinterpret_cast<u64 *>(count_out), lazy);
    mark(2);
    if (geo.n_tiles) {
        if (geo.tile_bins <= (u32)kSmallBins) {
            const u64 want = (geo.n_tiles + 3) / 4, cap = (u64)info->sms * 16;
            const unsigned grid = (unsigned)(want < cap ? want : cap);
            u64 *const co = reinterpret_cast<u64 *>(count_out);
            if (fold) {
                if (lazy) {     // the residue keeps G; only the words move
                    if (geo.w == 1u) gather_fixup_fold<unsigned char, false><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo, header_flags, co, lazy);
                    else gather_fixup_fold<unsigned short, false><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo, header_flags, co, lazy);
                } else {
                    if (geo.w == 1u) gather_fixup_fold<unsigned char, true><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo, header_flags, co, lazy);
                    else gather_fixup_fold<unsigned short, true><<<grid, kGatherThreads, 0, st>>>(residue, packed, scratch, geo, header_flags, co, lazy);
                }
            } else if (lazy) {
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
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, nullptr, 0.f, ADACOMP_GRAD_F32,
                         g_static_scratch_addr[dev], ADACOMP_QUANT_BIN_MAX_MEAN);
}


int lazy_state_init(void *state, uint64_t n, uint32_t L_T, void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(state, 0, lazy_state_bytes(make_geometry(n, L_T)), st) != cudaSuccess) return ADACOMP_ERR_CUDA;
    lazy_init_kernel<<<1, 1, 0, st>>>(static_cast<unsigned char *>(state), n, L_T);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int residue_flush(float *residue, void *state, uint64_t n, uint32_t L_T, void *stream)
{
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

ADACOMP_STATUS_HOOKS(pack)

}  // namespace adacomp_impl
