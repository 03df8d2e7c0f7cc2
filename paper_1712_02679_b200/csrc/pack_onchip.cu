// pack() of a layer that fits on the chip, in one kernel and one visit of the residue (Algorithm 2; scale of
// Section 2.5).  Every sent element's new residue needs the layer-wide scale, which is known only when every bin
// has been seen; the three-kernel pack() therefore writes residue = G first and revisits the sent elements.  Here
// the tiles stay in shared memory instead: each CTA keeps the G of up to four tiles, all CTAs meet once (a
// cooperative launch: they are all resident), every CTA works the scale out from the exact sum, subtracts
// sign(G) * scale from the sent elements in shared memory and writes each tile of the residue once.
// Traffic: dW and residue read once, residue written once, words and counts: the algorithmic 12.1 bytes per
// element.  Capacity: 4 tiles x 2 CTAs per SM (4.7 M elements on 148 SMs); larger layers take the three kernels.
// Bin lengths: the seven of the specialised tile pass (tiles of exactly 4000 elements); fp32 gradient, no flags.
//
// Phase 1 is tile_pass_fast's tile code (thread t < 160 owns 25 consecutive elements; a bin is SPB adjacent
// segments) with the residue tile loaded straight into the slot it stays in.  The meeting point is a counter in
// the scratch's control block; the wait on it is bounded like every other wait of the library.
#include "pack_onchip.cuh"

namespace adacomp_impl {

template <int SPB, typename Word>
__global__ void __launch_bounds__(kFastThreads, 2)
pack_onchip(PassArgs a, u64 *count_out, u32 header_flags)
{
    extern __shared__ __align__(128) unsigned char smem[];
    u32 *s_mask = reinterpret_cast<u32 *>(smem + OnchipSmem::kMaskAt);
    u64 *s_sums = reinterpret_cast<u64 *>(smem + OnchipSmem::kSumsAt);
    u64 *s_acc = reinterpret_cast<u64 *>(smem + OnchipSmem::kAccAt);
    u64 *s_res_bar = reinterpret_cast<u64 *>(smem + OnchipSmem::kBarAt);
    u64 *s_grad_bar = s_res_bar + kOnchipSlots;
    volatile u32 *s_misc = reinterpret_cast<volatile u32 *>(smem + OnchipSmem::kMiscAt);     // [0] scale bits, [1] abort
    volatile u32 *s_tcnt = s_misc + 4;                                                       // [4] words of the CTA's tiles

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const Geometry &geo = a.geo;
    // a CTA's tiles are neighbours (the launcher sizes the grid so that no CTA has more than kOnchipSlots)
    const u64 per_cta = (geo.n_tiles + gridDim.x - 1) / gridDim.x;
    const u64 first = blockIdx.x * per_cta;
    const int my_tiles = (int)min((u64)kOnchipSlots, geo.n_tiles > first ? min(per_cta, geo.n_tiles - first) : 0);
    const u64 full_tiles = geo.n / (u64)kFastTile;
    u32 *tile_cnt = reinterpret_cast<u32 *>(a.scratch + geo.tile_cnt_at);

    if (tid < kWindows + 1) s_acc[tid] = 0;
    if (tid == 0) {
        s_misc[1] = 0;
        for (int s = 0; s < kOnchipSlots + kOnchipStages; s++) mbar_init(&s_res_bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    auto slot_of = [&](int i) { return reinterpret_cast<float *>(smem + OnchipSmem::kSlotsAt) + i * kFastTile; };
    auto stage_of = [&](int i) { return reinterpret_cast<float *>(smem + OnchipSmem::kGradAt) + (i % kOnchipStages) * kFastTile; };
    auto issue_grad = [&](int i) {          // (service lane 0) the gradient of the CTA's tile i
        const u64 tile = first + (u64)i;
        if (i >= my_tiles || tile >= full_tiles) return;
        u64 *bar = &s_grad_bar[i % kOnchipStages];
        mbar_arrive_expect_tx(bar, kTileBytes);
        bulk_load(stage_of(i), a.grad + tile * (u64)kFastTile, kTileBytes, bar);
    };
    if (service && lane == 0) {
        for (int i = 0; i < my_tiles; i++) {
            const u64 tile = first + (u64)i;
            if (tile >= full_tiles) continue;           // the ragged last tile is read with plain loads
            mbar_arrive_expect_tx(&s_res_bar[i], kTileBytes);
            bulk_load(slot_of(i), a.residue + tile * (u64)kFastTile, kTileBytes, &s_res_bar[i]);
        }
        issue_grad(0);
        issue_grad(1);
    }

    // ================= phase 1: G, bin maxima, selection, words, counts; G stays in the slot =================
    for (int i = 0; i < my_tiles; i++) {
        const u64 tile = first + (u64)i;
        const OnchipTile t{a.grad, a.residue, tile, geo.n, geo.n_bins, a.packed + geo.bin_cnt_at,
                           a.scratch + geo.slots_at + tile * geo.slot_bytes, tile_cnt, a.factor, a.wait_limit, tile < full_tiles};
        onchip_tile<SPB, Word>(smem, i, t);
        if (service && lane == 0) issue_grad(i + kOnchipStages);          // the stage of tile i is free again
    }
    // ================= all CTAs meet: every bin has been seen =================
    if (service && lane < kWindows) {
        const u64 v = s_acc[lane];
        if (v) atomicAdd(reinterpret_cast<u64 *>(a.scratch) + lane, v);
    }
    __syncthreads();
    if (tid == 0) {
        u32 *meet = reinterpret_cast<u32 *>(a.scratch + kCtlMeetAt);
        __threadfence();
        atomicAdd(meet, 1u);
        const long long t0 = clock64();
        while (*reinterpret_cast<volatile u32 *>(meet) < gridDim.x) {
            if (clock64() - t0 > a.wait_limit) {
                raise_status(ADACOMP_DEV_TIMEOUT);      // (what follows reads whatever is there; every access stays in bounds)
                break;
            }
        }
        __threadfence();
    }
    __syncthreads();
    // the exact sum (warp 0), the tiles' counts (everyone) and the bin counts' running sums (warps 1..4), all in flight together
    {
        const u64 window = (warp == 0 && lane < kWindows) ? __ldcg(reinterpret_cast<const u64 *>(a.scratch) + lane) : 0ull;
        u64 below = 0, all = 0;
        for (u64 t = tid; t < geo.n_tiles; t += kFastThreads) {
            const u64 c = min(__ldcg(&tile_cnt[t]), (u32)kFastTile);
            if (t < first) below += c;
            all += c;
        }
        for (int d = 16; d > 0; d >>= 1) {
            below += __shfl_xor_sync(0xffffffffu, below, d);
            all += __shfl_xor_sync(0xffffffffu, all, d);
        }
        if (lane == 0) {
            s_sums[warp * 2] = below;
            s_sums[warp * 2 + 1] = all;
        }
        if (warp == 0) {
            if (lane < kWindows) s_acc[lane] = window;
            __syncwarp();
            if (lane == 0) {
                const double S = windows_to_double(s_acc);
                const float scale = geo.n_bins ? __double2float_rn(__ddiv_rn(S, (double)geo.n_bins)) : 0.f;
                s_misc[0] = __float_as_uint(scale);
            }
        }
        __syncthreads();
    }
    u64 off0 = 0, n_sel = 0;
    for (int wv = 0; wv < 6; wv++) {
        off0 += s_sums[wv * 2];
        n_sel += s_sums[wv * 2 + 1];
    }
    const float scale = __uint_as_float(s_misc[0]);

    // ================= phase 2: the sent elements' residues, one store per tile, the words' final place =================
    if (!service) {
        for (int i = 0; i < my_tiles; i++) {
            float *pr = slot_of(i) + tid * kSeg;
            u32 mask = s_mask[i * kTileSegs + tid];
            while (mask) {
                const int j = __ffs(mask) - 1;
                mask &= mask - 1;
                const float gq = pr[j];
                pr[j] = gq < 0.f ? __fadd_rn(gq, scale) : __fsub_rn(gq, scale);      // G - sign(G) * scale
            }
        }
    }
    fence_async_smem();
    __syncthreads();
    for (int i = 0; i < my_tiles; i++) {
        const u64 tile = first + (u64)i;
        const u64 base = tile * (u64)kFastTile;
        if (tile < full_tiles) {
            if (tid == 0) {
                bulk_store(a.residue + base, slot_of(i), kTileBytes);
                bulk_commit();
            }
        } else {
            const int elems = (int)(geo.n - base);
            for (int e = tid; e < elems; e += kFastThreads) a.residue[base + e] = slot_of(i)[e];
        }
    }
    // (the CTA's tiles are neighbours, so their words are one run of the stream)
    u64 *tile_off = reinterpret_cast<u64 *>(a.packed + geo.tile_off_at);
    Word *payload = reinterpret_cast<Word *>(a.packed + geo.payload_at);
    {
        const u32 c0 = my_tiles > 0 ? min(s_tcnt[0], (u32)kFastTile) : 0u, c1 = my_tiles > 1 ? min(s_tcnt[1], (u32)kFastTile) : 0u;
        const u32 c2 = my_tiles > 2 ? min(s_tcnt[2], (u32)kFastTile) : 0u, c3 = my_tiles > 3 ? min(s_tcnt[3], (u32)kFastTile) : 0u;
        const u32 cum1 = c0, cum2 = c0 + c1, cum3 = cum2 + c2, total = cum3 + c3;
        if (tid < my_tiles) tile_off[first + tid] = off0 + (tid == 0 ? 0u : tid == 1 ? cum1 : tid == 2 ? cum2 : cum3);
        const unsigned char *slots = a.scratch + geo.slots_at + first * geo.slot_bytes;
        constexpr int kAhead = 4;       // words a thread has in flight
        for (u32 v0 = tid; v0 < total; v0 += kAhead * kFastThreads) {
            u32 word[kAhead];
#pragma unroll
            for (int k = 0; k < kAhead; k++) {
                const u32 v = v0 + k * kFastThreads;
                const int ti = (int)(v >= cum1) + (int)(v >= cum2) + (int)(v >= cum3);
                const u32 j = v - (ti == 0 ? 0u : ti == 1 ? cum1 : ti == 2 ? cum2 : cum3);
                word[k] = v < total ? (u32) reinterpret_cast<const Word *>(slots + ti * geo.slot_bytes)[j] : 0u;
            }
#pragma unroll
            for (int k = 0; k < kAhead; k++) {
                const u32 v = v0 + k * kFastThreads;
                if (v < total) payload[off0 + v] = (Word)word[k];
            }
        }
    }
    // ================= the header (one CTA) =================
    if (blockIdx.x == 0) onchip_header(a.packed, geo, header_flags, scale, n_sel, count_out);
    if (tid == 0) bulk_wait_read_all();     // the stores have read shared memory before the CTA gives it up
}

template <int SPB, typename Word>
static bool onchip_allow(int *per_sm)
{
    if (cudaFuncSetAttribute(pack_onchip<SPB, Word>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)OnchipSmem::kBytes) != cudaSuccess)
        return false;
    int per = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, pack_onchip<SPB, Word>, kFastThreads, OnchipSmem::kBytes);
    *per_sm = *per_sm < per ? *per_sm : per;
    return per > 0;
}

void init_pack_onchip_info(DeviceInfo &d)
{
    int dev = 0, coop = 0, per = 2;
    d.onchip_ctas = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop)
        return;
    if (!(onchip_allow<2, unsigned char>(&per) && onchip_allow<4, unsigned short>(&per) && onchip_allow<5, unsigned short>(&per) &&
          onchip_allow<8, unsigned short>(&per) && onchip_allow<10, unsigned short>(&per) && onchip_allow<20, unsigned short>(&per) &&
          onchip_allow<40, unsigned short>(&per)))
        return;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
    d.onchip_ctas = sms * per;              // CTAs that are resident together: kOnchipSlots tiles each
}

u64 onchip_tile_capacity(const DeviceInfo &d) { return (u64)d.onchip_ctas * kOnchipSlots; }

template <int SPB, typename Word>
static int onchip_launch(PassArgs &args, u64 *count_out, u32 header_flags, unsigned grid, cudaStream_t st)
{
    void *params[] = {&args, &count_out, &header_flags};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(pack_onchip<SPB, Word>), dim3(grid), dim3(kFastThreads), params,
                                       OnchipSmem::kBytes, st) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

// The whole of pack() for a layer of at most onchip_tile_capacity() tiles (the caller has zeroed the control block).
int launch_pack_onchip(PassArgs &args, u64 *count_out, u32 header_flags, const DeviceInfo &info, cudaStream_t st)
{
    const u64 n_tiles = args.geo.n_tiles;
    // as few tiles per CTA as the resident CTAs allow (every CTA then has the same number, give or take one)
    const u64 per_cta = (n_tiles + (u64)info.onchip_ctas - 1) / (u64)info.onchip_ctas;
    const unsigned grid = (unsigned)((n_tiles + per_cta - 1) / per_cta);
    switch (args.geo.L_T) {
    case 50u: return onchip_launch<2, unsigned char>(args, count_out, header_flags, grid, st);
    case 100u: return onchip_launch<4, unsigned short>(args, count_out, header_flags, grid, st);
    case 125u: return onchip_launch<5, unsigned short>(args, count_out, header_flags, grid, st);
    case 200u: return onchip_launch<8, unsigned short>(args, count_out, header_flags, grid, st);
    case 250u: return onchip_launch<10, unsigned short>(args, count_out, header_flags, grid, st);
    case 500u: return onchip_launch<20, unsigned short>(args, count_out, header_flags, grid, st);
    case 1000u: return onchip_launch<40, unsigned short>(args, count_out, header_flags, grid, st);
    default: return ADACOMP_ERR_UNSUPPORTED;
    }
}

ADACOMP_STATUS_HOOKS(pack_onchip)

}  // namespace adacomp_impl
