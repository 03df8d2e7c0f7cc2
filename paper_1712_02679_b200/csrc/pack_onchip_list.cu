// pack() of a whole parameter list that fits on the chip, in one kernel (see pack_onchip.cu for the single layer):
// the tiles of all layers are numbered through, a CTA keeps up to four neighbouring tiles' G in shared memory
// (they may lie in different layers, of different bin lengths), all CTAs meet once, and every CTA then works out,
// for each of its tiles, the tile's layer's scale (Section 2.5) and the tile's place in that layer's stream,
// finishes the sent elements' residues in shared memory and writes each residue tile once.  The CTA that holds a
// layer's first tile writes that layer's header.  Two launches (control blocks cleared, this kernel) replace the
// four of the batch kernels; it takes lists of fp32 gradients with the paper's two bin lengths, 50 and 500 (the
// tile code of more bin lengths side by side in one kernel left the compiler spilling kilobytes), eager mode, the
// paper's quantiser, with or without a factor per layer.
#include "pack_onchip.cuh"

namespace adacomp_impl {

template <int N>
__global__ void __launch_bounds__(kFastThreads, 2)
pack_onchip_list(const __grid_constant__ BatchArgsT<N> b, long long wait_limit)
{
    extern __shared__ __align__(128) unsigned char smem[];
    u32 *s_mask = reinterpret_cast<u32 *>(smem + OnchipSmem::kMaskAt);
    u64 *s_acc = reinterpret_cast<u64 *>(smem + OnchipSmem::kAccAt);
    u64 *s_res_bar = reinterpret_cast<u64 *>(smem + OnchipSmem::kBarAt);
    u64 *s_grad_bar = s_res_bar + kOnchipSlots;
    volatile u32 *s_misc = reinterpret_cast<volatile u32 *>(smem + OnchipSmem::kMiscAt);     // [1] abort
    volatile u32 *s_tcnt = s_misc + 4;                                                       // [4] words of the CTA's tiles
    __shared__ u32 s_tile_first[N];
    __shared__ int s_li[kOnchipSlots];                  // the CTA's tiles: layer,
    __shared__ u32 s_lt[kOnchipSlots];                  // number in the layer,
    __shared__ u64 s_off[kOnchipSlots], s_all[kOnchipSlots];    // words of the layer before the tile, words of the layer,
    __shared__ u32 s_scale[kOnchipSlots];               // the layer's scale (bits)
    __shared__ u64 s_win[kOnchipSlots][kWindows + 1];
    __shared__ u64 s_part[6][2 * kOnchipSlots];         // per warp: partial sums of tile counts

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool service = warp == 5;
    const int n_layers = (int)b.n_layers;
    // a CTA's tiles are neighbours (the launcher sizes the grid so that no CTA has more than kOnchipSlots)
    const u32 per_cta = (b.total_tiles + gridDim.x - 1) / gridDim.x;
    const u32 first = blockIdx.x * per_cta;
    const int my_tiles = (int)min((u32)kOnchipSlots, b.total_tiles > first ? min(per_cta, b.total_tiles - first) : 0u);

    for (int l = tid; l < n_layers; l += kFastThreads) s_tile_first[l] = b.layer[l].tile_first;
    if (tid < kWindows + 1) s_acc[tid] = 0;
    if (tid == 0) {
        s_misc[1] = 0;
        for (int s = 0; s < kOnchipSlots + kOnchipStages; s++) mbar_init(&s_res_bar[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid < my_tiles) {
        const u32 gt = first + (u32)tid;
        int lo = 0, hi = n_layers;                      // the largest l with tile_first[l] <= gt
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_tile_first[mid] <= gt) lo = mid; else hi = mid;
        }
        s_li[tid] = lo;
        s_lt[tid] = gt - s_tile_first[lo];
    }
    __syncthreads();

    auto slot_of = [&](int i) { return reinterpret_cast<float *>(smem + OnchipSmem::kSlotsAt) + i * kFastTile; };
    auto stage_of = [&](int i) { return reinterpret_cast<float *>(smem + OnchipSmem::kGradAt) + (i % kOnchipStages) * kFastTile; };
    // (every layer here has tiles of exactly 4000 elements; all but a layer's last are whole, and that one may be)
    auto whole_tile = [&](int i) {
        const Geometry &g = b.layer[s_li[i]].geo;
        return (u64)s_lt[i] + 1 < g.n_tiles || g.n == g.n_tiles * (u64)kFastTile;
    };
    auto issue_grad = [&](int i) {          // (service lane 0) the gradient of the CTA's tile i
        if (i >= my_tiles || !whole_tile(i)) return;
        u64 *bar = &s_grad_bar[i % kOnchipStages];
        mbar_arrive_expect_tx(bar, kTileBytes);
        bulk_load(stage_of(i), b.layer[s_li[i]].grad + (u64)s_lt[i] * (u64)kFastTile, kTileBytes, bar);
    };
    if (service && lane == 0) {
        for (int i = 0; i < my_tiles; i++) {
            if (!whole_tile(i)) continue;               // a ragged last tile is read with plain loads
            mbar_arrive_expect_tx(&s_res_bar[i], kTileBytes);
            bulk_load(slot_of(i), b.layer[s_li[i]].residue + (u64)s_lt[i] * (u64)kFastTile, kTileBytes, &s_res_bar[i]);
        }
        issue_grad(0);
        issue_grad(1);
    }
    auto flush = [&](int li) {              // (service warp) this CTA's share of layer li's exact sum
        if (lane < kWindows) {
            const u64 v = s_acc[lane];
            if (v) atomicAdd(reinterpret_cast<u64 *>(b.layer[li].packed + b.layer[li].geo.scratch_at) + lane, v);
            s_acc[lane] = 0;
        }
        __syncwarp();
    };

    // ================= phase 1: G, bin maxima, selection, words, counts; G stays in the slot =================
    for (int i = 0; i < my_tiles; i++) {
        const int li = s_li[i];
        const BatchLayer &L = b.layer[li];
        const Geometry &geo = L.geo;
        if (service && i > 0 && li != s_li[i - 1]) flush(s_li[i - 1]);      // (before this tile's maxima are added)
        unsigned char *scratch = L.packed + geo.scratch_at;
        const u64 tile = s_lt[i];
        const OnchipTile t{L.grad, L.residue, tile, geo.n, geo.n_bins, L.packed + geo.bin_cnt_at,
                           scratch + geo.slots_at + tile * geo.slot_bytes, reinterpret_cast<u32 *>(scratch + geo.tile_cnt_at),
                           L.factor, wait_limit, whole_tile(i)};
        switch (geo.L_T) {                  // (uniform: the whole CTA works on the tile; the launcher lets 50 and 500 in)
        case 50u: onchip_tile<2, unsigned char>(smem, i, t); break;
        default: onchip_tile<20, unsigned short>(smem, i, t); break;        // 500
        }
        if (service && lane == 0) issue_grad(i + kOnchipStages);          // the stage of tile i is free again
    }
    if (service && my_tiles > 0) flush(s_li[my_tiles - 1]);

    // ================= all CTAs meet: every bin of every layer has been seen =================
    __syncthreads();
    if (tid == 0) {
        u32 *meet = reinterpret_cast<u32 *>(b.layer[0].packed + b.layer[0].geo.scratch_at + kCtlMeetAt);
        __threadfence();
        atomicAdd(meet, 1u);
        const long long t0 = clock64();
        while (*reinterpret_cast<volatile u32 *>(meet) < gridDim.x) {
            if (clock64() - t0 > wait_limit) {
                raise_status(ADACOMP_DEV_TIMEOUT);      // (what follows reads whatever is there; every access stays in bounds)
                break;
            }
        }
        __threadfence();
    }
    __syncthreads();
    // per tile of the CTA: the words of its layer before it and in all (everyone; the four tiles' loads in flight
    // together), the layer's exact sum (warp i)
    {
        u64 below[kOnchipSlots], all[kOnchipSlots];
#pragma unroll
        for (int i = 0; i < kOnchipSlots; i++) {
            below[i] = all[i] = 0;
            if (i < my_tiles) {
                const BatchLayer &L = b.layer[s_li[i]];
                const u32 *tile_cnt = reinterpret_cast<const u32 *>(L.packed + L.geo.scratch_at + L.geo.tile_cnt_at);
                const u32 lt = s_lt[i], n_tiles = (u32)L.geo.n_tiles;
                if (warp == i && lane < kWindows)
                    s_win[i][lane] = __ldcg(reinterpret_cast<const u64 *>(L.packed + L.geo.scratch_at) + lane);
                for (u32 t = tid; t < n_tiles; t += kFastThreads) {
                    const u64 c = min(__ldcg(&tile_cnt[t]), (u32)kFastTile);
                    if (t < lt) below[i] += c;
                    all[i] += c;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kOnchipSlots; i++) {
            for (int d = 16; d > 0; d >>= 1) {
                below[i] += __shfl_xor_sync(0xffffffffu, below[i], d);
                all[i] += __shfl_xor_sync(0xffffffffu, all[i], d);
            }
            if (lane == 0) {
                s_part[warp][2 * i] = below[i];
                s_part[warp][2 * i + 1] = all[i];
            }
        }
        __syncthreads();
        if (tid < 2 * kOnchipSlots) {
            u64 v = 0;
            for (int wv = 0; wv < 6; wv++) v += s_part[wv][tid];
            if (tid & 1) s_all[tid >> 1] = v; else s_off[tid >> 1] = v;
        }
    }
    if (warp < my_tiles && lane == 0) {
        const Geometry &geo = b.layer[s_li[warp]].geo;
        const double S = windows_to_double(s_win[warp]);
        s_scale[warp] = __float_as_uint(geo.n_bins ? __double2float_rn(__ddiv_rn(S, (double)geo.n_bins)) : 0.f);
    }
    __syncthreads();

    // ================= phase 2: the sent elements' residues, one store per tile, the words' final place =================
    if (!service) {
        for (int i = 0; i < my_tiles; i++) {
            const float scale = __uint_as_float(s_scale[i]);
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
        const BatchLayer &L = b.layer[s_li[i]];
        const u64 base = (u64)s_lt[i] * (u64)kFastTile;
        if (whole_tile(i)) {
            if (tid == 0) {
                bulk_store(L.residue + base, slot_of(i), kTileBytes);
                bulk_commit();
            }
        } else {
            const int elems = (int)(L.geo.n - base);
            for (int e = tid; e < elems; e += kFastThreads) L.residue[base + e] = slot_of(i)[e];
        }
    }
    // the words' final place: the loads of all the CTA's tiles first, then the stores
    {
        constexpr int kAhead = 4;           // rounds of a tile's words a thread has in flight
        u32 word[kOnchipSlots][kAhead];
#pragma unroll
        for (int i = 0; i < kOnchipSlots; i++) {
            if (i < my_tiles) {
                const BatchLayer &L = b.layer[s_li[i]];
                const u32 cnt = min(s_tcnt[i], (u32)kFastTile);
                const unsigned char *slot = L.packed + L.geo.scratch_at + L.geo.slots_at + (u64)s_lt[i] * L.geo.slot_bytes;
#pragma unroll
                for (int k = 0; k < kAhead; k++) {
                    const u32 j = tid + k * kFastThreads;
                    word[i][k] = 0;
                    if (j < cnt) word[i][k] = L.geo.w == 1u ? (u32)slot[j] : (u32) reinterpret_cast<const unsigned short *>(slot)[j];
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kOnchipSlots; i++) {
            if (i < my_tiles) {
                const BatchLayer &L = b.layer[s_li[i]];
                const Geometry &geo = L.geo;
                const u32 cnt = min(s_tcnt[i], (u32)kFastTile);
                const u64 off = s_off[i];
                const unsigned char *slot = L.packed + geo.scratch_at + geo.slots_at + (u64)s_lt[i] * geo.slot_bytes;
                unsigned char *payload = L.packed + geo.payload_at;
                if (tid == 0) reinterpret_cast<u64 *>(L.packed + geo.tile_off_at)[s_lt[i]] = off;
                if (geo.w == 1u) {
#pragma unroll
                    for (int k = 0; k < kAhead; k++) {
                        const u32 j = tid + k * kFastThreads;
                        if (j < cnt) payload[off + j] = (unsigned char)word[i][k];
                    }
                    for (u32 j = tid + kAhead * kFastThreads; j < cnt; j += kFastThreads) payload[off + j] = slot[j];     // (a dense tile)
                } else {
                    const unsigned short *src = reinterpret_cast<const unsigned short *>(slot);
                    unsigned short *dst = reinterpret_cast<unsigned short *>(payload) + off;
#pragma unroll
                    for (int k = 0; k < kAhead; k++) {
                        const u32 j = tid + k * kFastThreads;
                        if (j < cnt) dst[j] = (unsigned short)word[i][k];
                    }
                    for (u32 j = tid + kAhead * kFastThreads; j < cnt; j += kFastThreads) dst[j] = src[j];
                }
                // the CTA with a layer's first tile writes the layer's header
                if (s_lt[i] == 0u)
                    onchip_header(L.packed, geo, L.factor != 0.f ? kFlagFactor : 0u, __uint_as_float(s_scale[i]), s_all[i], L.count_out);
            }
        }
    }
    if (tid == 0) bulk_wait_read_all();     // the stores have read shared memory before the CTA gives it up
}

template <int N>
static int list_allow()
{
    if (cudaFuncSetAttribute(pack_onchip_list<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)OnchipSmem::kBytes) != cudaSuccess)
        return 0;
    int per = 0;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, pack_onchip_list<N>, kFastThreads, OnchipSmem::kBytes);
    return per;
}

void init_pack_onchip_list_info(DeviceInfo &d)
{
    d.onchip_list_ctas = 0;
    if (d.onchip_ctas <= 0) return;         // (no cooperative launch, or the single-layer kernel does not fit)
    const int a = list_allow<kBatchSmall>(), c = list_allow<kBatchMax>();
    const int per = a < c ? a : c;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
    if (per > 0) d.onchip_list_ctas = sms * (per < 2 ? per : 2);
}

template <int N>
static int list_launch(const BatchArgsT<N> &b, const DeviceInfo &info, long long wait_limit, cudaStream_t st)
{
    const u64 ctas = (u64)info.onchip_list_ctas;
    const u64 per_cta = ((u64)b.total_tiles + ctas - 1) / ctas;
    const unsigned grid = (unsigned)(((u64)b.total_tiles + per_cta - 1) / per_cta);
    void *params[] = {const_cast<BatchArgsT<N> *>(&b), &wait_limit};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void *>(pack_onchip_list<N>), dim3(grid), dim3(kFastThreads), params,
                                       OnchipSmem::kBytes, st) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

// Whether the one-kernel form takes this batch: every layer an fp32 gradient with bin length 50 or 500
// (the caller has checked eager mode and the quantiser), all tiles resident at once.
bool onchip_list_takes(const BatchArgs &b, const DeviceInfo &info)
{
#ifdef ADACOMP_NO_ONCHIP_LIST
    return false;
#endif
    if (info.onchip_list_ctas <= 0 || b.n_layers == 0 || b.total_tiles == 0) return false;
    // (up to two tiles per CTA: beyond that the batch kernels' pipelines, which keep loads, work and stores going side
    // by side, beat this kernel's burst of loads at the start and of stores at the end when the data come from DRAM:
    // the LSTM list, three tiles per CTA, 26.9 against 22.7 us per learner)
    if ((u64)b.total_tiles > (u64)info.onchip_list_ctas * 2) return false;
    for (u32 i = 0; i < b.n_layers; i++) {
        const BatchLayer &L = b.layer[i];
        if ((L.geo.L_T != 50u && L.geo.L_T != 500u) || L.grad_type != ADACOMP_GRAD_F32 || L.lazy != nullptr || L.geo.n_tiles == 0) return false;
    }
    return true;
}

// The layers' control blocks must be zero (launch_batch's clear kernel has run).
int launch_pack_onchip_list(const BatchArgs &b, const DeviceInfo &info, long long wait_limit, cudaStream_t st)
{
    if (b.n_layers <= (u32)kBatchSmall) {
        static thread_local BatchArgsT<kBatchSmall> small;
        small.n_layers = b.n_layers;
        small.total_tiles = b.total_tiles;
        for (u32 i = 0; i < b.n_layers; i++) small.layer[i] = b.layer[i];
        return list_launch(small, info, wait_limit, st);
    }
    return list_launch(b, info, wait_limit, st);
}

ADACOMP_STATUS_HOOKS(pack_onchip_list)

}  // namespace adacomp_impl
