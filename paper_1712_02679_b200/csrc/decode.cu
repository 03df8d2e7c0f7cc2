// unpack() and the ordered sum of one tensor: the plain decoders and their launcher (see decode_words.cuh).
#include "internal.h"

namespace adacomp_impl {

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


void init_decode_opt_info(DeviceInfo &d);       // decode_opt.cu

void init_decode_info(DeviceInfo &d)
{
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum, kDecodeThreads, 0);
    d.decode_per_sm = per_sm < 1 ? 1 : per_sm;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum_warps<0, 4>, kDecodeLaunch, 0);
    d.decode_warps_per_sm = per_sm < 1 ? 1 : per_sm;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_sum_warps<0, 4, true>, kDecodeLaunch, 0);
    d.decode_one_per_sm = per_sm < 1 ? 1 : per_sm;
    d.decode_pair_per_sm = 0;
    if (cudaFuncSetAttribute(decode_sum_warps<0, 5, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)kPairSmemBytes) == cudaSuccess) {
        int per = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, decode_sum_warps<0, 5, false, 2>, 6 * 32, kPairSmemBytes);
        d.decode_pair_per_sm = per;
    }
    init_decode_opt_info(d);
}

// `ep` (optional): the optimizer step that takes the place of the store to dst (dst is null then).
int decompress_impl(const void *const *packed, uint32_t k, float *dst, void *stream, uint64_t hint_n,
                    uint32_t hint_L_T, const Epilogue *ep)
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
    args.wait_limit = debug_waits().limit;
    args.withhold = debug_waits().withhold_decode;
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
        return launch_decode_opt(args, *ep, *info, hint_n, hint_L_T, st);
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


ADACOMP_STATUS_HOOKS(decode)

}  // namespace adacomp_impl
