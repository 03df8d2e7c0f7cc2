// unpack(), averageGradients() and updateWeights() in one kernel: the decoders with an optimizer step (SGD with
// momentum, Adam) in place of the store, and their launcher (see decode_words.cuh: decode_sum_warps, Epilogue).
#include "internal.h"

namespace adacomp_impl {

void init_decode_opt_info(DeviceInfo &d)
{
    auto opt_ready = [&](auto kernel, int threads, u32 smem) -> int {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
        int per = 0;
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per, kernel, threads, smem);
        return per;
    };
    d.decode_opt_per_sm[0][0] = opt_ready(decode_sum_warps<1, 4>, 5 * 32, opt_smem_bytes(1));
    d.decode_opt_per_sm[0][1] = opt_ready(decode_sum_warps<1, 8>, 9 * 32, opt_smem_bytes(1));
    d.decode_opt_per_sm[1][0] = opt_ready(decode_sum_warps<2, 4>, 5 * 32, opt_smem_bytes(2));
    d.decode_opt_per_sm[1][1] = opt_ready(decode_sum_warps<2, 8>, 9 * 32, opt_smem_bytes(2));
    // (the kernels of the one-bin tiles: same shared memory and launch bounds as their four-warp siblings)
    if (!opt_ready(decode_sum_warps<1, 4, true>, 5 * 32, opt_smem_bytes(1))) d.decode_opt_per_sm[0][0] = 0;
    if (!opt_ready(decode_sum_warps<2, 4, true>, 5 * 32, opt_smem_bytes(2))) d.decode_opt_per_sm[1][0] = 0;
}

int launch_decode_opt(const DecodeArgs &args, const Epilogue &ep_ref, const DeviceInfo &info_ref, uint64_t hint_n,
                      uint32_t hint_L_T, cudaStream_t st)
{
    const Epilogue *ep = &ep_ref;
    const DeviceInfo *info = &info_ref;

        // (the optimizer entry points always pass the shape)
        // (eight warps where they divide the tile's bins, unless four can work a lane per bin; Adam's two CTAs per
        // SM need the eight all the same: 7.0 against 6.1 ms at 2^30 elements, L_T = 50)
        const Geometry og = make_geometry(hint_n, hint_L_T ? hint_L_T : 1u);
        const bool eight = hint_L_T && og.tile_bins % 8u == 0 && (ep->adam || !lanes_shape(og.tile_bins, 4u, og.w));
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
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

ADACOMP_STATUS_HOOKS(decode_opt)

}  // namespace adacomp_impl
