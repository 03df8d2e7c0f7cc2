// Pipelined tile pass, bin lengths 1000 and the any-bin form (see pack_tile.cuh: tile_pass_fast).
#include "pack_fast.cuh"

namespace adacomp_impl {

bool fast_tile_pass_d(const PassArgs *args, unsigned grid, cudaStream_t st)
{
    if (!args)
        return fast_forms_allow<40, unsigned short>() && fast_forms_allow<0, unsigned char>() && fast_forms_allow<0, unsigned short>();
    switch (args->geo.L_T) {
    case 1000u: fast_forms_launch<40, unsigned short>(*args, grid, st); return true;
    default:
        // every other bin length of the pipelined kernel: its any-bin form (16-bit gradients only where a tile of
        // them is a multiple of 16 bytes, which the caller has checked)
        if (!any_fast_L_T(args->geo.L_T)) return false;
        if (args->geo.L_T <= 64u) fast_forms_launch<0, unsigned char>(*args, grid, st);
        else fast_forms_launch<0, unsigned short>(*args, grid, st);
        return true;
    }
}

ADACOMP_STATUS_HOOKS(pack_fast_d)

}  // namespace adacomp_impl
