// Pipelined tile pass, bin lengths 250, 500 (see pack_tile.cuh: tile_pass_fast).
#include "pack_fast.cuh"

namespace adacomp_impl {

bool fast_tile_pass_c(const PassArgs *args, unsigned grid, cudaStream_t st)
{
    if (!args)
        return fast_forms_allow<10, unsigned short>() && fast_forms_allow<20, unsigned short>();
    switch (args->geo.L_T) {
    case 250u: fast_forms_launch<10, unsigned short>(*args, grid, st); return true;
    case 500u: fast_forms_launch<20, unsigned short>(*args, grid, st); return true;
    default: return false;
    }
}

ADACOMP_STATUS_HOOKS(pack_fast_c)

}  // namespace adacomp_impl
