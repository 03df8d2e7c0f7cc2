// Pipelined tile pass, bin lengths 50, 100 (see pack_tile.cuh: tile_pass_fast).
#include "pack_fast.cuh"

namespace adacomp_impl {

bool fast_tile_pass_a(const PassArgs *args, unsigned grid, cudaStream_t st)
{
    if (!args)
        return fast_forms_allow<2, unsigned char>() && fast_forms_allow<4, unsigned short>();
    switch (args->geo.L_T) {
    case 50u: fast_forms_launch<2, unsigned char>(*args, grid, st); return true;
    case 100u: fast_forms_launch<4, unsigned short>(*args, grid, st); return true;
    default: return false;
    }
}

ADACOMP_STATUS_HOOKS(pack_fast_a)

}  // namespace adacomp_impl
