// Pipelined tile pass, bin lengths 125, 200 (see pack_tile.cuh: tile_pass_fast).
#include "pack_fast.cuh"

namespace adacomp_impl {

bool fast_tile_pass_b(const PassArgs *args, unsigned grid, cudaStream_t st)
{
    if (!args)
        return fast_forms_allow<5, unsigned short>() && fast_forms_allow<8, unsigned short>();
    switch (args->geo.L_T) {
    case 125u: fast_forms_launch<5, unsigned short>(*args, grid, st); return true;
    case 200u: fast_forms_launch<8, unsigned short>(*args, grid, st); return true;
    default: return false;
    }
}

ADACOMP_STATUS_HOOKS(pack_fast_b)

}  // namespace adacomp_impl
