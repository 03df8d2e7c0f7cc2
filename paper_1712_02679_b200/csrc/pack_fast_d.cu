// Pipelined tile pass, bin lengths 1000 and the any-bin form (see pack_tile.cuh: tile_pass_fast).
#include "pack_fast.cuh"

namespace adacomp_impl {

bool fast_tile_pass_d(const PassArgs *args, unsigned grid, cudaStream_t st)
{
    if (!args)
        return fast_forms_allow<40, unsigned short>() &&
               cudaFuncSetAttribute(tile_pass_fast<0, unsigned char, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FastSmem::kBytes) == cudaSuccess &&
               cudaFuncSetAttribute(tile_pass_fast<0, unsigned short, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FastSmem::kBytes) == cudaSuccess &&
               cudaFuncSetAttribute(tile_pass_fast<0, unsigned char, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FastSmem::kBytes) == cudaSuccess &&
               cudaFuncSetAttribute(tile_pass_fast<0, unsigned short, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FastSmem::kBytes) == cudaSuccess;
    switch (args->geo.L_T) {
    case 1000u: fast_forms_launch<40, unsigned short>(*args, grid, st); return true;
    default:
        // every other bin length of the pipelined kernel: its any-bin form (fp32 gradient)
        if (!any_fast_L_T(args->geo.L_T) || args->grad_bf16) return false;
        if (args->geo.L_T <= 64u) {
            if (args->lazy_state) tile_pass_fast<0, unsigned char, true, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(*args);
            else tile_pass_fast<0, unsigned char, false, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(*args);
        } else {
            if (args->lazy_state) tile_pass_fast<0, unsigned short, true, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(*args);
            else tile_pass_fast<0, unsigned short, false, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(*args);
        }
        return true;
    }
}

ADACOMP_STATUS_HOOKS(pack_fast_d)

}  // namespace adacomp_impl
