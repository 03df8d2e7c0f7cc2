// The pipelined tile pass's instances are spread over pack_fast_a.cu .. pack_fast_d.cu (a few bin lengths
// each) so that they compile side by side; this is what those files share.
#pragma once

#include "internal.h"

namespace adacomp_impl {

// eager / lazy-scale / bfloat16-gradient forms of the kernel for one bin length
template <int SPB, typename Word>
inline bool fast_forms_allow()
{
    const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
    const int bytes = (int)FastSmem::kBytes;
    return cudaFuncSetAttribute(tile_pass_fast<SPB, Word, false, false>, at, bytes) == cudaSuccess &&
           cudaFuncSetAttribute(tile_pass_fast<SPB, Word, true, false>, at, bytes) == cudaSuccess &&
           cudaFuncSetAttribute(tile_pass_fast<SPB, Word, false, true>, at, bytes) == cudaSuccess;
}
template <int SPB, typename Word>
inline void fast_forms_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    if (a.lazy_state) tile_pass_fast<SPB, Word, true, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
    else if (a.grad_bf16) tile_pass_fast<SPB, Word, false, true><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
    else tile_pass_fast<SPB, Word, false, false><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
}

}  // namespace adacomp_impl
