// The pipelined tile pass's instances are spread over pack_fast_a.cu .. pack_fast_d.cu (a few bin lengths
// each) so that they compile side by side; this is what those files share.
#pragma once

#include "internal.h"

namespace adacomp_impl {

// the forms of the kernel for one bin length: eager / lazy-scale, each for the three gradient formats
template <int SPB, typename Word, bool LAZY>
inline bool fast_formats_allow()
{
    const cudaFuncAttribute at = cudaFuncAttributeMaxDynamicSharedMemorySize;
    const int bytes = (int)FastSmem::kBytes;
    return cudaFuncSetAttribute(tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_F32>, at, bytes) == cudaSuccess &&
           cudaFuncSetAttribute(tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_BF16>, at, bytes) == cudaSuccess &&
           cudaFuncSetAttribute(tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_F16>, at, bytes) == cudaSuccess;
}
template <int SPB, typename Word>
inline bool fast_forms_allow() { return fast_formats_allow<SPB, Word, false>() && fast_formats_allow<SPB, Word, true>(); }

template <int SPB, typename Word, bool LAZY>
inline void fast_formats_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    if (a.grad_type == ADACOMP_GRAD_BF16) tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_BF16><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
    else if (a.grad_type == ADACOMP_GRAD_F16) tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_F16><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
    else tile_pass_fast<SPB, Word, LAZY, ADACOMP_GRAD_F32><<<grid, kFastThreads, FastSmem::kBytes, st>>>(a);
}
template <int SPB, typename Word>
inline void fast_forms_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    if (a.lazy_state) fast_formats_launch<SPB, Word, true>(a, grid, st);
    else fast_formats_launch<SPB, Word, false>(a, grid, st);
}

}  // namespace adacomp_impl
