// The pipelined tile pass's instances are spread over pack_fast_a.cu .. pack_fast_d.cu (a few bin lengths
// each) so that they compile side by side; this is what those files share.
#pragma once

#include "internal.h"

namespace adacomp_impl {

// the forms of the kernel for one bin length: eager / lazy-scale, each for the three gradient formats
// 16-bit gradients in the specialised forms: three CTAs per SM (two stages with the half-size gradient tile packed
// against the residue).  At two CTAs per SM the kernel is latency- rather than memory-bound, so fewer bytes alone
// did not make it faster; with a third CTA the lazy-scale call runs 12-13 % faster than with fp32 gradients.
template <int SPB, int GT>
constexpr int fast_ctas() { return SPB != 0 && GT != 0 ? 3 : 2; }
template <int SPB, int GT>
constexpr unsigned fast_smem() { return fast_ctas<SPB, GT>() == 3 ? FastSmem3::kBytes : FastSmem::kBytes; }

template <int SPB, typename Word, bool LAZY, int GT>
inline bool fast_format_allow()
{
    return cudaFuncSetAttribute(tile_pass_fast<SPB, Word, LAZY, GT, fast_ctas<SPB, GT>()>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)fast_smem<SPB, GT>()) == cudaSuccess;
}
template <int SPB, typename Word, bool LAZY>
inline bool fast_formats_allow()
{
    return fast_format_allow<SPB, Word, LAZY, ADACOMP_GRAD_F32>() && fast_format_allow<SPB, Word, LAZY, ADACOMP_GRAD_BF16>() &&
           fast_format_allow<SPB, Word, LAZY, ADACOMP_GRAD_F16>();
}
template <int SPB, typename Word>
inline bool fast_forms_allow() { return fast_formats_allow<SPB, Word, false>() && fast_formats_allow<SPB, Word, true>(); }

// `grid`: two CTAs per SM, or the number of tiles if that is less
template <int SPB, typename Word, bool LAZY, int GT>
inline void fast_format_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    constexpr int ctas = fast_ctas<SPB, GT>();
    u64 g = grid;
    if (ctas == 3) {
        g = g / 2 * 3 > g ? g / 2 * 3 : g;
        g = a.geo.n_tiles < g ? a.geo.n_tiles : g;
    }
    tile_pass_fast<SPB, Word, LAZY, GT, ctas><<<(unsigned)g, kFastThreads, fast_smem<SPB, GT>(), st>>>(a);
}
template <int SPB, typename Word, bool LAZY>
inline void fast_formats_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    if (a.grad_type == ADACOMP_GRAD_BF16) fast_format_launch<SPB, Word, LAZY, ADACOMP_GRAD_BF16>(a, grid, st);
    else if (a.grad_type == ADACOMP_GRAD_F16) fast_format_launch<SPB, Word, LAZY, ADACOMP_GRAD_F16>(a, grid, st);
    else fast_format_launch<SPB, Word, LAZY, ADACOMP_GRAD_F32>(a, grid, st);
}
template <int SPB, typename Word>
inline void fast_forms_launch(const PassArgs &a, unsigned grid, cudaStream_t st)
{
    if (a.lazy_state) fast_formats_launch<SPB, Word, true>(a, grid, st);
    else fast_formats_launch<SPB, Word, false>(a, grid, st);
}

}  // namespace adacomp_impl
