// Batched pack(): the layer table of one launch set.
#pragma once

#include "pack_tile.cuh"

namespace adacomp_impl {

// ---------------------------------------------------------------------------------
// Batched pack(): many small layers in four launches instead of four launches per layer.
// The layer table travels in the kernel parameters; a global tile index runs over the tiles
// of all layers, and every CTA (tile pass) or warp (gather) looks its tile's layer up.
// Layers of 42 <= L_T <= 1000 (tiles of at most 4000 elements and 96 bins) qualify.
// ---------------------------------------------------------------------------------

constexpr int kBatchMax = 176;                       // layers per batched launch (the table is 32392 of the 32764 bytes of kernel parameters)
constexpr u64 kBatchLayerMaxElems = 1ull << 22;      // decode: larger layers take the single-layer kernels
// pack(): layers up to this size share a batch's launches when the pipelined batch tile pass is there (a
// layer alone ramps its pipeline up and down over a few tiles per CTA and pays four launches and a finalize
// of its own: below 2^24 elements it runs at under half the speed it has inside a batch)
constexpr u64 kPackBatchMaxElems = 1ull << 25;
constexpr u32 kBatchSmemBytes = 4000 * 10 + 4 * kSmallBins + 4 * (kSmallBins + 1) + 16;

struct BatchLayer {
    const float *grad;
    float *residue;
    unsigned char *packed;
    u64 *count_out;
    Geometry geo;
    u32 tile_first;                                  // global index of the layer's first tile
    u32 grad_type;                                   // ADACOMP_GRAD_*: what `grad` points to
    unsigned char *lazy;                             // lazy-scale mode: the layer's state (else null)
    float factor;                                    // 0: H = G + dW (Algorithm 2); else H = residue + factor * dW
    u32 inv_L_T;                                     // ceil(2^32 / L_T): a thread's first bin without a division
};

// The table comes in two sizes: kernel parameters are copied at every launch, and a launch with the
// full 27 KB table costs several microseconds more than one with the small table.
constexpr int kBatchSmall = 16;

template <int N>
struct BatchArgsT {
    u32 n_layers, total_tiles;
    BatchLayer layer[N];
};
typedef BatchArgsT<kBatchMax> BatchArgs;


}  // namespace adacomp_impl
