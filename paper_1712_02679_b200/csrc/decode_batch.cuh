// Batched decode-sum: the layer table of one launch.
#pragma once

#include "decode_words.cuh"

namespace adacomp_impl {

// ---------------------------------------------------------------------------------
// Batched decode-sum: many small layers in one launch.  The layer table (shapes, output and
// stream pointers) travels in the kernel parameters; every CTA builds the same tile index over
// all layers in shared memory and takes (layer, tile) items from it.  Layers of
// 42 <= L_T <= 1000 qualify (tiles of at most 4096 elements and 2..96 bins).
// ---------------------------------------------------------------------------------

constexpr int kDecBatchLayers = 192;
constexpr int kDecBatchPtrs = 2900;

struct DecodeBatchArgs {
    u32 n_layers, k;
    u64 n[kDecBatchLayers];
    u32 L_T[kDecBatchLayers];
    float *dst[kDecBatchLayers];                     // the layer's output; with `sgd` its weights
    float *aux[kDecBatchLayers];                     // with `opt`: its momentum (Adam: first moments)
    float *aux2[kDecBatchLayers];                    // Adam: its second moments
    float lr, mu, beta2, eps;
    u32 opt;                                         // 1 SGD, 2 Adam: the optimizer step takes the place of the store (see Epilogue)
    const unsigned char *stream[kDecBatchPtrs];      // [layer * k + learner]
};


// The batched warp decoder's ring of slots (dynamic shared memory).  Deeper rings for more learners were
// measured: they cost a CTA per SM and the decode of a list is bound by the warps' fixed work per learner and
// tile, so more warps beat more tiles in flight (8 learners: 0.20 ms with this ring, 0.21 ms with twice it).
constexpr u32 kBatchRingBytes = 19200u;

}  // namespace adacomp_impl
