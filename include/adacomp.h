/*
 * adacomp.h - C ABI of libadacomp: AdaComp residual gradient compression on one
 * NVIDIA B200 (sm_100a).
 *
 * The library implements the two per-layer functions of the AdaComp paper
 * (Chen et al., "AdaComp: Adaptive Residual Gradient Compression for
 * Data-Parallel Distributed Training"): pack() of Algorithm 2 and the
 * unpack()-then-sum half of Algorithm 1.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device pointers valid on the current device;
 *     "host" pointers are ordinary process memory.  `stream` is a cudaStream_t
 *     passed as void* (NULL = the legacy default stream).
 *   - The caller owns every buffer.  The library allocates no memory and keeps
 *     no per-call state; all work is enqueued on `stream` and the call returns
 *     without synchronising (adacomp_device_status is the one exception).
 *   - grad, residue, dst and packed buffers must be 16-byte aligned.
 *   - Return value: ADACOMP_OK (0) or a negative ADACOMP_ERR_* code.  When an
 *     error code is returned nothing has been enqueued.  Conditions only the
 *     GPU can see set sticky bits (ADACOMP_DEV_*) read by adacomp_device_status;
 *     a kernel that meets one skips the affected work and finishes normally.
 *   - Arithmetic is IEEE binary32, round-to-nearest-even, denormals kept, no
 *     fused multiply-add.  Results are deterministic: the same inputs give the
 *     same bytes, whatever the launch geometry.
 *
 * Packed stream (little-endian; section offsets are a pure function of n, L_T)
 *   header, 64 bytes:
 *      0 u32 magic "ADC1" (0x31434441)    4 u16 version = 1
 *      6 u8  w = bytes per word (1 if L_T <= 64, else 2)
 *      7 u8  flags (bit 0: literal Algorithm-2 selection)
 *      8 u32 L_T                         12 u32 tile_bins
 *     16 u64 n                           24 u64 n_bins = ceil(n / L_T)
 *     32 u64 n_tiles = ceil(n_bins / tile_bins)
 *     40 u64 n_sel (elements sent)       48 f32 scale      52 u32 0
 *     56 u64 bytes_used (header + sections, the bytes a receiver needs)
 *   tile_off  u64[n_tiles + 1] at byte 64: index of each tile's first word
 *             (exclusive scan of the per-tile counts; last entry = n_sel);
 *             tile_bins = 4 * floor(1000 / L_T) for L_T <= 1000, else 1
 *   bin_cnt   n_bins entries of w bytes, 16-byte aligned: words sent per bin
 *   payload   n_sel words of w bytes, 16-byte aligned, zero padded to 16 bytes:
 *             word = (index_in_bin << 2) | code, code 01 = +scale, 11 = -scale,
 *             00 = no-op, 10 = reserved; bins in order, indices ascending.
 *   The word widths and the 2-bit ternary value follow the paper's Section
 *   "Experiment Results" (8-bit words below L_T = 64, 16-bit words up to 16K).
 *   Beyond bytes_used the buffer holds scratch the compressor needs.
 */
#ifndef ADACOMP_H
#define ADACOMP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ADACOMP_VERSION 1
#define ADACOMP_MAX_L_T 16384u
#define ADACOMP_MAX_STREAMS 64u

/* host-detected errors */
#define ADACOMP_OK 0
#define ADACOMP_ERR_NULL (-1)      /* a required pointer is NULL */
#define ADACOMP_ERR_L_T (-2)       /* L_T == 0 or L_T > ADACOMP_MAX_L_T */
#define ADACOMP_ERR_ALIGN (-3)     /* a buffer is not 16-byte aligned */
#define ADACOMP_ERR_STREAMS (-4)   /* k_streams == 0 or > ADACOMP_MAX_STREAMS */
#define ADACOMP_ERR_SIZE (-5)      /* n too large (n_bins must stay below 2^31) */
#define ADACOMP_ERR_FLAGS (-6)     /* unknown flag bits */
#define ADACOMP_ERR_CUDA (-7)      /* a CUDA runtime call failed */
#define ADACOMP_ERR_UNSUPPORTED (-9) /* lazy mode: an L_T it does not take (see adacomp_compress_lazy), or flags given */
#define ADACOMP_ERR_STATIC_SCRATCH (-8) /* adacomp_compress_static: tensor beyond the built-in scratch */

/* size of the scratch array built into the library for adacomp_compress_static */
#define ADACOMP_STATIC_SCRATCH_BYTES (8u << 20)

/* device-detected conditions (sticky bits) */
#define ADACOMP_DEV_NONFINITE 1u        /* a bin maximum was inf or NaN */
#define ADACOMP_DEV_HEADER_MISMATCH 2u  /* streams disagree on n / L_T / w, or bad magic */
#define ADACOMP_DEV_RESERVED_CODE 4u    /* ternary code 10 met while decoding */
#define ADACOMP_DEV_TIMEOUT 8u          /* a bounded device-side wait gave up */
#define ADACOMP_DEV_BAD_STREAM 16u      /* a word points outside its bin / tensor */

/* flags of adacomp_compress_ex */
#define ADACOMP_FLAG_LITERAL 1u       /* Algorithm 2 as printed: |H| >= g_max only */
#define ADACOMP_FLAG_GENERIC_PATH 256u /* use the any-L_T kernel even where a specialised one exists */
#define ADACOMP_FLAG_STREAMING 512u    /* use the streaming kernels even for a layer small enough for the one-kernel form */

/* gradient formats (adacomp_options.grad_type): values narrower than binary32 are widened exactly as they are read */
#define ADACOMP_GRAD_F32 0u
#define ADACOMP_GRAD_BF16 1u
#define ADACOMP_GRAD_F16 2u

/* quantisers (adacomp_options.quantiser): what the one value per layer, sent with the words, is */
#define ADACOMP_QUANT_BIN_MAX_MEAN 0u  /* the paper's (Section 2.5): the average of the bin maxima over all bins */
#define ADACOMP_QUANT_SENT_MEAN 1u     /* the average |G| of the elements that are sent (Section 2.5 leaves the function open) */

/* Library ABI version (ADACOMP_VERSION).  Host only, no CUDA call. */
int adacomp_version(void);

/* Static, human-readable text for an ADACOMP_ERR_* code.  Host only. */
const char *adacomp_strerror(int code);

/*
 * Bytes the caller must allocate for `packed_out` of a layer of n elements:
 * header + directory + bin counts + worst-case payload (every element sent) +
 * the compressor's scratch.  Returns 0 for an invalid L_T.  Host only.
 */
size_t adacomp_packed_capacity(uint64_t n, uint32_t L_T);

/*
 * pack() - Algorithm 2 ("Details of pack()") with the scale of Section 2.5.
 *   grad       device, const float[n]: dW of this step.
 *   residue    device, float[n], in/out: the learner's residual gradient.
 *              On return of the stream it holds G - Gq where sent, G elsewhere.
 *   n, L_T     element count (0 is a valid no-op that writes only a header)
 *              and bin length, 1 <= L_T <= 16384.
 *   packed_out device, adacomp_packed_capacity(n, L_T) bytes; receives the stream.
 *   count_out  device, uint64_t[2]: {n_sel, bytes_used}.
 * Computes G = residue + dW, H = G + dW, g_max = per-bin max |G|,
 * scale = mean of g_max over all bins (exact sum, rounded once), sends element i
 * of bin b when g_max[b] > 0, G[i] != 0 and (|H[i]| >= g_max[b] or |G[i]| == g_max[b]),
 * quantises it to sign(G) * scale and subtracts that from the residue.
 */
int adacomp_compress(const float *grad, float *residue, uint64_t n, uint32_t L_T,
                     void *packed_out, uint64_t *count_out, void *stream);

/*
 * adacomp_compress for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework that
 * hands out a fixed arena and forbids further allocation, in a latency-critical loop
 * where an allocation would synchronise the device, or in a component that is only ever
 * given its input and output buffers.  adacomp_compress needs scratch behind the stream
 * (roughly one more word per element, see adacomp_packed_capacity); here that scratch is
 * an array of ADACOMP_STATIC_SCRATCH_BYTES (8 MiB) built into the library instead, so
 *   packed_out needs only the stream itself: 64 + 8 * (n_tiles + 1) + w * n_bins +
 *              w * n bytes with each section rounded up to 16 (adacomp_packed_capacity
 *              is always a safe upper bound);
 *   the tensor must be small enough for the array: about 8.3 M elements at L_T <= 64
 *              and 4.1 M above (the scratch holds w bytes per element plus 4 bytes per
 *              tile).  Larger tensors return ADACOMP_ERR_STATIC_SCRATCH and nothing is
 *              enqueued; use adacomp_compress for those.
 * Arguments, results and error codes are otherwise those of adacomp_compress, and the
 * bytes written to packed_out, count_out and residue are identical.
 *
 * The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.
 * The array lives in the library's device image, so every GPU that loads the library
 * holds the 8 MiB until the process exits.  The first call on each device looks up the
 * array's device address (with that device current); make that first call before any
 * stream capture.  Every call on a device shares the one array, and it keeps the previous
 * call's contents: the call clears the part that must start from zero itself, but two
 * calls that overlap on the GPU (different streams, no dependency between them) race on
 * it and corrupt each other's output.  Calls on one stream are safe.  (The address
 * look-up itself needs no lock: host threads that make the first call together all find
 * the same address.)
 */
int adacomp_compress_static(const float *grad, float *residue, uint64_t n, uint32_t L_T,
                            void *packed_out, uint64_t *count_out, void *stream);

/* As adacomp_compress, with ADACOMP_FLAG_* bits.
 * Which kernels run never changes a byte of the result.  A layer of one of the bin lengths 50, 100, 125, 200,
 * 250, 500, 1000 whose 4000-element tiles all fit in the shared memory of the CTAs that are resident together
 * (4 tiles per CTA, 2 CTAs per SM: 4.7 M elements on 148 SMs) is packed by one cooperative kernel that visits
 * the residue once; ADACOMP_FLAG_STREAMING takes the streaming kernels instead (a tile pass, the scale, and a
 * second visit of the sent elements), which larger layers always take. */
int adacomp_compress_ex(const float *grad, float *residue, uint64_t n, uint32_t L_T,
                        void *packed_out, uint64_t *count_out, void *stream, uint32_t flags);

/*
 * adacomp_compress with another multiplier in the paper's self-adjusting selection (Section 2.4:
 * the value compared with the bin maximum is the old residue plus a multiple of the latest
 * gradient; multiples from 1.5 to 3.0 were studied and 2 was chosen).  The test
 * value becomes H = residue + factor * dW, one rounded multiplication and one rounded addition in
 * binary32; everything else (G, bin maxima, scale, forced bin maximum, quantisation, residue,
 * stream layout) is as in adacomp_compress, which keeps Algorithm 2's H = G + dW with two additions
 * (for factor 2 the two can differ in the last place).  factor = 1 makes H = G: only the bin maxima
 * are sent, which is Section 5's local selection without the soft threshold ("LS").
 *   factor   0 < factor <= 1e30, else ADACOMP_ERR_FLAGS.
 * The stream's header carries bit 1 in its flags byte.  Runs at the speed of adacomp_compress.
 */
int adacomp_compress_scaled(const float *grad, float *residue, uint64_t n, uint32_t L_T,
                            void *packed_out, uint64_t *count_out, void *stream, float factor);

/*
 * adacomp_compress for a gradient that arrives in bfloat16 (the paper's setting is training on
 * reduced-precision accelerators, Section 1; it fixes no format).  Each value is widened exactly
 * to binary32 (a bfloat16 is the upper half of a binary32) as it is read, and Algorithm 2 then runs
 * unchanged: the residue, the scale and the stream are what adacomp_compress gives for the widened
 * gradient.  The call reads 2 bytes per element of gradient instead of 4.
 *   grad_bf16   device, n bfloat16 values (uint16 bit patterns), 16-byte aligned; read-only.
 * Other arguments, ownership and errors as for adacomp_compress.
 */
int adacomp_compress_bf16(const void *grad_bf16, float *residue, uint64_t n, uint32_t L_T,
                          void *packed_out, uint64_t *count_out, void *stream);

/*
 * The same for a gradient in IEEE binary16 (half precision): every value, subnormals, infinities and NaNs
 * included, has an exact binary32 counterpart, which is what Algorithm 2 then sees.
 *   grad_f16   device, n binary16 values (uint16 bit patterns), 16-byte aligned; read-only.
 */
int adacomp_compress_f16(const void *grad_f16, float *residue, uint64_t n, uint32_t L_T,
                         void *packed_out, uint64_t *count_out, void *stream);

/*
 * pack() with every option at once: the variants above are this call with one field set.
 *   flags       ADACOMP_FLAG_* bits (adacomp_compress_ex).
 *   grad_type   ADACOMP_GRAD_*: what `grad` points to (adacomp_compress_bf16 / _f16).
 *   factor      0: Algorithm 2's H = G + dW; else H = residue + factor * dW (adacomp_compress_scaled).
 *   quantiser   ADACOMP_QUANT_*: the value Q = sign(G) * scale is made with.  The paper's scale is the average of
 *               the bin maxima over all bins; ADACOMP_QUANT_SENT_MEAN takes the average |G| of the sent elements
 *               instead (an exact sum, rounded once to double, divided by their number, rounded to binary32; 0
 *               when nothing is sent), which makes the squared error of the sent elements smallest.  The
 *               selection, the words and the decoder do not change; the stream's header carries bit 2 in its
 *               flags byte.
 *   lazy_state  NULL, or the layer's lazy-scale state (adacomp_compress_lazy).
 * Combinations: a factor and a 16-bit gradient go with lazy-scale mode wherever that mode exists
 * (L_T 41..1000 and the multiples of 4 up to 4000), except a 16-bit gradient at a bin length whose tiles
 * are an odd multiple of 4 elements (L_T 43, 45, 47, ... : their 16-bit tiles do not start on the 16-byte
 * boundaries that bulk copies need; eager mode takes the any-L_T kernel there, lazy-scale mode returns
 * ADACOMP_ERR_UNSUPPORTED); flags exclude lazy-scale mode.  `opt` NULL means all zero.  Other arguments,
 * results and errors as for adacomp_compress.
 */
typedef struct {
    uint32_t flags;
    uint32_t grad_type;
    float factor;
    uint32_t quantiser;
    void *lazy_state;
} adacomp_options;

int adacomp_compress_opt(const void *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                         uint64_t *count_out, const adacomp_options *opt, void *stream);


/*
 * unpack() of k learners' streams and their sum (Algorithm 1: unpack(), and the
 * summation inside averageGradients()).
 *   packed     HOST array of k device pointers to packed streams of one layer.
 *   k_streams  1 .. ADACOMP_MAX_STREAMS.
 *   dst        device, float[n] (n is read from the first stream's header on the
 *              device); fully overwritten: dst[i] = sum over l = 0..k-1, in that
 *              order and starting from +0.0f, of +-scale_l where learner l sent i.
 * Streams that disagree on n, L_T or word size set ADACOMP_DEV_HEADER_MISMATCH
 * and dst is left untouched.
 */
int adacomp_decompress_accumulate(const void *const *packed, uint32_t k_streams, float *dst,
                                  void *stream);

/*
 * adacomp_decompress_accumulate for a caller that knows the tensor's shape on the host (the plain
 * call reads n and L_T from the first stream's header on the device and must launch a full grid;
 * here the grid is sized to the tensor, which matters for small layers).  Streams whose headers do
 * not carry exactly (n, L_T) set ADACOMP_DEV_HEADER_MISMATCH and dst is left untouched.
 */
int adacomp_decompress_accumulate_ex(const void *const *packed, uint32_t k_streams, float *dst,
                                     uint64_t n, uint32_t L_T, void *stream);

/*
 * unpack(), averageGradients() and updateWeights() of Algorithm 1 ("Computation Steps") in one
 * pass over the layer: the k streams are decoded and summed as adacomp_decompress_accumulate does,
 * and each finished piece of the sum feeds the optimizer step on the spot, so that the dense
 * gradient is never written to memory.  The paper names "SGD with momentum" (momentum 0.9,
 * Section "Discussions") and prints no formula; the step taken is the plain heavy-ball one, every
 * operation rounded to binary32 on its own (no fused multiply-add):
 *     s    = ordered sum of the k decoded streams, from +0.0f
 *     mean = s / k                      (one IEEE division by float(k))
 *     v'   = (mu * v) + mean
 *     w'   = w - (lr * v')
 * for every element of the layer, the ones nobody sent included (mean = +0 there).
 *   packed     HOST array of k device pointers to packed streams of one layer.
 *   weights    device, float[n], read and written in place (w).
 *   momentum   device, float[n], read and written in place (v).
 *   n, L_T     the layer's shape; streams whose headers do not carry exactly (n, L_T) set
 *              ADACOMP_DEV_HEADER_MISMATCH and neither array is touched.
 *   lr, mu     learning rate and momentum coefficient.
 * weights and momentum must be 16-byte aligned, must not overlap each other or the streams, and
 * stay owned by the caller.  Asynchronous on `stream`; errors as for the other entry points.
 */
int adacomp_decompress_average_sgd(const void *const *packed, uint32_t k_streams, float *weights,
                                   float *momentum, uint64_t n, uint32_t L_T, float lr, float mu,
                                   void *stream);

/*
 * adacomp_decompress_average_sgd for a list of layers (a model's parameter list) in one call, as
 * adacomp_decompress_accumulate_multi_ex is to adacomp_decompress_accumulate_ex: small layers of
 * the paper's bin lengths share launches, the others take the single-layer kernels.
 *   packed     HOST array of n_layers * k_streams device pointers, packed[t * k_streams + l] =
 *              learner l's stream of layer t.
 *   weights, momentum   HOST arrays of n_layers device pointers (float[n[t]] each), updated in place.
 *   n, L_T     HOST arrays of n_layers shapes.
 * One learning rate and one momentum coefficient serve every layer of the call.
 */
int adacomp_decompress_average_sgd_multi(const void *const *packed, uint32_t k_streams,
                                         float *const *weights, float *const *momentum,
                                         const uint64_t *n, const uint32_t *L_T, uint32_t n_layers,
                                         float lr, float mu, void *stream);

/*
 * As adacomp_decompress_average_sgd, with an Adam step in place of the SGD step (the paper reports
 * AdaComp with Adam as well, Section "Experiments", and prints no formula).  The step is Kingma and
 * Ba's Algorithm 1 in the order its Section 2 suggests, every operation rounded to binary32 on its
 * own (IEEE division and square root, no fused multiply-add):
 *     mean = s / k
 *     m'   = (beta1 * m) + ((1 - beta1) * mean)
 *     v'   = (beta2 * v) + ((1 - beta2) * (mean * mean))
 *     w'   = w - ((step_size * m') / (sqrt(v') + eps))
 *   weights, m, v   device, float[n] each, read and written in place (v must be >= 0).
 *   step_size       alpha * sqrt(1 - beta2^t) / (1 - beta1^t): the bias correction is the caller's,
 *                   who knows the step count t.
 *   eps             > 0.
 * Everything else as for adacomp_decompress_average_sgd; the _multi form takes a list of layers as
 * adacomp_decompress_average_sgd_multi does.
 */
int adacomp_decompress_average_adam(const void *const *packed, uint32_t k_streams, float *weights,
                                    float *m, float *v, uint64_t n, uint32_t L_T, float step_size,
                                    float beta1, float beta2, float eps, void *stream);
int adacomp_decompress_average_adam_multi(const void *const *packed, uint32_t k_streams,
                                          float *const *weights, float *const *m, float *const *v,
                                          const uint64_t *n, const uint32_t *L_T, uint32_t n_layers,
                                          float step_size, float beta1, float beta2, float eps,
                                          void *stream);

/* adacomp_decompress_accumulate_multi with the layers' shapes (HOST arrays n[n_layers], L_T[n_layers]). */
int adacomp_decompress_accumulate_multi_ex(const void *const *packed, uint32_t k_streams,
                                           float *const *dst, const uint64_t *n, const uint32_t *L_T,
                                           uint32_t n_layers, void *stream);

/*
 * adacomp_compress_ex with four caller-created cudaEvent_t handles (HOST array, as
 * void*) recorded on `stream` around the three kernels of pack(): events[0] before and
 * events[1] after the tile pass, events[2] after the scale/scan kernel, events[3] after
 * the gather / residue fix-up.  For measurement; the results are those of
 * adacomp_compress_ex.  The paper reports no timing of pack() (Section "Experiments").
 */
int adacomp_compress_profile(const float *grad, float *residue, uint64_t n, uint32_t L_T,
                             void *packed_out, uint64_t *count_out, void *stream, uint32_t flags,
                             void *const *events, void *lazy_state /* NULL: as adacomp_compress_ex */);

/*
 * Lazy-scale pack(): the same stream, bit for bit, in one pass over the residue.
 *
 * In Algorithm 2 the residue of a sent element is G - Gq, and Gq = sign(G) * scale needs the
 * layer-wide scale (Section 2.5), known only after every bin has been seen.  adacomp_compress
 * therefore revisits the sent elements once the scale exists.  The lazy form does not: it leaves
 * G in `residue`, records which elements were sent (one bit each) and the scale in `state`, and the
 * NEXT adacomp_compress_lazy applies "- sign(G) * scale" to those elements as it loads them - the
 * same single binary32 subtraction, so every later stream, scale and residue is identical.
 *
 *   state    device, adacomp_lazy_state_bytes(n, L_T) bytes, 16-byte aligned, set up once per
 *            tensor by adacomp_lazy_state_init and then passed to every call for that tensor.
 *   residue  between calls it is NOT the paper's residue: run adacomp_residue_flush before
 *            reading it (checkpointing), before handing it to adacomp_compress, or before
 *            changing L_T.  After a flush it is exactly what adacomp_compress would have left.
 * L_T from 41 to 1000, and the multiples of 4 from 1004 to 4000, are supported (the paper's two
 * settings, 50 and 500, among them: the bin lengths the pipelined tile pass takes): others return
 * ADACOMP_ERR_UNSUPPORTED (adacomp_lazy_state_bytes returns 0).  A state that does not belong to
 * (n, L_T) sets ADACOMP_DEV_HEADER_MISMATCH and nothing is written.
 */
size_t adacomp_lazy_state_bytes(uint64_t n, uint32_t L_T);
int adacomp_lazy_state_init(void *state, uint64_t n, uint32_t L_T, void *stream);
int adacomp_compress_lazy(const float *grad, float *residue, void *state, uint64_t n, uint32_t L_T,
                          void *packed_out, uint64_t *count_out, void *stream);
/* Applies the pending "- sign(G) * scale" to the elements the last lazy call sent; clears the marks. */
int adacomp_residue_flush(float *residue, void *state, uint64_t n, uint32_t L_T, void *stream);

/*
 * pack() for a gradient that lives in HOST memory (Algorithm 1: serializeGrad() ->
 * pack() -> exchange()).  Copies grad_host[n] (pinned memory advised) to the device
 * staging buffer grad_stage[n], runs adacomp_compress on it, then copies count_dev to
 * count_host[2] and the first bytes_used bytes of packed_dev to packed_host.
 * UNLIKE the other calls this one synchronises `stream` before it returns.
 * packed_host_cap smaller than bytes_used returns ADACOMP_ERR_SIZE (residue is then
 * already updated).  residue, packed_dev, count_dev: as in adacomp_compress.
 */
int adacomp_compress_host(const float *grad_host, float *grad_stage, float *residue, uint64_t n,
                          uint32_t L_T, void *packed_dev, uint64_t *count_dev, void *packed_host,
                          uint64_t packed_host_cap, uint64_t *count_host, void *stream);

/*
 * unpack()-and-sum for streams received into HOST memory (Algorithm 1: exchange() ->
 * unpack() -> averageGradients()).  Copies packed_host[l][0 .. packed_bytes[l]) to the
 * device buffers packed_stage[l] (all three are HOST arrays of k entries), runs
 * adacomp_decompress_accumulate into dst_dev[n] and copies it to dst_host[n].
 * Synchronises `stream` before it returns.
 */
int adacomp_decompress_accumulate_host(const void *const *packed_host, const uint64_t *packed_bytes,
                                       void *const *packed_stage, uint32_t k_streams, float *dst_dev,
                                       float *dst_host, uint64_t n, void *stream);

/* One tensor of a multi-tensor call; every tensor is its own layer (own bins, own scale). */
typedef struct {
    const float *grad;
    float *residue;
    uint64_t n;
    uint32_t L_T;
    uint32_t flags;
    void *packed_out;
    uint64_t *count_out;
} adacomp_layer_desc;

/*
 * pack() of every layer in `layers` (HOST array of n_layers descriptors) on one stream.  Every layer gets what
 * adacomp_compress would give it, bit for bit; the layers are independent, and the order in which the kernels
 * take them is not the list's.  Layers share launches: a small list (bin lengths 50 and 500, at most two
 * 4000-element tiles per resident CTA in all) is packed by two launches, lists of layers with bin lengths 42..1000
 * and fewer than 2^25 elements each by four launches per batch of up to 176 layers, other layers one by one.
 * The descriptors are read during the call only.
 */
int adacomp_compress_multi(const adacomp_layer_desc *layers, uint32_t n_layers, void *stream);

/*
 * adacomp_compress_multi in lazy-scale mode (see adacomp_compress_lazy): states[t] (HOST array of device
 * pointers) is layer t's state, adacomp_lazy_state_bytes(n, L_T) bytes, set up once by
 * adacomp_lazy_state_init; every layer's residue holds G between calls until adacomp_residue_flush.
 * Streams, scales and (flushed) residues are those of adacomp_compress_multi, bit for bit.
 * Every layer needs flags 0 and a bin length the lazy mode takes, else ADACOMP_ERR_UNSUPPORTED and
 * nothing is launched.  A state that is not its layer's sets ADACOMP_DEV_HEADER_MISMATCH; that
 * layer is left untouched and its stream is empty.
 */
int adacomp_compress_multi_lazy(const adacomp_layer_desc *layers, void *const *states, uint32_t n_layers,
                                void *stream);

/*
 * adacomp_compress_multi with options per layer: opts (HOST array of n_layers adacomp_options, or NULL for
 * none) gives layer t its gradient format (layers[t].grad then points to values of that format), the factor of
 * its selection test and, when lazy_state is set, lazy-scale mode with that state.  opts[t].flags must be 0:
 * a layer's flags are those of its descriptor.  Layers share launches as in adacomp_compress_multi; a list
 * in which only some layers have a lazy-scale state is packed layer by layer.  Results are those of
 * adacomp_compress_opt layer by layer, bit for bit; every layer is checked before anything is launched.
 */
int adacomp_compress_multi_opt(const adacomp_layer_desc *layers, const adacomp_options *opts, uint32_t n_layers,
                               void *stream);


/*
 * unpack()-and-sum of every layer: packed[t * k_streams + l] (HOST array) is
 * learner l's stream of layer t, dst[t] (HOST array of device pointers) its output.
 */
int adacomp_decompress_accumulate_multi(const void *const *packed, uint32_t k_streams,
                                        float *const *dst, uint32_t n_layers, void *stream);

/*
 * Makes `device` the calling host thread's current CUDA device for this library.  Every entry
 * point works on the calling thread's current device; a process that selects its GPU through
 * another copy of the CUDA runtime (PyTorch's, say) calls this once per thread with the same
 * ordinal so that both agree.  Not needed in single-GPU processes.
 */
int adacomp_set_device(int device);

/*
 * Synchronises `stream`, then copies the current device's sticky ADACOMP_DEV_* bits to
 * *host_out.  The bits stay set until adacomp_device_status_reset.
 */
int adacomp_device_status(uint32_t *host_out, void *stream);

/*
 * Stream version 2, for the wire.  The paper's rate figures (Section "Experiment Results": 8 or 16 bits per sent
 * element, 40x at L_T = 50 and 200x at L_T = 500) count the words alone; the streams above also carry a count per bin
 * so that a decoder can find a word's bin (1 or 2 bytes per L_T elements: 29.3x on the wire against 34.9x by the
 * paper's accounting at L_T = 50).  Version 2 tells the bins apart with one of the word's own spare bits instead:
 *   word = (index_in_bin << 2) | (first_of_bin << 1) | negative
 * and a bin that sends nothing is one marker word (first_of_bin set, index L_T), so every bin owns exactly one
 * flagged word.  Layout: the 64-byte header (version 2; bytes 52..55: bins that send nothing), the tile directory
 * (u64 offsets in version-2 words), the words, zero-padded to 16 bytes; no count section.  Words are 8 bits wide for
 * L_T <= 63 and 16 bits up to 16383 (the marker's index must fit); L_T = 16384 has no version-2 form.
 * The decoders read version 1; these two calls re-encode a stream either way (three small kernels each), so that
 * exchange() can put version 2 on the wire:
 *   adacomp_stream_to_v2    packed: device, a version-1 stream of shape (n, L_T) as adacomp_compress* leaves it;
 *                           out_v2: device, out_capacity >= adacomp_v2_capacity(n, L_T) bytes, 16-byte aligned;
 *                           count_out: device, uint64_t[2] {words incl. markers, bytes_used} (may be NULL).
 *   adacomp_stream_from_v2  in_v2: device, a version-2 stream; packed_out: device, out_capacity >= the stream part
 *                           of adacomp_packed_capacity(n, L_T) (that value always suffices); receives the
 *                           version-1 stream, byte for byte what the sender converted.
 * A header that is not of the given shape and version sets ADACOMP_DEV_HEADER_MISMATCH and nothing else is written;
 * a stream that contradicts itself sets ADACOMP_DEV_BAD_STREAM and every write stays inside the output.
 * Host errors as for adacomp_compress (ADACOMP_ERR_SIZE: out_capacity too small; ADACOMP_ERR_L_T also for 16384).
 */
size_t adacomp_v2_capacity(uint64_t n, uint32_t L_T);
int adacomp_stream_to_v2(const void *packed, void *out_v2, uint64_t out_capacity, uint64_t *count_out, uint64_t n,
                         uint32_t L_T, void *stream);
int adacomp_stream_from_v2(const void *in_v2, void *packed_out, uint64_t out_capacity, uint64_t n, uint32_t L_T,
                           void *stream);

/*
 * Testing aid for the bounded device-side waits (every wait of a kernel on a copy in flight gives up after a
 * limit, raises ADACOMP_DEV_TIMEOUT, lets the copies it did start land and returns; no kernel spins without a
 * limit).  This call lets a test see that path run without anything being wrong with the device:
 *   wait_cycles            the limit, in GPU clock cycles, of the waits in adacomp_compress* (single layer,
 *                          pipelined tile pass) and in adacomp_decompress_* (single tensor, L_T above 40);
 *                          0 restores the default of about two seconds.
 *   withhold_pack_tile     CTA 0 of the next tile passes announces the copies of its tile number i (i >= 1,
 *                          counted over the CTA's own tiles) and never starts them; 0: none.
 *   withhold_decode_item   the same for work item i of CTA 0 of the next decodes; 0: none.
 * A kernel that meets a withheld copy times out: the tiles / items its CTA 0 had not finished are reported as
 * empty (pack) or left unwritten (decode), every other CTA's work is complete, and the kernels behind stay
 * inside their buffers.  Host only; the settings are process-wide and stay until the next call.  Not meant
 * for production code.  (The paper has no counterpart.)
 */
int adacomp_debug_waits(uint64_t wait_cycles, uint32_t withhold_pack_tile, uint32_t withhold_decode_item);

/* Enqueues a clear of the sticky bits on `stream`. */
int adacomp_device_status_reset(void *stream);

#ifdef __cplusplus
}
#endif
#endif /* ADACOMP_H */
