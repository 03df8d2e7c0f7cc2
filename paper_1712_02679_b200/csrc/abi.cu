// libadacomp's C ABI (include/adacomp.h): argument checks and dispatch to the launchers in the other files,
// this device's record and its sticky status word.
#include "internal.h"

namespace adacomp_impl {


DeviceInfo g_info[64];

DebugWaits g_debug_waits = {kWaitCycles, 0u, 0u};
const DebugWaits &debug_waits() { return g_debug_waits; }

int device_info(DeviceInfo *&out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return ADACOMP_ERR_CUDA;
    DeviceInfo &d = g_info[dev];
    if (d.sms == 0) {
        int sms = 0, optin = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return ADACOMP_ERR_CUDA;
        d.smem_optin = optin;
        init_decode_info(d);
        init_pack_info(d);
        init_pack_batch_info(d);        // (after init_pack_info: it needs fast_ready)
        init_pack_onchip_info(d);
        init_pack_onchip_list_info(d);
        init_decode_batch_info(d);
        d.sms = sms;
    }
    out = &d;
    return ADACOMP_OK;
}

}  // namespace adacomp_impl

using namespace adacomp_impl;

// ---------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------

extern "C" {

int adacomp_version(void) { return ADACOMP_VERSION; }

const char *adacomp_strerror(int code)
{
    switch (code) {
    case ADACOMP_OK: return "ok";
    case ADACOMP_ERR_NULL: return "a required pointer is NULL";
    case ADACOMP_ERR_L_T: return "L_T must be in 1..16384";
    case ADACOMP_ERR_ALIGN: return "a buffer is not 16-byte aligned";
    case ADACOMP_ERR_STREAMS: return "k_streams must be in 1..64";
    case ADACOMP_ERR_SIZE: return "tensor too large for this bin length";
    case ADACOMP_ERR_FLAGS: return "unknown flag bits";
    case ADACOMP_ERR_CUDA: return "a CUDA runtime call failed";
    case ADACOMP_ERR_UNSUPPORTED: return "lazy mode supports L_T = 41..1000 (and multiples of 4 up to 4000) without flags only";
    case ADACOMP_ERR_STATIC_SCRATCH:
        return "tensor needs more scratch than the library's built-in array holds; use adacomp_compress";
    default: return "unknown error code";
    }
}

size_t adacomp_packed_capacity(uint64_t n, uint32_t L_T)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return 0;
    return (size_t)make_geometry(n, L_T).capacity;
}

int adacomp_compress(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                     uint64_t *count_out, void *stream)
{
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0);
}

int adacomp_compress_static(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                            uint64_t *count_out, void *stream)
{
    return compress_static_impl(grad, residue, n, L_T, packed_out, count_out, stream);
}

int adacomp_compress_ex(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                        uint64_t *count_out, void *stream, uint32_t flags)
{
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, flags);
}

int adacomp_decompress_accumulate(const void *const *packed, uint32_t k_streams, float *dst, void *stream)
{
    return decompress_impl(packed, k_streams, dst, stream);
}

int adacomp_decompress_accumulate_ex(const void *const *packed, uint32_t k_streams, float *dst, uint64_t n,
                                     uint32_t L_T, void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    return decompress_impl(packed, k_streams, dst, stream, n, L_T);
}

// Decode-sum of a list of layers whose shapes the caller knows.  `opt` (optional; its pointers unused):
// `dst` then holds the layers' weights, `aux` their momentum (Adam: first moments), `aux2` (Adam) their
// second moments, and every layer gets the optimizer step instead of a store.
int decompress_multi_impl(const void *const *packed, uint32_t k_streams, float *const *dst, float *const *aux,
                          float *const *aux2, const uint64_t *n, const uint32_t *L_T, uint32_t n_layers, void *stream,
                          const Epilogue *opt)
{
    if (opt && n_layers && (!aux || (opt->adam && !aux2))) return ADACOMP_ERR_NULL;
    if (n_layers && (!packed || !dst || !n || !L_T)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    for (uint32_t t = 0; t < n_layers; t++) {
        if (L_T[t] == 0 || L_T[t] > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
        if (!dst[t] || (opt && !aux[t]) || (opt && opt->adam && !aux2[t])) return ADACOMP_ERR_NULL;
        if (misaligned(dst[t]) || (opt && misaligned(aux[t])) || (opt && opt->adam && misaligned(aux2[t])))
            return ADACOMP_ERR_ALIGN;
        for (uint32_t l = 0; l < k_streams; l++) {
            if (!packed[(size_t)t * k_streams + l]) return ADACOMP_ERR_NULL;
            if (misaligned(packed[(size_t)t * k_streams + l])) return ADACOMP_ERR_ALIGN;
        }
    }
    if (n_layers == 0) return ADACOMP_OK;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // small layers of the paper's bin lengths share launches; the rest are decoded one by one
    static thread_local DecodeBatchArgs batch;
    batch.n_layers = 0;
    batch.k = k_streams;
    batch.opt = !opt ? 0u : opt->adam ? 2u : 1u;
    batch.lr = opt ? opt->lr : 0.f;
    batch.mu = opt ? opt->mu : 0.f;
    batch.beta2 = opt ? opt->beta2 : 0.f;
    batch.eps = opt ? opt->eps : 0.f;
    u64 batch_tiles = 0;
    // (the batched warp decoder, and with it layers of up to 2^25 elements for plain decode-sum; with an
    // optimizer step larger layers keep the single-tensor kernels, which stage the optimizer's arrays by bulk copies)
    const int opt_form = !opt ? 0 : opt->adam ? 2 : 1;
    const bool warps_batch = info->dec_batch_warps_per_sm[opt_form] > 0;
    const u64 batch_max_elems = warps_batch && !opt ? kPackBatchMaxElems : kBatchLayerMaxElems;
    auto flush = [&]() -> int {
        if (batch.n_layers == 0) return ADACOMP_OK;
        const int launched = launch_decode_batch(batch, batch_tiles, *info, st);
        batch.n_layers = 0;
        batch_tiles = 0;
        return launched;
    };
    const uint32_t per_batch = (uint32_t)kDecBatchPtrs / k_streams < (uint32_t)kDecBatchLayers
                                   ? (uint32_t)kDecBatchPtrs / k_streams : (uint32_t)kDecBatchLayers;
    for (uint32_t t = 0; t < n_layers; t++) {
        const bool small = info->dec_batch_per_sm > 0 && L_T[t] >= 42u && L_T[t] <= 1000u &&
                           n[t] < batch_max_elems && n_layers > 1;
        if (small) {
            const u32 i = batch.n_layers++;
            batch.n[i] = n[t];
            batch.L_T[i] = L_T[t];
            batch.dst[i] = dst[t];
            batch.aux[i] = opt ? aux[t] : nullptr;
            batch.aux2[i] = opt && opt->adam ? aux2[t] : nullptr;
            for (uint32_t l = 0; l < k_streams; l++)
                batch.stream[(size_t)i * k_streams + l] = static_cast<const unsigned char *>(packed[(size_t)t * k_streams + l]);
            batch_tiles += decode_items(n[t], L_T[t]);
            if (batch.n_layers == per_batch) {
                rc = flush();
                if (rc != ADACOMP_OK) return rc;
            }
        } else if (opt) {
            Epilogue ep = *opt;
            ep.weights = dst[t];
            ep.momentum = aux[t];
            ep.second = opt->adam ? aux2[t] : nullptr;
            rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, nullptr, stream, n[t], L_T[t], &ep);
            if (rc != ADACOMP_OK) return rc;
        } else {
            rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, dst[t], stream, n[t], L_T[t]);
            if (rc != ADACOMP_OK) return rc;
        }
    }
    return flush();
}

int adacomp_decompress_accumulate_multi_ex(const void *const *packed, uint32_t k_streams, float *const *dst,
                                           const uint64_t *n, const uint32_t *L_T, uint32_t n_layers, void *stream)
{
    return decompress_multi_impl(packed, k_streams, dst, nullptr, nullptr, n, L_T, n_layers, stream, nullptr);
}

int adacomp_decompress_average_sgd_multi(const void *const *packed, uint32_t k_streams, float *const *weights,
                                         float *const *momentum, const uint64_t *n, const uint32_t *L_T,
                                         uint32_t n_layers, float lr, float mu, void *stream)
{
    const Epilogue opt = {nullptr, nullptr, nullptr, lr, mu, 0.f, 0.f, 0.f, 0u, 0.f};
    return decompress_multi_impl(packed, k_streams, weights, momentum, nullptr, n, L_T, n_layers, stream, &opt);
}

int adacomp_decompress_average_adam_multi(const void *const *packed, uint32_t k_streams, float *const *weights,
                                          float *const *m, float *const *v, const uint64_t *n, const uint32_t *L_T,
                                          uint32_t n_layers, float step_size, float beta1, float beta2, float eps,
                                          void *stream)
{
    const Epilogue opt = {nullptr, nullptr, nullptr, step_size, beta1, beta2, eps, 0.f, 1u, 0.f};
    return decompress_multi_impl(packed, k_streams, weights, m, v, n, L_T, n_layers, stream, &opt);
}

int adacomp_compress_profile(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                             uint64_t *count_out, void *stream, uint32_t flags, void *const *events,
                             void *lazy_state)
{
    if (!events) return ADACOMP_ERR_NULL;
    for (int i = 0; i < 4; i++)
        if (!events[i]) return ADACOMP_ERR_NULL;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, flags, events, lazy_state);
}

size_t adacomp_lazy_state_bytes(uint64_t n, uint32_t L_T)
{
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return 0;
    return (size_t)lazy_state_bytes(make_geometry(n, L_T));
}

int adacomp_lazy_state_init(void *state, uint64_t n, uint32_t L_T, void *stream)
{
    if (!state) return ADACOMP_ERR_NULL;
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return ADACOMP_ERR_UNSUPPORTED;
    if (misaligned(state)) return ADACOMP_ERR_ALIGN;
    return lazy_state_init(state, n, L_T, stream);
}

int adacomp_compress_lazy(const float *grad, float *residue, void *state, uint64_t n, uint32_t L_T,
                          void *packed_out, uint64_t *count_out, void *stream)
{
    if (!state) return ADACOMP_ERR_NULL;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, state);
}

int adacomp_residue_flush(float *residue, void *state, uint64_t n, uint32_t L_T, void *stream)
{
    if (!state || (n && !residue)) return ADACOMP_ERR_NULL;
    if (!fast_L_T(L_T) && !any_fast_L_T(L_T)) return ADACOMP_ERR_UNSUPPORTED;
    if (misaligned(residue) || misaligned(state)) return ADACOMP_ERR_ALIGN;
    return residue_flush(residue, state, n, L_T, stream);
}

int adacomp_compress_host(const float *grad_host, float *grad_stage, float *residue, uint64_t n, uint32_t L_T,
                          void *packed_dev, uint64_t *count_dev, void *packed_host, uint64_t packed_host_cap,
                          uint64_t *count_host, void *stream)
{
    if (!count_host || !packed_host || (n && (!grad_host || !grad_stage))) return ADACOMP_ERR_NULL;
    // every check pack() makes on the host comes before the first copy: an error code means nothing was enqueued
    if (!packed_dev || !count_dev || (n && !residue)) return ADACOMP_ERR_NULL;
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    if (misaligned(grad_stage) || misaligned(residue) || misaligned(packed_dev) ||
        (reinterpret_cast<uintptr_t>(count_dev) & 7u))
        return ADACOMP_ERR_ALIGN;
    if ((n + L_T - 1) / L_T >= (1ull << 31)) return ADACOMP_ERR_SIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n && cudaMemcpyAsync(grad_stage, grad_host, n * sizeof(float), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    int rc = compress_impl(grad_stage, residue, n, L_T, packed_dev, count_dev, stream, 0);
    if (rc != ADACOMP_OK) return rc;
    if (cudaMemcpyAsync(count_host, count_dev, 2 * sizeof(uint64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    if (count_host[1] > packed_host_cap) return ADACOMP_ERR_SIZE;
    if (cudaMemcpyAsync(packed_host, packed_dev, count_host[1], cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    return ADACOMP_OK;
}

int adacomp_decompress_accumulate_host(const void *const *packed_host, const uint64_t *packed_bytes,
                                       void *const *packed_stage, uint32_t k_streams, float *dst_dev,
                                       float *dst_host, uint64_t n, void *stream)
{
    if (!packed_host || !packed_bytes || !packed_stage || !dst_dev || (n && !dst_host)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (uint32_t l = 0; l < k_streams; l++) {
        if (!packed_host[l] || !packed_stage[l]) return ADACOMP_ERR_NULL;
        if (cudaMemcpyAsync(packed_stage[l], packed_host[l], packed_bytes[l], cudaMemcpyHostToDevice, st) != cudaSuccess)
            return ADACOMP_ERR_CUDA;
    }
    int rc = decompress_impl(packed_stage, k_streams, dst_dev, stream);
    if (rc != ADACOMP_OK) return rc;
    if (n && cudaMemcpyAsync(dst_host, dst_dev, n * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ADACOMP_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

// `states` (optional): lazy-scale mode, states[t] the state of layer t.  `opts` (optional): per layer the gradient
// format and the selection's factor (and, in place of `states`, the lazy-scale state); its flags are not used,
// the layer's own are.
static int compress_multi_impl(const adacomp_layer_desc *layers, void *const *states, uint32_t n_layers, void *stream,
                               const adacomp_options *opts = nullptr)
{
    if (n_layers && !layers) return ADACOMP_ERR_NULL;
    auto state_of = [&](uint32_t t) -> void * { return states ? states[t] : opts ? opts[t].lazy_state : nullptr; };
    auto factor_of = [&](uint32_t t) { return opts ? opts[t].factor : 0.f; };
    auto type_of = [&](uint32_t t) { return opts ? opts[t].grad_type : (uint32_t)ADACOMP_GRAD_F32; };
    auto quant_of = [&](uint32_t t) { return opts ? opts[t].quantiser : (uint32_t)ADACOMP_QUANT_BIN_MAX_MEAN; };
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        if (opts) {
            const adacomp_options &o = opts[t];
            if (o.quantiser > ADACOMP_QUANT_SENT_MEAN || o.flags != 0u || o.grad_type > ADACOMP_GRAD_F16) return ADACOMP_ERR_FLAGS;
            if (o.factor != 0.f && !(o.factor > 0.f && o.factor <= 1e30f)) return ADACOMP_ERR_FLAGS;
            if (o.lazy_state) {
                if (misaligned(o.lazy_state)) return ADACOMP_ERR_ALIGN;
                if (d.flags != 0 || !(fast_L_T(d.L_T) || any_fast_L_T(d.L_T))) return ADACOMP_ERR_UNSUPPORTED;
                if (o.grad_type != ADACOMP_GRAD_F32 && !fast_L_T(d.L_T) && d.L_T >= 1u && d.L_T <= ADACOMP_MAX_L_T &&
                    make_geometry(d.n, d.L_T).tile_elems % 8u != 0)
                    return ADACOMP_ERR_UNSUPPORTED;
            }
        }
        if (!d.packed_out || !d.count_out || (d.n && (!d.grad || !d.residue))) return ADACOMP_ERR_NULL;
        if (d.L_T == 0 || d.L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
        if (d.flags & ~(ADACOMP_FLAG_LITERAL | ADACOMP_FLAG_GENERIC_PATH | ADACOMP_FLAG_STREAMING)) return ADACOMP_ERR_FLAGS;
        if (misaligned(d.grad) || misaligned(d.residue) || misaligned(d.packed_out) ||
            (reinterpret_cast<uintptr_t>(d.count_out) & 7u))
            return ADACOMP_ERR_ALIGN;
        if ((d.n + d.L_T - 1) / d.L_T >= (1ull << 31)) return ADACOMP_ERR_SIZE;
        if (states) {
            if (!states[t]) return ADACOMP_ERR_NULL;
            if (misaligned(states[t])) return ADACOMP_ERR_ALIGN;
            if (d.flags != 0 || !(fast_L_T(d.L_T) || any_fast_L_T(d.L_T))) return ADACOMP_ERR_UNSUPPORTED;
        }
    }
    if (n_layers == 0) return ADACOMP_OK;
    DeviceInfo *info = nullptr;
    int rc = device_info(info);
    if (rc != ADACOMP_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // small layers share four launches per batch; the rest go through the single-layer path
    static thread_local BatchArgs batch;
    batch.n_layers = 0;
    batch.total_tiles = 0;
    // (a batch is eager or lazy-scale as a whole: with per-layer options the layers of either kind go to the
    // single-layer path unless all of them are lazy-scale or none is)
    bool any_lazy = false, all_lazy = n_layers > 0;
    for (uint32_t t = 0; t < n_layers; t++) {
        any_lazy = any_lazy || state_of(t) != nullptr;
        all_lazy = all_lazy && state_of(t) != nullptr;
    }
    const bool batch_lazy = any_lazy && all_lazy, mixed = any_lazy && !all_lazy;
    // (the batch kernels know the paper's quantiser only: a layer with the other one is packed on its own)
    auto batched_at = [&](uint32_t t) {
        return !mixed && quant_of(t) == ADACOMP_QUANT_BIN_MAX_MEAN && info->batch_per_sm > 0 && batchable(layers[t], *info) &&
               (!batch_lazy || info->batch_fast_ready);
    };
    // (a lone layer gains nothing from the batch kernels, and the single-layer path may pack it in one kernel)
    uint32_t to_batch = 0;
    for (uint32_t t = 0; t < n_layers; t++) to_batch += batched_at(t) ? 1u : 0u;
    const bool lone = to_batch == 1;
    for (uint32_t t = 0; t < n_layers; t++) {
        const adacomp_layer_desc &d = layers[t];
        if (batched_at(t) && !lone) continue;
        rc = compress_impl(d.grad, d.residue, d.n, d.L_T, d.packed_out, d.count_out, stream, d.flags, nullptr,
                           state_of(t), factor_of(t), type_of(t), nullptr, quant_of(t));
        if (rc != ADACOMP_OK) return rc;
    }
    if (lone || to_batch == 0) return ADACOMP_OK;
    // A batch whose layers all have the bin length 50, or all 500, runs a tile pass with the tile's shape compiled
    // in (pack_batch.cu).  The layers of such a bin length get batches of their own when they are worth the extra
    // launches (a few thousand tiles: the shorter tile code saves about a microsecond per tile and CTA, a batch
    // costs four launches); layers are independent, so the order in which they are packed is free.
    constexpr u64 kOwnBatchTiles = 3000;     // (of the bin length 50: the form for 500 measured no faster than the mixed one)
    u64 tiles_of[2] = {0, 0};           // [L_T 500, L_T 50]
    uint32_t others = 0;
    for (uint32_t t = 0; t < n_layers; t++) {
        if (!batched_at(t)) continue;
        const u32 lt = layers[t].L_T;
        if (lt == 500u || lt == 50u) tiles_of[lt == 50u] += make_geometry(layers[t].n, lt).n_tiles;
        else others++;
    }
    const bool own[2] = {false, tiles_of[1] >= kOwnBatchTiles && (tiles_of[0] != 0 || others != 0)};
    auto class_of = [&](uint32_t t) { return layers[t].L_T == 500u && own[0] ? 0 : layers[t].L_T == 50u && own[1] ? 1 : 2; };
    for (int cls = 0; cls < 3; cls++) {
        // (more layers than a table holds: batches of equal size, so that none is left with a layer or two)
        uint32_t members = 0;
        for (uint32_t t = 0; t < n_layers; t++) members += batched_at(t) && class_of(t) == cls ? 1u : 0u;
        if (!members) continue;
        const uint32_t n_batches = (members + (uint32_t)kBatchMax - 1) / (uint32_t)kBatchMax;
        const uint32_t per_batch = (members + n_batches - 1) / n_batches;
        for (uint32_t t = 0; t < n_layers; t++) {
            if (!batched_at(t) || class_of(t) != cls) continue;
            const adacomp_layer_desc &d = layers[t];
            BatchLayer &L = batch.layer[batch.n_layers++];
            L.grad = d.grad;
            L.residue = d.residue;
            L.packed = static_cast<unsigned char *>(d.packed_out);
            L.count_out = reinterpret_cast<u64 *>(d.count_out);
            L.geo = make_geometry(d.n, d.L_T);
            L.tile_first = batch.total_tiles;
            L.grad_type = type_of(t);
            L.factor = factor_of(t);
            L.inv_L_T = (u32)(((1ull << 32) + d.L_T - 1) / d.L_T);
            L.lazy = static_cast<unsigned char *>(state_of(t));
            batch.total_tiles += (u32)L.geo.n_tiles;
            if (batch.n_layers == per_batch) {
                rc = launch_batch(batch, *info, st, batch_lazy);
                if (rc != ADACOMP_OK) return rc;
                batch.n_layers = 0;
                batch.total_tiles = 0;
            }
        }
        rc = launch_batch(batch, *info, st, batch_lazy);
        if (rc != ADACOMP_OK) return rc;
        batch.n_layers = 0;
        batch.total_tiles = 0;
    }
    return ADACOMP_OK;
}

int adacomp_compress_multi_opt(const adacomp_layer_desc *layers, const adacomp_options *opts, uint32_t n_layers, void *stream)
{
    return compress_multi_impl(layers, nullptr, n_layers, stream, opts);
}

int adacomp_compress_multi(const adacomp_layer_desc *layers, uint32_t n_layers, void *stream)
{
    return compress_multi_impl(layers, nullptr, n_layers, stream);
}

int adacomp_compress_multi_lazy(const adacomp_layer_desc *layers, void *const *states, uint32_t n_layers, void *stream)
{
    if (n_layers && !states) return ADACOMP_ERR_NULL;
    return compress_multi_impl(layers, states, n_layers, stream);
}

int adacomp_decompress_accumulate_multi(const void *const *packed, uint32_t k_streams, float *const *dst,
                                        uint32_t n_layers, void *stream)
{
    if (n_layers && (!packed || !dst)) return ADACOMP_ERR_NULL;
    if (k_streams == 0 || k_streams > ADACOMP_MAX_STREAMS) return ADACOMP_ERR_STREAMS;
    for (uint32_t t = 0; t < n_layers; t++) {
        int rc = decompress_impl(packed + (size_t)t * k_streams, k_streams, dst[t], stream);
        if (rc != ADACOMP_OK) return rc;
    }
    return ADACOMP_OK;
}

int adacomp_compress_bf16(const void *grad_bf16, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                          uint64_t *count_out, void *stream)
{
    return compress_impl(static_cast<const float *>(grad_bf16), residue, n, L_T, packed_out, count_out, stream, 0, nullptr,
                         nullptr, 0.f, ADACOMP_GRAD_BF16);
}

int adacomp_compress_f16(const void *grad_f16, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                         uint64_t *count_out, void *stream)
{
    return compress_impl(static_cast<const float *>(grad_f16), residue, n, L_T, packed_out, count_out, stream, 0, nullptr,
                         nullptr, 0.f, ADACOMP_GRAD_F16);
}

int adacomp_compress_opt(const void *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                         uint64_t *count_out, const adacomp_options *opt, void *stream)
{
    const adacomp_options none = {0u, ADACOMP_GRAD_F32, 0.f, ADACOMP_QUANT_BIN_MAX_MEAN, nullptr};
    const adacomp_options &o = opt ? *opt : none;
    return compress_impl(static_cast<const float *>(grad), residue, n, L_T, packed_out, count_out, stream, o.flags, nullptr,
                         o.lazy_state, o.factor, o.grad_type, nullptr, o.quantiser);
}

int adacomp_compress_scaled(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                            uint64_t *count_out, void *stream, float factor)
{
    if (!(factor > 0.f && factor <= 1e30f)) return ADACOMP_ERR_FLAGS;
    return compress_impl(grad, residue, n, L_T, packed_out, count_out, stream, 0, nullptr, nullptr, factor);
}

int adacomp_decompress_average_sgd(const void *const *packed, uint32_t k_streams, float *weights, float *momentum,
                                   uint64_t n, uint32_t L_T, float lr, float mu, void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    const Epilogue ep = {weights, momentum, nullptr, lr, mu, 0.f, 0.f, 0.f, 0u, 0.f};
    return decompress_impl(packed, k_streams, nullptr, stream, n, L_T, &ep);
}

int adacomp_decompress_average_adam(const void *const *packed, uint32_t k_streams, float *weights, float *m, float *v,
                                    uint64_t n, uint32_t L_T, float step_size, float beta1, float beta2, float eps,
                                    void *stream)
{
    if (L_T == 0 || L_T > ADACOMP_MAX_L_T) return ADACOMP_ERR_L_T;
    const Epilogue ep = {weights, m, v, step_size, beta1, beta2, eps, 0.f, 1u, 0.f};
    return decompress_impl(packed, k_streams, nullptr, stream, n, L_T, &ep);
}

size_t adacomp_v2_capacity(uint64_t n, uint32_t L_T)
{
    if (L_T == 0 || L_T >= ADACOMP_MAX_L_T) return 0;
    const Geometry g = make_geometry(n, L_T);
    return (size_t)(align_up(kHeaderBytes + 8 * (g.n_tiles + 1), 16) + align_up(n * (L_T <= 63u ? 1u : 2u), 16));
}

int adacomp_stream_to_v2(const void *packed, void *out_v2, uint64_t out_capacity, uint64_t *count_out, uint64_t n,
                         uint32_t L_T, void *stream)
{
    return stream_convert(packed, out_v2, out_capacity, count_out, n, L_T, true, stream);
}

int adacomp_stream_from_v2(const void *in_v2, void *packed_out, uint64_t out_capacity, uint64_t n, uint32_t L_T,
                           void *stream)
{
    return stream_convert(in_v2, packed_out, out_capacity, nullptr, n, L_T, false, stream);
}

int adacomp_debug_waits(uint64_t wait_cycles, uint32_t withhold_pack_tile, uint32_t withhold_decode_item)
{
    g_debug_waits.limit = wait_cycles ? (long long)(wait_cycles < (1ull << 40) ? wait_cycles : (1ull << 40)) : kWaitCycles;
    g_debug_waits.withhold_pack = withhold_pack_tile;
    g_debug_waits.withhold_decode = withhold_decode_item;
    return ADACOMP_OK;
}

int adacomp_set_device(int device)
{
    return cudaSetDevice(device) == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

int adacomp_device_status(uint32_t *host_out, void *stream)
{
    if (!host_out) return ADACOMP_ERR_NULL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ADACOMP_ERR_CUDA;
    u32 v = 0;
    const bool ok = status_read_pack(&v) &&
                    status_read_pack_fast_a(&v) &&
                    status_read_pack_fast_b(&v) &&
                    status_read_pack_fast_c(&v) &&
                    status_read_pack_fast_d(&v) &&
                    status_read_pack_batch(&v) &&
                    status_read_pack_onchip(&v) &&
                    status_read_pack_onchip_list(&v) &&
                    status_read_decode(&v) &&
                    status_read_decode_opt(&v) &&
                    status_read_decode_batch(&v) &&
                    status_read_wire(&v);
    if (!ok) return ADACOMP_ERR_CUDA;
    *host_out = v;
    return ADACOMP_OK;
}

int adacomp_device_status_reset(void *stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    status_reset_pack(st);
    status_reset_pack_fast_a(st);
    status_reset_pack_fast_b(st);
    status_reset_pack_fast_c(st);
    status_reset_pack_fast_d(st);
    status_reset_pack_batch(st);
    status_reset_pack_onchip(st);
    status_reset_pack_onchip_list(st);
    status_reset_decode(st);
    status_reset_decode_opt(st);
    status_reset_decode_batch(st);
    status_reset_wire(st);
    return cudaGetLastError() == cudaSuccess ? ADACOMP_OK : ADACOMP_ERR_CUDA;
}

}  // extern "C"
