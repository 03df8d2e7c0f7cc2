// Host-side declarations shared by the translation units of libadacomp: what each of them tells the others
// about this device, and the launchers they call across files.
#pragma once

#include "pack_batch.cuh"
#include "decode_batch.cuh"

namespace adacomp_impl {

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    int decode_per_sm = 0;
    int decode_warps_per_sm = 0, decode_one_per_sm = 0;
    int decode_pair_per_sm = 0;         // 0: the kernel of pair_path() cannot be launched on this device
    int decode_opt_per_sm[2][2] = {{0, 0}, {0, 0}};     // [SGD, Adam][4, 8 decoding warps]; 0: unavailable on this device
    int batch_per_sm = 0;
    bool batch_fast_ready = false;      // the pipelined batch tile pass can be launched       // 0: batched pack() unavailable on this device
    int dec_batch_per_sm = 0;   // 0: batched decode unavailable on this device
    int dec_batch_warps_per_sm[3] = {0, 0, 0};      // CTAs of the batched warp decoder per SM, by optimizer form
    bool fast_ready = false;
    int onchip_ctas = 0;        // CTAs of the one-kernel pack() that are resident together; 0: unavailable on this device
    int onchip_list_ctas = 0;   // the same for the one-kernel pack() of a parameter list
};


// This device's record, filled on the first call (abi.cu asks every file below for its share).
int device_info(DeviceInfo *&out);
void init_pack_info(DeviceInfo &d);             // pack.cu, pack_fast_*.cu
void init_pack_batch_info(DeviceInfo &d);       // pack_batch.cu
void init_pack_onchip_info(DeviceInfo &d);      // pack_onchip.cu
void init_pack_onchip_list_info(DeviceInfo &d); // pack_onchip_list.cu (after init_pack_onchip_info)
void init_decode_info(DeviceInfo &d);           // decode.cu, decode_opt.cu
void init_decode_batch_info(DeviceInfo &d);     // decode_batch.cu

// pack_fast_a.cu .. pack_fast_d.cu: the instances of the pipelined tile pass, a few bin lengths per file.
// With `args` null: allows the kernels their dynamic shared memory (false: some kernel cannot be launched).
// Else: launches the kernel that takes args->geo.L_T (lazy-scale when args->lazy_state is set, the gradient
// format of args->grad_type) and returns true, or returns false when the bin length is another file's.
bool fast_tile_pass_a(const PassArgs *args, unsigned grid, cudaStream_t st);
bool fast_tile_pass_b(const PassArgs *args, unsigned grid, cudaStream_t st);
bool fast_tile_pass_c(const PassArgs *args, unsigned grid, cudaStream_t st);
bool fast_tile_pass_d(const PassArgs *args, unsigned grid, cudaStream_t st);

// abi.cu: what adacomp_debug_waits last set (the defaults: kWaitCycles, nothing withheld)
const DebugWaits &debug_waits();

// pack.cu
int compress_impl(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                  uint64_t *count_out, void *stream, uint32_t flags, void *const *events = nullptr,
                  void *lazy_state = nullptr, float factor = 0.f, uint32_t grad_type = ADACOMP_GRAD_F32,
                  unsigned char *own_scratch = nullptr, uint32_t quantiser = ADACOMP_QUANT_BIN_MAX_MEAN);
int compress_static_impl(const float *grad, float *residue, uint64_t n, uint32_t L_T, void *packed_out,
                         uint64_t *count_out, void *stream);
int lazy_state_init(void *state, uint64_t n, uint32_t L_T, void *stream);
int residue_flush(float *residue, void *state, uint64_t n, uint32_t L_T, void *stream);

// pack_batch.cu
int launch_batch(const BatchArgs &b, const DeviceInfo &info, cudaStream_t st, bool lazy = false);

// decode.cu (plain decoding), decode_opt.cu (with an optimizer step)
int decompress_impl(const void *const *packed, uint32_t k, float *dst, void *stream, uint64_t hint_n = 0,
                    uint32_t hint_L_T = 0, const Epilogue *ep = nullptr);
int launch_decode_opt(const DecodeArgs &args, const Epilogue &ep, const DeviceInfo &info, uint64_t hint_n,
                      uint32_t hint_L_T, cudaStream_t st);

// pack_onchip.cu: pack() of a layer whose tiles all fit in the resident CTAs' shared memory, in one kernel
u64 onchip_tile_capacity(const DeviceInfo &d);
int launch_pack_onchip(PassArgs &args, u64 *count_out, u32 header_flags, const DeviceInfo &info, cudaStream_t st);

// pack_onchip_list.cu: the same for a batch of layers (the layers' control blocks cleared before)
bool onchip_list_takes(const BatchArgs &b, const DeviceInfo &info);
int launch_pack_onchip_list(const BatchArgs &b, const DeviceInfo &info, long long wait_limit, cudaStream_t st);

// wire.cu: a packed stream re-encoded as version 2 (to_v2) or back as version 1
int stream_convert(const void *in, void *out, uint64_t out_capacity, uint64_t *count_out, uint64_t n, uint32_t L_T,
                   bool to_v2, void *stream);

// decode_batch.cu
int launch_decode_batch(const DecodeBatchArgs &batch, u64 batch_tiles, const DeviceInfo &info, cudaStream_t st);

inline bool batchable(const adacomp_layer_desc &d, const DeviceInfo &info)
{
    return d.flags == 0 && d.L_T >= 42u && d.L_T <= 1000u && d.n < (info.batch_fast_ready ? kPackBatchMaxElems : kBatchLayerMaxElems);
}

// every file with kernels: its status word (see common.cuh)
ADACOMP_STATUS_DECLARE(pack)
ADACOMP_STATUS_DECLARE(pack_fast_a)
ADACOMP_STATUS_DECLARE(pack_fast_b)
ADACOMP_STATUS_DECLARE(pack_fast_c)
ADACOMP_STATUS_DECLARE(pack_fast_d)
ADACOMP_STATUS_DECLARE(pack_batch)
ADACOMP_STATUS_DECLARE(pack_onchip)
ADACOMP_STATUS_DECLARE(pack_onchip_list)
ADACOMP_STATUS_DECLARE(decode)
ADACOMP_STATUS_DECLARE(decode_opt)
ADACOMP_STATUS_DECLARE(decode_batch)
ADACOMP_STATUS_DECLARE(wire)

}  // namespace adacomp_impl
