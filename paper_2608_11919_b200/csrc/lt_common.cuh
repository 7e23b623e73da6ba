// Internal declarations shared by the translation units of liblt_hybrid8 (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lt.h"

namespace lt {

// Tensors per launch: descriptors travel as kernel parameters (no device table, no copy to keep
// alive), and the parameter space of sm_100 holds 32764 bytes.
constexpr int kCap = 480;
constexpr int kMaxDevices = 64;   // device ordinals the per-device caches cover

constexpr int kFlagParamBf16 = 1;
constexpr int kFlagGradF32 = 2;
constexpr int kFlagVecOk = 4;   // every pointer allows 4-element vector access (after the common shift, if any)
constexpr int kFlagStateF32 = 16; // moments are plain fp32 arrays (mc / vc point to float)
constexpr int kFlagShiftPos = 8;  // bits 8-9: elements to skip until all four arrays are vector-aligned together
constexpr int kFlagBulkOk = 8;  // every pointer is 16-byte aligned (bulk prefetch of whole blocks allowed)

struct StepDesc {               // 64 bytes
    void* p;
    const void* g;
    uint8_t* mc;
    uint8_t* vc;
    float* am;
    float* av;
    int64_t numel;
    int32_t blk_end;            // exclusive end of this tensor's range of launch-wide block indices
    int32_t flags;
};

struct StepScalars {
    float beta1, beta2, omb1, omb2, step_size, inv_sqrt_bc2, decay, eps, max_norm;
    float one;                  // 1.0f, a run-time value on purpose (lt_step.cu, add2_rt)
    int32_t clip_on;
    int32_t precise_param;      // 1: IEEE sqrt and divide in the parameter update (tiny eps)
};

// Direct-lookup quantizer tables (one packed 32-bit word per bucket, see lt_api.cu). Two forms exist:
// "full" covers every float below 2 (exponent fields 0..127: 128 binades, the input needs no clamping),
// "compact" covers [2^-31, 2) (exponent fields 96..127: 32 binades, the kernel clamps smaller inputs up
// to 2^-31, which share the zero code). The signed table has 64 buckets per binade and two halves
// (positive, negative), the unsigned one 128 buckets per binade.
constexpr int lut_s_entries(bool full) { return (full ? 128 : 32) * 64 * 2; }
constexpr int lut_u_entries(bool full) { return (full ? 128 : 32) * 128; }

struct StepParams {
    StepDesc t[kCap];
    StepScalars s;
    const double* sqnorm;
    int32_t* status;
    const float* dev_scalars;   // non-null: {step_size, inv_sqrt_bc2} are read from the device (lt_step_state)
    int32_t n;
    int32_t total_blocks;
    int32_t param_bf16;         // parameter dtype of every tensor of this launch
};

struct NormDesc {               // 32 bytes
    const void* base16;         // gradient address rounded down to 16 bytes
    int64_t span_bytes;         // lead bytes + numel * element size
    int32_t item_end;           // exclusive end of this tensor's range of launch-wide work items
    int32_t lead_f32;           // lead bytes (0..15) | grad_is_f32 << 8
    int32_t slot;               // per-tensor output index (per-tensor norm kernel only)
    int32_t pad;
};

struct NormParams {
    NormDesc t[kCap];
    double* partials;           // workspace: one double per CTA
    unsigned int* ticket;       // workspace: arrival counter, zero between launches
    double* out;                // *out += total
    int32_t n;
    int32_t total_items;
};

struct DeviceInfo {
    int sm_count = 0;
    bool tables_ready = false;
};

// per-device lazy set-up (SM count, code tables in constant memory). Returns LT_OK or LT_ERR_CUDA.
int ensure_device(cudaStream_t stream, DeviceInfo** out);

// host copies of the code maps and of the search thresholds (mid-points rounded toward -inf)
const float* host_table(bool is_signed);
const float* host_mid_rd(bool is_signed);
const uint32_t* host_lut(bool is_signed, bool full);   // nullptr if the maps do not fit the bucket grid

int launch_state_init(const StepParams& p, int block, int sm_count, cudaStream_t s);
int launch_step(const StepParams& p, int block, int sm_count, cudaStream_t s);
int launch_adamw32(const StepParams& p, int sm_count, cudaStream_t s);   // tensors with fp32 moments
#ifndef LT_A32_ITEM
#define LT_A32_ITEM 8192
#endif
constexpr int kAdamw32Item = LT_A32_ITEM;   // elements per work item of that kernel (items restart at every tensor)
int launch_sqnorm(const NormParams& p, int sm_count, cudaStream_t s);
// Host-side checks of the fields the norm kernels read (grad, grad_dtype, numel); *live = non-empty tensors.
int validate_grads(const lt_tensor* t, int32_t n, int* live);
// Packs tensors [*i, n) into one launch's descriptors: at most kCap non-empty tensors and fewer than 2^31
// work items; advances *i past what it took. P->n == 0 when nothing was left. slot = index in the list.
void pack_norm(const lt_tensor* t, int32_t n, int32_t* i, NormParams* P);
int launch_step_state_advance(lt_step_state* d_state, float lr, float beta1, float beta2, const double* d_sqnorm,
                              cudaStream_t s);
int upload_tables(cudaStream_t s);

// Launch shape of the norm kernels: one 1024-thread CTA per SM, eight 16-byte loads per thread and item
// (128 KiB in flight per SM). Measured on 15 GB of bf16 gradients, sustained: 6.8 TB/s, against 6.2 TB/s for two
// 512-thread CTAs with four loads per thread (half the bytes in flight), 6.6 for 512 x 8 x 2, 6.9 for 1024 x 10 x 1.
#ifndef LT_NORM_THREADS
#define LT_NORM_THREADS 1024
#define LT_NORM_VPT 8
#define LT_NORM_CTAS 1
#endif
constexpr int kNormThreads = LT_NORM_THREADS;
constexpr int kNormVecPerThread = LT_NORM_VPT;
constexpr int kNormCtasPerSm = LT_NORM_CTAS;
constexpr int kNormItemBytes = kNormThreads * kNormVecPerThread * 16;
constexpr int kNormMaxCtas = 1024;
constexpr int64_t kWorkspaceBytes = 256 + kNormMaxCtas * 8;

}  // namespace lt
