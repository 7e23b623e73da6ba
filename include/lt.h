/* lt.h -- C ABI of the fused global-norm clip + block-wise 8-bit AdamW optimizer step (sm_100a).
 *
 * The operator is the optimizer-side component the paper calls the hybrid 8-bit operator (Sec. 3.5):
 * Adam moments held as 8-bit codes with block-wise scales, updated by an AdamW step, coupled with a
 * fast global-norm gradient clip. Here every step of it runs on the GPU, on the caller's stream.
 *
 * Conventions for every function
 *   - returns LT_OK (0) or a negative lt_status; never throws, never aborts, never synchronises the
 *     stream (one exception: the FIRST call on a device uploads the code tables and waits for that
 *     upload; make that call before any stream capture);
 *   - never allocates or frees device memory;
 *   - lt_tensor arrays, lt_hparams and out-parameters of the host-side queries are HOST memory read
 *     during the call; every pointer INSIDE an lt_tensor, and d_sqnorm / d_status / d_workspace, are
 *     DEVICE pointers owned by the caller that must stay valid until the enqueued work has run;
 *   - arguments are validated on the host before anything is launched: a call that returns an
 *     error has enqueued nothing (LT_ERR_CUDA excepted: a launch itself failed).
 *
 * Data layout. A tensor is a flat array of `numel` elements. Its 8-bit state is one byte per element
 * per moment (m_code: index into the signed 256-entry map; v_code: index into the unsigned map) and
 * one fp32 scale per block of `block` consecutive elements per moment (the block's absolute maximum).
 * Blocks restart at every tensor; the last block of a tensor may be short. The value-zero state is
 * m_code = 127, v_code = 0, scales = 0.
 */
#ifndef LT_H_
#define LT_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    LT_OK = 0,
    LT_ERR_INVALID_ARG = -1,  /* null pointer, negative size, bad enum, bad hyper-parameter */
    LT_ERR_ALIGNMENT = -2,    /* a pointer is not aligned to its element size */
    LT_ERR_UNSUPPORTED = -3,  /* block size not a power of two in [256, 16384] */
    LT_ERR_CUDA = -4,         /* a CUDA call or launch failed (the CUDA error is consumed) */
    LT_ERR_WORKSPACE = -5     /* workspace missing, misaligned or smaller than lt_workspace_bytes() */
} lt_status;

typedef enum { LT_F32 = 0, LT_BF16 = 1 } lt_dtype;

/* How a tensor's Adam moments are stored. The paper's measured configuration is a hybrid (Sec. 3.5 and the
 * variant-configuration table): ordinary fp32 Adam states for most parameters, 8-bit states for a 2 % slice. */
typedef enum { LT_STATE_U8 = 0, LT_STATE_F32 = 1 } lt_state_dtype;

/* A CUDA stream handle (cudaStream_t / CUstream); NULL is the default stream. */
typedef struct CUstream_st* lt_stream;

typedef struct {
    void* param;          /* device [numel] of param_dtype; read and written by lt_hybrid8_step      */
    const void* grad;     /* device [numel] of grad_dtype; read only, never rescaled in place        */
    uint8_t* m_code;      /* device [numel]                                                         */
    uint8_t* v_code;      /* device [numel]                                                         */
    float* m_absmax;      /* device [ceil(numel / block)]                                           */
    float* v_absmax;      /* device [ceil(numel / block)]                                           */
    int64_t numel;        /* >= 0; a tensor with 0 elements is skipped                               */
    int32_t param_dtype;  /* lt_dtype                                                               */
    int32_t grad_dtype;   /* lt_dtype                                                               */
    int32_t state_dtype;  /* lt_state_dtype. LT_STATE_F32: m_code and v_code point to float[numel]
                             (4-byte aligned) holding the moments themselves; m_absmax / v_absmax are
                             ignored and may be NULL; value-zero state is all zeros                    */
    int32_t reserved;     /* set to 0                                                               */
} lt_tensor;

/* Hyper-parameters of one optimizer step (the paper's training-configuration table uses
 * beta1 0.9, beta2 0.999, eps 1e-8, lr 1e-5, weight_decay 0.01, max_norm 1.0). `step` is the 1-based
 * step count, supplied by the caller. max_norm <= 0 or +inf disables clipping. */
typedef struct {
    float lr, beta1, beta2, eps, weight_decay, max_norm;
    int64_t step;
} lt_hparams;

/* Bytes of 8-bit state for a tensor of `numel` elements: codes per moment (= numel) and scales per
 * moment (= 4 * ceil(numel / block)). The paper's optimizer-memory rows (full 8-bit vs 2 % 8-bit
 * Adam states, solver-snapshot table) are consistent with exactly this footprint at block 4096. */
int lt_hybrid8_state_bytes(int64_t numel, int32_t block, int64_t* code_bytes, int64_t* absmax_bytes);

/* Copies the 256-entry code map (signed: first moment, unsigned: second moment) to host memory.
 * Decade e = 0..6 with scale 10^(e-6) holds 2^e (signed) or 2^(e+1) (unsigned) cell mid-points of a
 * uniform grid on [0.1, 1]; plus 0.0 and +1.0 (the paper gives the format a name only -- an 8-bit AdamW
 * format held in CPU memory, Sec. 3.5 --; this map is this library's reading of it). */
int lt_hybrid8_code_table(int32_t is_signed, float* out256);

/* Size in bytes of the device scratch lt_grad_sqnorm_multi needs (a constant, a few KB). The scratch
 * must be 256-byte aligned; its contents need no initialisation and mean nothing between calls.
 * Calls that run concurrently on the GPU must not share one scratch buffer. */
int64_t lt_workspace_bytes(void);

/* S0 -- puts the 8-bit state of every tensor to value zero (m_code 127, v_code 0, scales 0).
 * Uses m_code, v_code, m_absmax, v_absmax, numel. (Sec. 3.5: the moments of the 8-bit slice are held in an
 * 8-bit AdamW format.) */
int lt_hybrid8_state_init(const lt_tensor* tensors, int32_t n, int32_t block, lt_stream stream);

/* S1 -- multi-tensor squared L2 norm (Sec. 3.5: the clip takes a norm per tensor and combines them into
 * one global norm). ADDS sum_t sum_i grad[t][i]^2 to *d_sqnorm (device double). The caller zeroes
 * *d_sqnorm before the first chunk of an optimizer step and may call this once per chunk of the
 * tensor list. Uses grad, grad_dtype, numel. Accumulation is fp64 over exact squares; the
 * result is bit-reproducible for a given tensor list on a given device.
 * The launch finishes with a plain read-add-write of *d_sqnorm by one thread: calls that accumulate into
 * the same scalar must be ordered on the GPU (one stream, or events between streams). Two calls that may
 * overlap need a scalar each (and a scratch buffer each); add the scalars afterwards. */
int lt_grad_sqnorm_multi(const lt_tensor* tensors, int32_t n, double* d_sqnorm,
                         void* d_workspace, int64_t workspace_bytes, lt_stream stream);

/* S2..S5 -- the fused step (Sec. 3.5: dequantize the 8-bit moments, update them, requantize them with
 * fresh per-block scales, all under the clip's single scale). Reads S = *d_sqnorm, the squared norm
 * over ALL gradients of this optimizer step (the tensor list may be one chunk of them):
 *     c   = min(1, max_norm / (sqrt(S) + 1e-6))                       (1 if clipping is disabled)
 *     g   = c * grad;   m = QS[m_code] * m_absmax[b];   v = QU[v_code] * v_absmax[b]
 *     m'  = beta1 m + (1 - beta1) g;    v' = beta2 v + (1 - beta2) g^2
 *     p  <- p (1 - lr wd) - lr / (1 - beta1^t) * m' / (sqrt(v') / sqrt(1 - beta2^t) + eps)
 *     per block: m_absmax = max |m'|, v_absmax = max v', codes = nearest map entry of m'/m_absmax,
 *     v'/v_absmax (ties to the lower index; an all-zero block gets zero codes and scale 0).
 * Tensors with state_dtype LT_STATE_F32 get the same update with m, v read and written as fp32 (no
 * tables, no block scales); both kinds may be mixed in one list and share the clip factor.
 * If S is NaN or Inf nothing is written except bit 0 of *d_status (the skip-on-non-finite rule of the
 * paper's training-configuration table, safety-checks row); the caller clears d_status when it wants to.
 * d_sqnorm may be NULL only when clipping is disabled (no skip detection then). d_status may be NULL.
 * Status word: bit 0 (value 1) = this step was skipped because S is not finite. Bit 1 (value 2) = the
 * kernel found its shared-memory window laid out differently from what it was built for and did nothing
 * (a build or driver inconsistency, never expected; reported instead of risking a bad access). Bits are
 * only ever set, by atomic OR.
 * Moment arithmetic is IEEE fp32 with one rounding per operation (no fused multiply-add), so the stored
 * state is that of a plain evaluation of the formulas above. The parameter update uses the hardware's
 * approximate sqrt and reciprocal; its distance from the IEEE evaluation of the formula is bounded by
 *     6.6e-7 |update| + 1.2e-7 |p_new|      (update = the term subtracted from p (1 - lr wd)),
 * at any step size: within 1e-5 of max(|p_new|, |update|) for fp32 parameters. bf16 parameters whose result
 * cancels to below 2^-11 of p (1 - lr wd) take the IEEE formula instead, which keeps every rounded result
 * within one bf16 ulp (elements that are not flagged have |update| <= 2049 |p_new|, and the bound above is
 * then below half a bf16 ulp). With eps < 1e-12 the whole launch takes the IEEE formula (the approximate
 * sqrt flushes subnormal v'). */
int lt_hybrid8_step(const lt_tensor* tensors, int32_t n, int32_t block, const lt_hparams* hp,
                    const double* d_sqnorm, int32_t* d_status, lt_stream stream);

/* Per-tensor squared L2 norms, for logging (Sec. 3.5: the clip's first stage is a norm per tensor).
 * ADDS sum_i grad[t][i]^2 to d_out[t] for every tensor t of the list (device doubles,
 * one per list entry, zeroed by the caller; entries of empty tensors are left alone). Uses grad,
 * grad_dtype, numel. Each addend is an exact fp64 square; per-CTA partial sums reach d_out[t] through
 * fp64 atomic adds, so the last bits may differ from run to run -- use lt_grad_sqnorm_multi for the norm
 * that feeds the clip. No workspace. */
int lt_grad_sqnorm_per_tensor(const lt_tensor* tensors, int32_t n, double* d_out, lt_stream stream);

/* Skip bookkeeping, once per optimizer step, after the step's norm is complete (training-configuration
 * table, safety-checks row: a step with non-finite gradients is skipped, and three such steps in a row end
 * the run). Reads S = *d_sqnorm and updates the device word *d_skip_count: S finite -> 0, S NaN/Inf ->
 * previous value + 1. The caller reads it when it likes and applies its abort policy; nothing here
 * aborts. One thread of device work. */
int lt_skip_count_update(const double* d_sqnorm, int32_t* d_skip_count, lt_stream stream);

/* Step count and the two step-dependent scalars, resident on the DEVICE, so that a whole optimizer step
 * (norm, bookkeeping, update) can be recorded once in a CUDA graph and replayed every step with no host
 * arithmetic in between. (No counterpart in the paper, whose optimizer runs on the host.) The caller
 * allocates one lt_step_state on the device and zeroes it (step 0). */
typedef struct {
    int64_t step;          /* steps taken so far; lt_step_state_advance adds one          */
    float step_size;       /* lr / (1 - beta1^step)                                       */
    float inv_sqrt_bc2;    /* 1 / sqrt(1 - beta2^step)                                    */
} lt_step_state;

/* One thread of device work: d_state->step += 1, then step_size and inv_sqrt_bc2 for the new count from
 * hp->lr, hp->beta1, hp->beta2 (formed in fp64, rounded once to fp32, like the host path; the device's
 * fp64 pow may differ from the host's in the last bit, which can move step_size by one fp32 ulp).
 * d_sqnorm (device, may be NULL): when given and *d_sqnorm is NaN or Inf, nothing changes -- the step that
 * follows will be skipped, and a skipped step must not count towards the bias corrections. */
int lt_step_state_advance(lt_step_state* d_state, const lt_hparams* hp, const double* d_sqnorm, lt_stream stream);

/* lt_hybrid8_step with the step count taken from the device: identical except that hp->step is ignored
 * and step_size / inv_sqrt_bc2 are read from *d_state by the kernels. */
int lt_hybrid8_step_graph(const lt_tensor* tensors, int32_t n, int32_t block, const lt_hparams* hp,
                          const lt_step_state* d_state, const double* d_sqnorm, int32_t* d_status,
                          lt_stream stream);

/* Largest number of non-empty tensors one lt_grad_sqnorm_multi_noalloc call accepts. */
#define LT_NOALLOC_MAX_TENSORS 480

/* (No counterpart in the paper: an addition for callers that cannot allocate.)
 * lt_grad_sqnorm_multi without a workspace argument. Some callers have no way to obtain device
 * scratch at the point where they need the norm: code running under a framework allocator it must
 * not call into, a region where cudaMalloc is forbidden because it would synchronise the device or
 * break a capture in progress elsewhere in the process, or a plain C host that was handed gradient
 * pointers and nothing else. For them the scratch (an arrival counter and up to 512 per-CTA partial
 * sums, 4352 bytes) lives in a device array inside the library; every GPU that loads the library
 * holds those bytes until the process exits. The call allocates and frees nothing, on host-visible
 * CUDA APIs or otherwise.
 *   - Same result contract as lt_grad_sqnorm_multi: ADDS the sum of squares to *d_sqnorm.
 *   - At most LT_NOALLOC_MAX_TENSORS non-empty tensors per call (one launch over the fixed scratch);
 *     more returns LT_ERR_WORKSPACE and enqueues nothing. Split longer lists over several calls.
 *   - The first call on a device looks the array's device address up (and, if it is the library's
 *     first call on that device at all, uploads the code tables and waits for that upload): make the
 *     first call before any stream capture.
 *   - All calls on a device share the one array. It keeps the previous call's contents; the call
 *     clears the counter it needs at zero itself. Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on it and give wrong sums: order them. */
int lt_grad_sqnorm_multi_noalloc(const lt_tensor* tensors, int32_t n, double* d_sqnorm, lt_stream stream);

/* Name of a status code (static string). */
const char* lt_status_str(int status);

#ifdef __cplusplus
}
#endif
#endif /* LT_H_ */
