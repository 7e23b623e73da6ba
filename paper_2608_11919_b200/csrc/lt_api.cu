// Host side of the C ABI: argument validation, code-map construction, per-launch descriptor packing.
#include <cmath>
#include <cstring>
#include <mutex>

#include "lt_common.cuh"

namespace lt {

// ---- code maps (host) --------------------------------------------------------------------------
// Signed map: 127 negative magnitudes (descending), 0.0, 127 positive magnitudes, +1.0.
// Unsigned map: 0.0, 254 magnitudes, +1.0. Magnitudes of decade e: 10^(e-6) * (0.1 + 0.9 (j+.5)/n_e),
// n_e = 2^e (signed) or 2^(e+1) (unsigned), formed in double and rounded once to fp32.
struct HostTables {
    float qs[256], qu[256];
    float mid_s[256], mid_u[256];   // [k] = (T[k] + T[k+1]) / 2 rounded toward -inf; [255] = +inf
    uint32_t lut_u_full[lut_u_entries(true)], lut_s_full[lut_s_entries(true)];        // see build_lut
    uint32_t lut_u_compact[lut_u_entries(false)], lut_s_compact[lut_s_entries(false)];
    bool lut_ok;
    HostTables() {
        static const double decade[7] = {1e-6, 1e-5, 1e-4, 1e-3, 1e-2, 1e-1, 1e0};
        int is = 0, iu = 1;
        qu[0] = 0.0f;
        qs[127] = 0.0f;
        for (int e = 0; e < 7; ++e) {
            const int ns = 1 << e, nu = 2 << e;
            for (int j = 0; j < ns; ++j) {
                const float f = (float)(decade[e] * (0.1 + 0.9 * ((double)j + 0.5) / (double)ns));
                qs[128 + is] = f;
                qs[126 - is] = -f;
                ++is;
            }
            for (int j = 0; j < nu; ++j)
                qu[iu++] = (float)(decade[e] * (0.1 + 0.9 * ((double)j + 0.5) / (double)nu));
        }
        qs[255] = 1.0f;
        qu[255] = 1.0f;
        fill_mid(qs, mid_s);
        fill_mid(qu, mid_u);
        lut_ok = build_lut(mid_u, 7, false, 128, lut_u_full) && build_lut(mid_s, 6, true, 128, lut_s_full, true) &&
                 build_lut(mid_u, 7, false, 32, lut_u_compact) && build_lut(mid_s, 6, true, 32, lut_s_compact);
    }
    static int code_of(const float* mid, float x) {   // number of thresholds strictly below x
        int c = 0;
        for (int k = 0; k < 255; ++k) c += (x > mid[k]) ? 1 : 0;
        return c;
    }
    static float from_bits(uint32_t b) { float f; std::memcpy(&f, &b, 4); return f; }
    // Direct-lookup form of the search. A bucket is the set of floats below 2 that share sign,
    // exponent field (0..127, subnormals included) and the top `mbits` mantissa bits; `frac` is the
    // rest of the mantissa and H the bits above it (constant over the bucket). (A table may instead
    // cover only exponent fields 96..127; the kernel then clamps smaller magnitudes up to 2^-31, which
    // share the zero code.) The code map is so
    // coarse against that grid that a bucket holds at most one threshold T, so code(x) = base +
    // (x > T) with base = code of the bucket's smallest value. An entry packs both into one word so
    // that ONE integer add of the magnitude bits a = |x| decides; the code is the top byte of the sum:
    //   x >= 0:  entry = (base << 24 | 0xFFFFFF - frac(T)) - H;        sum = entry + a
    //            (carries into bits 24.. exactly when frac(x) > frac(T); no T: frac(T) = all ones)
    //   x <  0:  entry = ((base + 1) << 24 | frac(T)) + H;             sum = entry + ~a
    //            (= (base + 1) << 24 + frac(T) - frac(x) - 1, which keeps base + 1 exactly when
    //            frac(x) < frac(T), i.e. x > T; no T: frac(T) = 0)
    //            With neg_adds_iabs the kernel adds |u|_int of the raw bits u instead (one instruction):
    //            for u < 0, |u|_int = ~a - 0x7fffffff, so the entry carries + 0x7fffffff.
    // Unsigned map: 128 x 128 buckets. Signed map: 128 x 64 buckets of the magnitude, positive half
    // first, negative half second. Exponent fields 128..255 (|x| >= 2, Inf, NaN) cannot occur for a
    // normalised moment; the kernel masks the index so that even then the lookup stays inside the table.
    static bool build_lut(const float* mid, int mbits, bool is_signed, int binades, uint32_t* lut, bool neg_adds_iabs = false) {
        const int per_binade = 1 << mbits, half = binades * per_binade, fbits = 23 - mbits;
        const int e_first = 128 - binades;   // first exponent field covered
        const uint32_t fmask = (1u << fbits) - 1u;
        for (int h = 0; h < (is_signed ? 2 : 1); ++h) {
            for (int key = 0; key < half; ++key) {
                const uint32_t lo = ((uint32_t)(e_first + key / per_binade) << 23) | ((uint32_t)(key % per_binade) << fbits);
                const uint32_t hi = lo | fmask;
                const float xa = h == 0 ? from_bits(lo) : -from_bits(hi);   // smallest value of the bucket
                const float xb = h == 0 ? from_bits(hi) : -from_bits(lo);   // largest
                const int ca = code_of(mid, xa), cb = code_of(mid, xb);
                bool has_t = false;
                uint32_t tf = 0;
                if (cb == ca + 1) {
                    uint32_t tb; std::memcpy(&tb, &mid[ca], 4);
                    if (((tb & 0x7fffffffu) & ~fmask) != lo) return false;   // T must lie in this bucket
                    has_t = true;
                    tf = tb & fmask;
                } else if (cb != ca) {
                    return false;
                }
                if (h == 1 && ca + 1 > 255) return false;
                uint32_t e;
                if (h == 0) e = (((uint32_t)ca << 24) | (0xFFFFFFu - (has_t ? tf : fmask))) - lo;
                else e = (((uint32_t)(ca + 1) << 24) | (has_t ? tf : 0u)) + lo + (neg_adds_iabs ? 0x7fffffffu : 0u);
                lut[h * half + key] = e;
            }
        }
        return true;
    }
    // For fp32 x and a mid-point M that is exact in double: x > M  <=>  x > round_down(M).
    static void fill_mid(const float* T, float* mid) {
        for (int k = 0; k < 255; ++k) {
            const double m = ((double)T[k] + (double)T[k + 1]) * 0.5;
            float f = (float)m;
            if ((double)f > m) f = std::nextafterf(f, -INFINITY);
            mid[k] = f;
        }
        mid[255] = INFINITY;
    }
};

static const HostTables& host_tables() {
    static HostTables t;
    return t;
}
const float* host_table(bool is_signed) { return is_signed ? host_tables().qs : host_tables().qu; }
const float* host_mid_rd(bool is_signed) { return is_signed ? host_tables().mid_s : host_tables().mid_u; }
const uint32_t* host_lut(bool is_signed, bool full) {
    const HostTables& t = host_tables();
    if (!t.lut_ok) return nullptr;
    if (full) return is_signed ? t.lut_s_full : t.lut_u_full;
    return is_signed ? t.lut_s_compact : t.lut_u_compact;
}

// ---- per-device set-up ---------------------------------------------------------------------------
static std::mutex g_mu;
static DeviceInfo g_dev[kMaxDevices];

int ensure_device(cudaStream_t stream, DeviceInfo** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return LT_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceInfo& d = g_dev[dev];
    if (!d.tables_ready) {
        if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            d.sm_count <= 0) { cudaGetLastError(); return LT_ERR_CUDA; }
        if (upload_tables(stream) != LT_OK) return LT_ERR_CUDA;
        if (cudaStreamSynchronize(stream) != cudaSuccess) { cudaGetLastError(); return LT_ERR_CUDA; }
        d.tables_ready = true;
    }
    *out = &d;
    return LT_OK;
}

static bool valid_block(int32_t block) {
    return block >= 256 && block <= 16384 && (block & (block - 1)) == 0;
}
static bool valid_dtype(int32_t d) { return d == LT_F32 || d == LT_BF16; }
static int esize(int32_t d) { return d == LT_F32 ? 4 : 2; }
static bool aligned(const void* p, int a) { return ((uintptr_t)p % (uintptr_t)a) == 0; }

// which fields a call needs
enum { NEED_GRAD = 1, NEED_PARAM = 2, NEED_STATE = 4 };

static int validate_tensors(const lt_tensor* t, int32_t n, int need) {
    if (n < 0 || (n > 0 && t == nullptr)) return LT_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i) {
        const lt_tensor& x = t[i];
        if (x.numel < 0) return LT_ERR_INVALID_ARG;
        if (x.numel > ((int64_t)1 << 38)) return LT_ERR_UNSUPPORTED;   // keeps per-launch block counts in int32
        if (x.numel == 0) continue;
        if (need & NEED_GRAD) {
            if (!valid_dtype(x.grad_dtype) || x.grad == nullptr) return LT_ERR_INVALID_ARG;
            if (!aligned(x.grad, esize(x.grad_dtype))) return LT_ERR_ALIGNMENT;
        }
        if (need & NEED_PARAM) {
            if (!valid_dtype(x.param_dtype) || x.param == nullptr) return LT_ERR_INVALID_ARG;
            if (!aligned(x.param, esize(x.param_dtype))) return LT_ERR_ALIGNMENT;
        }
        if (need & NEED_STATE) {
            if (x.state_dtype != LT_STATE_U8 && x.state_dtype != LT_STATE_F32) return LT_ERR_INVALID_ARG;
            if (!x.m_code || !x.v_code) return LT_ERR_INVALID_ARG;
            if (x.state_dtype == LT_STATE_F32) {
                if (!aligned(x.m_code, 4) || !aligned(x.v_code, 4)) return LT_ERR_ALIGNMENT;
            } else {
                if (!x.m_absmax || !x.v_absmax) return LT_ERR_INVALID_ARG;
                if (!aligned(x.m_absmax, 4) || !aligned(x.v_absmax, 4)) return LT_ERR_ALIGNMENT;
            }
        }
    }
    return LT_OK;
}

// Packs tensors [*i, ...) into one launch's descriptors; advances *i.
// param_dtype >= 0: only tensors whose parameters have that dtype (a launch is dtype-uniform).
// state_dtype >= 0: only tensors with that kind of moments.
static void pack_step(const lt_tensor* t, int32_t n, int32_t block, int32_t* i, StepParams* P, bool with_pg,
                      int param_dtype, int state_dtype = -1) {
    int cnt = 0;
    int64_t blocks = 0;
    while (*i < n && cnt < kCap) {
        const lt_tensor& x = t[*i];
        if (x.numel == 0 || (param_dtype >= 0 && x.param_dtype != param_dtype) ||
            (state_dtype >= 0 && x.state_dtype != state_dtype)) { ++*i; continue; }
        const int64_t nb = (x.numel + block - 1) / block;
        if (blocks + nb > 0x7fffffff) break;   // next launch; one tensor alone always fits (numel <= 2^38)
        StepDesc& d = P->t[cnt];
        d.p = with_pg ? x.param : nullptr;
        d.g = with_pg ? x.grad : nullptr;
        d.mc = x.m_code; d.vc = x.v_code; d.am = x.m_absmax; d.av = x.v_absmax;
        d.numel = x.numel;
        blocks += nb;
        d.blk_end = (int32_t)blocks;
        int flags = 0;
        const bool st32 = x.state_dtype == LT_STATE_F32;
        if (st32) flags |= kFlagStateF32;
        bool vec = st32 ? (aligned(x.m_code, 16) && aligned(x.v_code, 16)) : (aligned(x.m_code, 4) && aligned(x.v_code, 4));
        if (with_pg) {
            if (x.param_dtype == LT_BF16) flags |= kFlagParamBf16;
            if (x.grad_dtype == LT_F32) flags |= kFlagGradF32;
            const int ps = esize(x.param_dtype), gs = esize(x.grad_dtype);
            vec = vec && aligned(x.param, 4 * ps) && aligned(x.grad, 4 * gs);
            if (!vec && !st32) {
                // tensors packed back to back: skipping `sh` elements may align all four arrays at once
                for (int sh = 1; sh < 4; ++sh) {
                    if (aligned((const char*)x.param + sh * ps, 4 * ps) && aligned((const char*)x.grad + sh * gs, 4 * gs) &&
                        aligned(x.m_code + sh, 4) && aligned(x.v_code + sh, 4)) {
                        vec = true;
                        flags |= sh << kFlagShiftPos;
                        break;
                    }
                }
            }
        }
        if (vec) flags |= kFlagVecOk;
        if (with_pg && aligned(x.param, 16) && aligned(x.grad, 16) && aligned(x.m_code, 16) && aligned(x.v_code, 16))
            flags |= kFlagBulkOk;
        d.flags = flags;
        ++cnt; ++*i;
    }
    P->n = cnt;
    P->total_blocks = (int32_t)blocks;
}

}  // namespace lt

using namespace lt;

extern "C" {

const char* lt_status_str(int status) {
    switch (status) {
        case LT_OK: return "LT_OK";
        case LT_ERR_INVALID_ARG: return "LT_ERR_INVALID_ARG";
        case LT_ERR_ALIGNMENT: return "LT_ERR_ALIGNMENT";
        case LT_ERR_UNSUPPORTED: return "LT_ERR_UNSUPPORTED";
        case LT_ERR_CUDA: return "LT_ERR_CUDA";
        case LT_ERR_WORKSPACE: return "LT_ERR_WORKSPACE";
        default: return "LT_ERR_UNKNOWN";
    }
}

int lt_hybrid8_state_bytes(int64_t numel, int32_t block, int64_t* code_bytes, int64_t* absmax_bytes) {
    if (numel < 0 || !code_bytes || !absmax_bytes) return LT_ERR_INVALID_ARG;
    if (!valid_block(block)) return LT_ERR_UNSUPPORTED;
    *code_bytes = numel;
    *absmax_bytes = 4 * ((numel + block - 1) / block);
    return LT_OK;
}

int lt_hybrid8_code_table(int32_t is_signed, float* out256) {
    if (!out256) return LT_ERR_INVALID_ARG;
    std::memcpy(out256, host_table(is_signed != 0), 256 * sizeof(float));
    return LT_OK;
}

int64_t lt_workspace_bytes(void) { return kWorkspaceBytes; }

int lt_hybrid8_state_init(const lt_tensor* tensors, int32_t n, int32_t block, lt_stream stream) {
    if (!valid_block(block)) return LT_ERR_UNSUPPORTED;
    int rc = validate_tensors(tensors, n, NEED_STATE);
    if (rc != LT_OK) return rc;
    DeviceInfo* dev = nullptr;
    if ((rc = ensure_device((cudaStream_t)stream, &dev)) != LT_OK) return rc;
    StepParams P;
    std::memset(&P.s, 0, sizeof(P.s));
    P.sqnorm = nullptr; P.status = nullptr; P.param_bf16 = 0; P.dev_scalars = nullptr;
    int32_t i = 0;
    while (i < n) {
        pack_step(tensors, n, block, &i, &P, false, -1);
        if (P.n == 0) continue;
        if ((rc = launch_state_init(P, block, dev->sm_count, (cudaStream_t)stream)) != LT_OK) return rc;
    }
    return LT_OK;
}

int lt_grad_sqnorm_multi(const lt_tensor* tensors, int32_t n, double* d_sqnorm,
                         void* d_workspace, int64_t workspace_bytes, lt_stream stream) {
    int rc = validate_grads(tensors, n, nullptr);
    if (rc != LT_OK) return rc;
    if (!d_sqnorm) return LT_ERR_INVALID_ARG;
    if (!aligned(d_sqnorm, 8)) return LT_ERR_ALIGNMENT;
    if (!d_workspace || workspace_bytes < kWorkspaceBytes || !aligned(d_workspace, 256)) return LT_ERR_WORKSPACE;
    DeviceInfo* dev = nullptr;
    if ((rc = ensure_device((cudaStream_t)stream, &dev)) != LT_OK) return rc;

    NormParams P;
    P.ticket = (unsigned int*)d_workspace;
    P.partials = (double*)((char*)d_workspace + 256);
    P.out = d_sqnorm;
    int32_t i = 0;
    while (i < n) {
        pack_norm(tensors, n, &i, &P);
        if (P.n == 0) continue;
        // the arrival counter must start at zero whatever an earlier (possibly failed) launch left
        if (cudaMemsetAsync(P.ticket, 0, 256, (cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return LT_ERR_CUDA; }
        if ((rc = launch_sqnorm(P, dev->sm_count, (cudaStream_t)stream)) != LT_OK) return rc;
    }
    return LT_OK;
}

static int step_impl(const lt_tensor* tensors, int32_t n, int32_t block, const lt_hparams* hp_in,
                     const lt_step_state* d_state, bool use_state, const double* d_sqnorm, int32_t* d_status,
                     lt_stream stream) {
    if (!valid_block(block)) return LT_ERR_UNSUPPORTED;
    if (!hp_in) return LT_ERR_INVALID_ARG;
    lt_hparams hp_local = *hp_in;
    if (use_state) {
        if (!d_state) return LT_ERR_INVALID_ARG;
        if (!aligned(d_state, 8)) return LT_ERR_ALIGNMENT;
        hp_local.step = 1;   // any valid count: the kernels read the real scalars from the device
    }
    const lt_hparams* hp = &hp_local;
    int rc = validate_tensors(tensors, n, NEED_GRAD | NEED_PARAM | NEED_STATE);
    if (rc != LT_OK) return rc;
    if (hp->step < 1 || !(hp->beta1 >= 0.0f && hp->beta1 < 1.0f) || !(hp->beta2 >= 0.0f && hp->beta2 < 1.0f) ||
        !(hp->eps >= 0.0f) || !std::isfinite(hp->lr) || !std::isfinite(hp->weight_decay) || std::isnan(hp->max_norm))
        return LT_ERR_INVALID_ARG;
    const bool clip_on = hp->max_norm > 0.0f && !std::isinf(hp->max_norm);
    if (clip_on && !d_sqnorm) return LT_ERR_INVALID_ARG;
    if (d_sqnorm && !aligned(d_sqnorm, 8)) return LT_ERR_ALIGNMENT;
    if (d_status && !aligned(d_status, 4)) return LT_ERR_ALIGNMENT;
    DeviceInfo* dev = nullptr;
    if ((rc = ensure_device((cudaStream_t)stream, &dev)) != LT_OK) return rc;

    StepParams P;
    // per-step scalars: formed in double, rounded once to fp32
    const double b1 = (double)hp->beta1, b2 = (double)hp->beta2, t = (double)hp->step;
    const double bc1 = 1.0 - std::pow(b1, t), bc2 = 1.0 - std::pow(b2, t);
    P.s.beta1 = hp->beta1; P.s.beta2 = hp->beta2;
    P.s.omb1 = (float)(1.0 - b1); P.s.omb2 = (float)(1.0 - b2);
    P.s.step_size = (float)((double)hp->lr / bc1);
    P.s.inv_sqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    P.s.decay = (float)(1.0 - (double)hp->lr * (double)hp->weight_decay);
    P.s.eps = hp->eps;
    P.s.one = 1.0f;
    P.s.max_norm = hp->max_norm;
    P.s.clip_on = clip_on ? 1 : 0;
    // The approximate parameter update (hardware sqrt and reciprocal approximations) is within
    // 6.6e-7 |update| + 1.2e-7 |p'| of the defined one (derivation in lt_update.cuh): inside 1e-5 of
    // max(|p'|, |update|) for fp32 parameters at any step size, and inside one bf16 ulp under the kernels'
    // cancellation guard. One case is outside that derivation: the fast path flushes a subnormal v' to zero,
    // which is harmless only against a sane eps (sqrt of a subnormal is at most 1.1e-19: against
    // eps >= 1e-12 its loss is below 1.1e-7 of the denominator). Smaller eps takes the exact path.
    const bool precise = hp->eps < 1e-12f;
    P.sqnorm = d_sqnorm;
    P.status = d_status;
    P.dev_scalars = use_state ? &d_state->step_size : nullptr;
    for (int st = LT_STATE_U8; st <= LT_STATE_F32; ++st) {
        for (int dt = LT_F32; dt <= LT_BF16; ++dt) {   // one parameter dtype and one state kind per launch
            P.param_bf16 = (dt == LT_BF16) ? 1 : 0;
            P.s.precise_param = precise ? 1 : 0;
            int32_t i = 0;
            while (i < n) {
                pack_step(tensors, n, st == LT_STATE_F32 ? kAdamw32Item : block, &i, &P, true, dt, st);
                if (P.n == 0) continue;
                rc = st == LT_STATE_F32 ? launch_adamw32(P, dev->sm_count, (cudaStream_t)stream)
                                        : launch_step(P, block, dev->sm_count, (cudaStream_t)stream);
                if (rc != LT_OK) return rc;
            }
        }
    }
    return LT_OK;
}

int lt_hybrid8_step(const lt_tensor* tensors, int32_t n, int32_t block, const lt_hparams* hp,
                    const double* d_sqnorm, int32_t* d_status, lt_stream stream) {
    return step_impl(tensors, n, block, hp, nullptr, false, d_sqnorm, d_status, stream);
}

int lt_hybrid8_step_graph(const lt_tensor* tensors, int32_t n, int32_t block, const lt_hparams* hp,
                          const lt_step_state* d_state, const double* d_sqnorm, int32_t* d_status,
                          lt_stream stream) {
    return step_impl(tensors, n, block, hp, d_state, true, d_sqnorm, d_status, stream);
}

int lt_step_state_advance(lt_step_state* d_state, const lt_hparams* hp, const double* d_sqnorm, lt_stream stream) {
    if (!d_state || !hp) return LT_ERR_INVALID_ARG;
    if (!aligned(d_state, 8) || (d_sqnorm && !aligned(d_sqnorm, 8))) return LT_ERR_ALIGNMENT;
    if (!(hp->beta1 >= 0.0f && hp->beta1 < 1.0f) || !(hp->beta2 >= 0.0f && hp->beta2 < 1.0f) || !std::isfinite(hp->lr))
        return LT_ERR_INVALID_ARG;
    return launch_step_state_advance(d_state, hp->lr, hp->beta1, hp->beta2, d_sqnorm, (cudaStream_t)stream);
}

}  // extern "C"
