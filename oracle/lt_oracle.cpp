// lt_oracle.cpp -- CPU oracle for the fused global-norm clip + block-wise 8-bit AdamW step.
//
// TEST INFRASTRUCTURE, NOT PRODUCT. Only the test suite, the smoke check and the benchmark's
// cpu_baseline / reference legs may build, load or call this file. It shares no code, header,
// table or constant generator with the CUDA library; the CUDA library never calls it.
//
// What it follows. The paper (Sec. 3.5, "Hybrid 8-bit operator") describes the operator in words:
// a slice of the Adam moments is held as 8-bit codes with one scale per block, the update
// decodes them, takes an AdamW step and encodes them again; the clip takes a norm per tensor,
// combines these into one global norm and multiplies every gradient by one factor; a step whose
// gradients are not finite is left out (training-configuration table, safety-checks row);
// hyper-parameters come from the same table
// (beta1 0.9, beta2 0.999, eps 1e-8, lr 1e-5, weight decay 0.01, max grad norm 1.0); block size
// 4096 comes from the variant-configuration table. The paper prints no formulas for the
// quantization map, tie handling, epsilon placement or rounding, so this file takes one written
// reading of each (listed below, O-1 .. O-8) and applies it step by step, single-threaded, with no
// blocking, fusion or reordering.
//
// Arithmetic. The norm is accumulated sequentially in fp64. Every per-element operation is IEEE
// fp32, round-to-nearest-even, one rounding per written operation, no fused multiply-add: build
// with -ffp-contract=off (the build script does). Per-step scalars are formed in fp64 and rounded
// once to fp32.
//
// Pins (tests that check this file against something other than itself) are in
// tests/test_oracle_pins.py. Parity status: every function below is pinned by a closed form, an
// invariant, a library routine or brute force, EXCEPT the numeric values of a multi-step
// trajectory with quantization on -- the paper prints no worked example, so that is
// "parity unpinned" beyond its per-step invariants (scale == block max, error bound per code gap,
// brute-force nearest code) and its agreement with the unquantized fp32 trajectory within that
// bound.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <algorithm>
#include <vector>

namespace {

// ---- O-1: code tables ------------------------------------------------------------------------
// Seven decades e = 0..6 with scale d_e = 10^(e-6) (decimal literals). Decade e of the signed map
// has 2^e cells, of the unsigned map 2^(e+1) cells; a cell's value is the mid-point of a uniform
// grid on [0.1, 1] times d_e, formed in double and rounded once to fp32. The signed map takes both
// signs (2 * 127 values) plus 0.0 and +1.0; the unsigned map takes 254 values plus 0.0 and +1.0.
// Sorted ascending each has exactly 256 entries. There is no -1.0.
const double kDecade[7] = {1e-6, 1e-5, 1e-4, 1e-3, 1e-2, 1e-1, 1e0};

void build_table(bool is_signed, float out[256]) {
    std::vector<float> v;
    for (int e = 0; e < 7; ++e) {
        const int cells = is_signed ? (1 << e) : (1 << (e + 1));
        for (int j = 0; j < cells; ++j) {
            const double mag = kDecade[e] * (0.1 + 0.9 * ((double)j + 0.5) / (double)cells);
            const float f = (float)mag;
            v.push_back(f);
            if (is_signed) v.push_back(-f);
        }
    }
    v.push_back(0.0f);
    v.push_back(1.0f);
    std::sort(v.begin(), v.end());
    for (int i = 0; i < 256; ++i) out[i] = (i < (int)v.size()) ? v[i] : 0.0f;
}

struct Tables {
    float qs[256];
    float qu[256];
    Tables() { build_table(true, qs); build_table(false, qu); }
};
const Tables& tables() { static Tables t; return t; }

// ---- O-2: quantizer --------------------------------------------------------------------------
// nearest(T, x): index minimising |T[i] - x| evaluated exactly; ties go to the lower index.
// The brute-force form is the definition. The search form counts the mid-points strictly below x;
// a mid-point of two fp32 numbers is exact in double, so both forms agree on every input.
int nearest_brute(const float* T, float x) {
    int best = 0;
    double bestd = std::fabs((double)T[0] - (double)x);
    for (int i = 1; i < 256; ++i) {
        const double d = std::fabs((double)T[i] - (double)x);
        if (d < bestd) { bestd = d; best = i; }
    }
    return best;
}

int nearest_search(const float* T, float x) {
    // smallest i such that x <= mid(i), mid(i) = (T[i] + T[i+1]) / 2, i in 0..254; else 255
    int lo = 0, hi = 255;
    while (lo < hi) {
        const int k = (lo + hi) >> 1;
        const double mid = ((double)T[k] + (double)T[k + 1]) * 0.5;
        if ((double)x > mid) lo = k + 1; else hi = k;
    }
    return lo;
}

// ---- element types ----------------------------------------------------------------------------
enum { DT_F32 = 0, DT_BF16 = 1 };

inline float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f; std::memcpy(&f, &u, 4); return f;
}
// round-to-nearest-even; NaN stays NaN (quiet)
inline uint16_t f32_to_bf16(float f) {
    uint32_t u; std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    const uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}
inline float load_elem(const void* p, int dt, int64_t i) {
    return dt == DT_F32 ? ((const float*)p)[i] : bf16_to_f32(((const uint16_t*)p)[i]);
}
inline void store_elem(void* p, int dt, int64_t i, float x) {
    if (dt == DT_F32) ((float*)p)[i] = x; else ((uint16_t*)p)[i] = f32_to_bf16(x);
}

}  // namespace

extern "C" {

// One parameter tensor with its gradient and 8-bit state. Host pointers.
struct lto_tensor {
    void* param;          // [numel] param_dtype
    const void* grad;     // [numel] grad_dtype, never written
    uint8_t* m_code;      // [numel]
    uint8_t* v_code;      // [numel]
    float* m_absmax;      // [ceil(numel / block)]
    float* v_absmax;      // [ceil(numel / block)]
    int64_t numel;
    int32_t param_dtype;  // 0 = fp32, 1 = bf16
    int32_t grad_dtype;
    int32_t state_dtype;  // 0 = 8-bit codes + block scales; 1 = plain fp32 moments: m_code / v_code are
                          //     float[numel] and the scale arrays are unused (the paper's "hybrid" split,
                          //     Sec. 3.5: most parameters keep ordinary Adam states, a 2 % slice is 8-bit)
    int32_t reserved;
};

struct lto_hparams {
    float lr, beta1, beta2, eps, weight_decay, max_norm;
    int64_t step;  // 1-based
};

// O-1
void lto_code_table(int is_signed, float out[256]) {
    std::memcpy(out, is_signed ? tables().qs : tables().qu, 256 * sizeof(float));
}

// O-2
int lto_nearest(int is_signed, float x) {
    return nearest_search(is_signed ? tables().qs : tables().qu, x);
}
int lto_nearest_brute(int is_signed, float x) {
    return nearest_brute(is_signed ? tables().qs : tables().qu, x);
}

// State footprint: one byte per element per moment, one fp32 scale per block per moment.
void lto_state_bytes(int64_t numel, int32_t block, int64_t* code_bytes, int64_t* absmax_bytes) {
    *code_bytes = numel;
    *absmax_bytes = 4 * ((numel + block - 1) / block);
}

// ---- O-3: norm and clip factor ---------------------------------------------------------------
// S += sum of squares, added one element at a time in index order, in fp64.
double lto_sqnorm_accumulate(const void* grad, int32_t grad_dtype, int64_t numel, double S) {
    for (int64_t i = 0; i < numel; ++i) {
        const double g = (double)load_elem(grad, grad_dtype, i);
        S += g * g;
    }
    return S;
}

double lto_grad_sqnorm_multi(const lto_tensor* t, int32_t n, double S) {
    for (int32_t k = 0; k < n; ++k) S = lto_sqnorm_accumulate(t[k].grad, t[k].grad_dtype, t[k].numel, S);
    return S;
}

// c = min(1, max_norm / (sqrt(S) + 1e-6)) formed in fp64 and rounded to fp32. max_norm <= 0 or
// +inf disables clipping (c = 1). *nonfinite is set when S is NaN or Inf and clipping is enabled,
// or when S is NaN/Inf at all (a non-finite gradient): the step must then be skipped.
float lto_clip_factor(double S, float max_norm, int32_t* nonfinite) {
    *nonfinite = std::isfinite(S) ? 0 : 1;
    if (*nonfinite) return 0.0f;
    if (!(max_norm > 0.0f) || std::isinf(max_norm)) return 1.0f;
    const double gnorm = std::sqrt(S);
    const double c = std::min(1.0, (double)max_norm / (gnorm + 1e-6));
    return (float)c;
}

// ---- O-4: per-step scalars -------------------------------------------------------------------
struct lto_scalars { float step_size, inv_sqrt_bc2, decay, omb1, omb2, beta1, beta2, eps; };

void lto_step_scalars(const lto_hparams* hp, lto_scalars* s) {
    const double b1 = (double)hp->beta1, b2 = (double)hp->beta2;
    const double t = (double)hp->step;
    const double bc1 = 1.0 - std::pow(b1, t);
    const double bc2 = 1.0 - std::pow(b2, t);
    s->step_size = (float)((double)hp->lr / bc1);
    s->inv_sqrt_bc2 = (float)(1.0 / std::sqrt(bc2));
    s->decay = (float)(1.0 - (double)hp->lr * (double)hp->weight_decay);
    s->omb1 = (float)(1.0 - b1);
    s->omb2 = (float)(1.0 - b2);
    s->beta1 = hp->beta1;
    s->beta2 = hp->beta2;
    s->eps = hp->eps;
}

// ---- O-8: state init --------------------------------------------------------------------------
// Value-zero state: the signed code of 0.0 is 127, the unsigned code of 0.0 is 0, scales 0.
void lto_state_init(const lto_tensor* t, int32_t n, int32_t block) {
    for (int32_t k = 0; k < n; ++k) {
        const int64_t nb = (t[k].numel + block - 1) / block;
        if (t[k].state_dtype == 1) {
            float* m = (float*)t[k].m_code; float* v = (float*)t[k].v_code;
            for (int64_t i = 0; i < t[k].numel; ++i) { m[i] = 0.0f; v[i] = 0.0f; }
            continue;
        }
        for (int64_t i = 0; i < t[k].numel; ++i) { t[k].m_code[i] = 127; t[k].v_code[i] = 0; }
        for (int64_t b = 0; b < nb; ++b) { t[k].m_absmax[b] = 0.0f; t[k].v_absmax[b] = 0.0f; }
    }
}

// ---- O-5 / O-6: one tensor, all blocks, given the clip factor c --------------------------------
// use_brute != 0 swaps the nearest-code search for the definitional argmin (tests only).
void lto_step_tensor(const lto_tensor* tt, int32_t block, const lto_scalars* s, float c, int32_t use_brute) {
    const float* QS = tables().qs;
    const float* QU = tables().qu;
    const int64_t N = tt->numel;
    std::vector<float> m2(block), v2(block);
    for (int64_t b0 = 0, b = 0; b0 < N; b0 += block, ++b) {
        const int64_t len = std::min<int64_t>(block, N - b0);
        const float am_old = tt->m_absmax[b];
        const float av_old = tt->v_absmax[b];
        float am = 0.0f, av = 0.0f;
        for (int64_t j = 0; j < len; ++j) {
            const int64_t i = b0 + j;
            // O-5
            const float g = load_elem(tt->grad, tt->grad_dtype, i) * c;
            const float m = QS[tt->m_code[i]] * am_old;
            const float v = QU[tt->v_code[i]] * av_old;
            const float t1 = s->beta1 * m;
            const float t2 = s->omb1 * g;
            const float mm = t1 + t2;
            const float gg = g * g;
            const float t3 = s->beta2 * v;
            const float t4 = s->omb2 * gg;
            const float vv = t3 + t4;
            const float sq = std::sqrt(vv);
            const float t5 = sq * s->inv_sqrt_bc2;
            const float den = t5 + s->eps;
            const float q = mm / den;
            const float p = load_elem(tt->param, tt->param_dtype, i);
            const float t6 = p * s->decay;
            const float t7 = s->step_size * q;
            const float p2 = t6 - t7;
            store_elem(tt->param, tt->param_dtype, i, p2);
            m2[j] = mm;
            v2[j] = vv;
            am = std::max(am, std::fabs(mm));
            av = std::max(av, vv);
        }
        // O-6
        tt->m_absmax[b] = am;
        tt->v_absmax[b] = av;
        for (int64_t j = 0; j < len; ++j) {
            const int64_t i = b0 + j;
            int mc = 127, vc = 0;
            if (am > 0.0f) {
                const float x = m2[j] / am;
                mc = use_brute ? nearest_brute(QS, x) : nearest_search(QS, x);
            }
            if (av > 0.0f) {
                const float x = v2[j] / av;
                vc = use_brute ? nearest_brute(QU, x) : nearest_search(QU, x);
            }
            tt->m_code[i] = (uint8_t)mc;
            tt->v_code[i] = (uint8_t)vc;
        }
    }
}

// O-7 applied to a tensor whose moments are plain fp32 arrays (state_dtype 1): the same element
// arithmetic as O-5 without the table lines, and no O-6.
void lto_step_tensor_fp32state(const lto_tensor* tt, const lto_scalars* s, float c) {
    float* m = (float*)tt->m_code;
    float* v = (float*)tt->v_code;
    for (int64_t i = 0; i < tt->numel; ++i) {
        const float g = load_elem(tt->grad, tt->grad_dtype, i) * c;
        const float t1 = s->beta1 * m[i];
        const float t2 = s->omb1 * g;
        const float mm = t1 + t2;
        const float gg = g * g;
        const float t3 = s->beta2 * v[i];
        const float t4 = s->omb2 * gg;
        const float vv = t3 + t4;
        const float sq = std::sqrt(vv);
        const float t5 = sq * s->inv_sqrt_bc2;
        const float den = t5 + s->eps;
        const float q = mm / den;
        const float p = load_elem(tt->param, tt->param_dtype, i);
        const float t6 = p * s->decay;
        const float t7 = s->step_size * q;
        store_elem(tt->param, tt->param_dtype, i, t6 - t7);
        m[i] = mm;
        v[i] = vv;
    }
}

// Whole step over a tensor list given the total squared norm S of ALL gradients of this optimizer
// step (the list may be one chunk of them). Returns 0; *status bit 0 is set (and nothing else is
// touched) when S is not finite.
int32_t lto_hybrid8_step(const lto_tensor* t, int32_t n, int32_t block, const lto_hparams* hp,
                         double S, int32_t* status, int32_t use_brute) {
    int32_t nonfinite = 0;
    const float c = lto_clip_factor(S, hp->max_norm, &nonfinite);
    if (nonfinite) { *status |= 1; return 0; }
    lto_scalars s;
    lto_step_scalars(hp, &s);
    for (int32_t k = 0; k < n; ++k) {
        if (t[k].state_dtype == 1) lto_step_tensor_fp32state(&t[k], &s, c);
        else lto_step_tensor(&t[k], block, &s, c, use_brute);
    }
    return 0;
}

// ---- O-7: the same update with quantization disabled (fp32 moments) --------------------------
// Used only to pin the Adam arithmetic against closed forms and a library AdamW.
void lto_step_fp32state(float* param, const float* grad, float* m, float* v, int64_t numel,
                        const lto_hparams* hp, float c) {
    lto_scalars s;
    lto_step_scalars(hp, &s);
    for (int64_t i = 0; i < numel; ++i) {
        const float g = grad[i] * c;
        const float t1 = s.beta1 * m[i];
        const float t2 = s.omb1 * g;
        const float mm = t1 + t2;
        const float gg = g * g;
        const float t3 = s.beta2 * v[i];
        const float t4 = s.omb2 * gg;
        const float vv = t3 + t4;
        const float sq = std::sqrt(vv);
        const float t5 = sq * s.inv_sqrt_bc2;
        const float den = t5 + s.eps;
        const float q = mm / den;
        const float t6 = param[i] * s.decay;
        const float t7 = s.step_size * q;
        param[i] = t6 - t7;
        m[i] = mm;
        v[i] = vv;
    }
}

// Dequantize a code array (tests: error-bound and invariance checks).
void lto_dequant(int32_t is_signed, const uint8_t* code, const float* absmax, int64_t numel,
                 int32_t block, float* out) {
    const float* T = is_signed ? tables().qs : tables().qu;
    for (int64_t i = 0; i < numel; ++i) out[i] = T[code[i]] * absmax[i / block];
}

}  // extern "C"
