// Element arithmetic shared by the two update kernels (8-bit state: lt_step.cu, fp32 state: lt_adamw32.cu):
// the clip prologue (S2), the moment update and the parameter update (S4), in scalar and in packed
// two-element form. Not part of the C ABI.
//
// What is exact: m' and v' are formed with one IEEE round-to-nearest-even per written operation and no
// fused multiply-add, in the order  beta * m + (1 - beta) * g. The parameter update, whose result never
// feeds back into the state, uses the hardware's approximate sqrt and reciprocal unless PRECISE.
#pragma once

#include "lt_common.cuh"

namespace lt {

struct StepRegs {   // per-thread copies of the step scalars
    float c, beta1, beta2, omb1, omb2, step_size, isb2, decay, eps;
    float one;      // 1.0f known only at run time, see add2_rt
};

// S2: clip factor c = min(1, max_norm / (sqrt(S) + 1e-6)) from the device scalar, or skip the whole step
// on a non-finite S (bit 0 of the status word). Returns false when the step is skipped.
__device__ __forceinline__ bool load_step_regs(const StepParams& P, StepRegs& r) {
    r.c = 1.0f;
    if (P.sqnorm != nullptr) {
        const double S = *P.sqnorm;
        if (!isfinite(S)) {
            if (blockIdx.x == 0 && threadIdx.x == 0 && P.status != nullptr) atomicOr(P.status, 1);
            return false;
        }
        if (P.s.clip_on) r.c = (float)fmin(1.0, (double)P.s.max_norm / (sqrt(S) + 1e-6));
    }
    r.beta1 = P.s.beta1; r.beta2 = P.s.beta2; r.omb1 = P.s.omb1; r.omb2 = P.s.omb2;
    r.step_size = P.s.step_size; r.isb2 = P.s.inv_sqrt_bc2; r.decay = P.s.decay; r.eps = P.s.eps;
    r.one = P.s.one;
    if (P.dev_scalars != nullptr) { r.step_size = P.dev_scalars[0]; r.isb2 = P.dev_scalars[1]; }
    return true;
}

__device__ __forceinline__ float sqrt_approx(float x) { float r; asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float rcp_approx_ftz(float x) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }
__device__ __forceinline__ float rcp_approx(float x) { float r; asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// Three-input minimum / maximum (one instruction on sm_100); like fminf / fmaxf, a NaN operand is ignored.
__device__ __forceinline__ float fmin3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// The parameter update exactly as defined (IEEE sqrt and divide, one rounding per operation).
__device__ __forceinline__ float param_exact(const StepRegs& r, float p, float mm, float vv) {
    const float den = __fadd_rn(__fmul_rn(__fsqrt_rn(vv), r.isb2), r.eps);
    return __fsub_rn(__fmul_rn(p, r.decay), __fmul_rn(r.step_size, __fdiv_rn(mm, den)));
}

// Error of the approximate parameter path against the defined one. sqrt.approx and rcp.approx are within
// 2^-23 relative, the two roundings around them add 2^-24 each, so the approximate quotient is within
// 3 * 2^-23 of m' / (sqrt(v') / sqrt(bc2) + eps); the defined path's own four roundings allow 2^-22 and the
// product with the step size 2^-24. With u = step_size * m' / den (the update) and p' the new parameter,
//     |p'_approx - p'_defined|  <=  5.5 * 2^-23 |u| + 2^-23 |p'|  =  6.6e-7 |u| + 1.2e-7 |p'|.
// fp32 parameters: that is below 1e-5 * max(|p'|, |u|) for every input, which is the tolerance fp32
// parameters are held to (relative to the larger of the result and the update that formed it).
// bf16 parameters: a bf16 ulp is at least 2^-8 |p'|; two values less than half of that apart round to
// bf16 numbers at most one ulp apart, so the rounded results agree within one ulp as long as
// 6.6e-7 |u| < 2^-9 |p'|, i.e. |u| < 2950 |p'|. cancel_risk(pn, pd) < 0 flags |p'| < 2^-11 |p * decay|;
// an element that is not flagged has |u| <= |p * decay| + |p'| <= 2049 |p'|, inside that bound. Flagged
// elements (about 2 in 10^7) take param_exact.
__device__ __forceinline__ float cancel_risk(float pn, float pd) { return __fmaf_rn(fabsf(pn), 2048.0f, -fabsf(pd)); }

// Packed two-element fp32 instructions of sm_100 (mul / fma on a 64-bit register pair, each half rounded to
// nearest even like the scalar instruction). Inline PTX with explicit .rn. One hazard, measured on this
// toolchain (CUDA 12.9): the assembler contracts a packed multiply that feeds a packed add into one packed
// FMA -- with -fmad=false, with explicit .rn on both, and also when the add is written as fma(x, 1.0, y)
// with a literal one -- which changes m' and v' (single rounding of beta * m + t instead of the defined
// two). The two-rounding sum is therefore written add2_rt(x, y, one) = fma(x, one, y) with `one` a RUN-TIME
// 1.0 from the kernel parameters: x * 1 + y is the exact sum rounded once, and the assembler cannot fold a
// multiplier it does not know.
__device__ __forceinline__ float2 dup2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\tfma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 add2_rt(float2 x, float2 y, float2 one) { return fma2(x, one, y); }

// S4, moments of one element / of a pair: m' = beta1 m + (1 - beta1) c g, v' = beta2 v + (1 - beta2) (c g)^2.
__device__ __forceinline__ void moments_one(const StepRegs& r, float g, float m, float v, float& mm, float& vv) {
    const float gc = __fmul_rn(g, r.c);
    mm = __fadd_rn(__fmul_rn(r.beta1, m), __fmul_rn(r.omb1, gc));
    vv = __fadd_rn(__fmul_rn(r.beta2, v), __fmul_rn(r.omb2, __fmul_rn(gc, gc)));
}
__device__ __forceinline__ void moments_pair(const StepRegs& r, float2 g, float2 m, float2 v, float2& mm, float2& vv) {
    const float2 gc = mul2(g, dup2(r.c));
    mm = add2_rt(mul2(dup2(r.beta1), m), mul2(dup2(r.omb1), gc), dup2(r.one));
    vv = add2_rt(mul2(dup2(r.beta2), v), mul2(dup2(r.omb2), mul2(gc, gc)), dup2(r.one));
}

// S4, new parameter of one element / of a pair; leaves p * decay in pd (the cancellation guard needs it).
// p * decay is rounded first, as the definition does: a single-rounding FMA of p * decay - update is the
// more accurate arithmetic but drifts away from the definition by ~6e-8 relative per step (with decay this
// close to 1 the rounded product is systematically p itself or one ulp below it).
template <bool PRECISE>
__device__ __forceinline__ float param_one(const StepRegs& r, float p, float mm, float vv, float& pd) {
    pd = __fmul_rn(p, r.decay);
    if (PRECISE) return param_exact(r, p, mm, vv);
    const float den = __fmaf_rn(sqrt_approx(vv), r.isb2, r.eps);
    const float q = __fmul_rn(mm, rcp_approx_ftz(den));
    return __fmaf_rn(-r.step_size, q, pd);
}
template <bool PRECISE>
__device__ __forceinline__ float2 param_pair(const StepRegs& r, float2 p, float2 mm, float2 vv, float2& pd) {
    pd = mul2(p, dup2(r.decay));
    if (PRECISE) return make_float2(param_exact(r, p.x, mm.x, vv.x), param_exact(r, p.y, mm.y, vv.y));
    const float2 sq = make_float2(sqrt_approx(vv.x), sqrt_approx(vv.y));   // no packed sqrt / reciprocal
    const float2 den = fma2(sq, dup2(r.isb2), dup2(r.eps));
    const float2 rc = make_float2(rcp_approx_ftz(den.x), rcp_approx_ftz(den.y));
    const float2 q = mul2(mm, rc);
    return fma2(dup2(-r.step_size), q, pd);
}

}  // namespace lt
