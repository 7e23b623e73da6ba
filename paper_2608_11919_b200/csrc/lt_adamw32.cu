// The same clipped AdamW update for tensors whose moments are plain fp32 arrays (the larger part of
// the paper's hybrid split, Sec. 3.5): read p, g, m, v, write p, m, v -- 26 bytes per parameter with
// fp32 parameters and bf16 gradients, a pure HBM stream with no tables and no block exchange.
//
// Work item = 8192 consecutive elements of one tensor (items restart at every tensor); 256-thread CTAs
// walk the items in a grid-stride loop, thread `tid` owning the 4-element groups (k * 256 + tid), k < 8,
// so every warp-wide access is one contiguous run and all 32 loads of a thread (24 of them 16 bytes) are in flight
// together: measured 6 % faster than two groups per thread, the kernel being bound by memory latency times
// bytes in flight (four groups +1 %, sixteen -3 % against eight).
// Moments are formed exactly as written (IEEE fp32, one rounding per operation, no fused
// multiply-add), so the state matches a plain evaluation bit for bit; the parameter update uses the
// approximate sqrt/reciprocal unless eps is tiny, as in the 8-bit kernel.
#include <cuda_bf16.h>

#include <atomic>

#include "lt_common.cuh"
#include "lt_update.cuh"

namespace lt {

namespace {

#ifndef LT_A32_NT
#define LT_A32_NT 256
#endif
#ifndef LT_A32_MINB
#define LT_A32_MINB 1
#endif
constexpr int kNT = LT_A32_NT;
constexpr int kK = kAdamw32Item / (4 * kNT);

// Two elements: moments in place, new parameters returned. GUARD (bf16 parameters on the approximate path):
// an element whose result cancels below 2^-11 of p * decay takes the exact formula (cancel_risk, lt_update.cuh).
template <bool PRECISE, bool GUARD>
__device__ __forceinline__ float2 update2(const StepRegs& r, float2 p, float2 g, float2& m, float2& v) {
    float2 pd;
    moments_pair(r, g, m, v, m, v);
    float2 pn = param_pair<PRECISE>(r, p, m, v, pd);
    if (GUARD && fminf(cancel_risk(pn.x, pd.x), cancel_risk(pn.y, pd.y)) < 0.0f) {
        pn.x = param_exact(r, p.x, m.x, v.x);
        pn.y = param_exact(r, p.y, m.y, v.y);
    }
    return pn;
}
template <bool PRECISE, bool GUARD>
__device__ __forceinline__ float update(const StepRegs& r, float p, float g, float& m, float& v) {
    float pd;
    moments_one(r, g, m, v, m, v);
    const float pn = param_one<PRECISE>(r, p, m, v, pd);
    if (GUARD && cancel_risk(pn, pd) < 0.0f) return param_exact(r, p, m, v);
    return pn;
}

template <bool PRECISE, bool P_BF16>
__global__ void __launch_bounds__(kNT, LT_A32_MINB) adamw32_kernel(const __grid_constant__ StepParams P) {
    const int tid = threadIdx.x;
    StepRegs r;
    if (!load_step_regs(P, r)) return;

    int t = 0, begin = 0;
    for (int w = blockIdx.x; w < P.total_blocks; w += gridDim.x) {
        while (w >= P.t[t].blk_end) { begin = P.t[t].blk_end; ++t; }
        const StepDesc& d = P.t[t];
        const int64_t e_base = (int64_t)(w - begin) * kAdamw32Item;
        const int64_t rem = d.numel - e_base;
        const int len = rem < kAdamw32Item ? (int)rem : kAdamw32Item;
        const bool g_f32 = (d.flags & kFlagGradF32) != 0;
        char* pp = (char*)d.p + e_base * (P_BF16 ? 2 : 4);
        const char* gp = (const char*)d.g + e_base * (g_f32 ? 4 : 2);
        float* mp = (float*)d.mc + e_base;
        float* vp = (float*)d.vc + e_base;
        if ((d.flags & kFlagVecOk) != 0 && !g_f32 && len == kAdamw32Item) {
            uint4 pr[kK]; uint2 gr[kK]; float4 mr[kK], vr[kK];
#pragma unroll
            for (int k = 0; k < kK; ++k) {
                const int e0 = (k * kNT + tid) * 4;
                if (P_BF16) { const uint2 q = *(const uint2*)(pp + e0 * 2); pr[k].x = q.x; pr[k].y = q.y; }
                else pr[k] = *(const uint4*)(pp + e0 * 4);
                gr[k] = *(const uint2*)(gp + e0 * 2);
                mr[k] = *(const float4*)(mp + e0);
                vr[k] = *(const float4*)(vp + e0);
            }
#pragma unroll
            for (int k = 0; k < kK; ++k) {
                const int e0 = (k * kNT + tid) * 4;
                float p[4], g[4], pn[4];
                if (P_BF16) {
                    p[0] = __uint_as_float(pr[k].x << 16); p[1] = __uint_as_float(pr[k].x & 0xffff0000u);
                    p[2] = __uint_as_float(pr[k].y << 16); p[3] = __uint_as_float(pr[k].y & 0xffff0000u);
                } else {
                    p[0] = __uint_as_float(pr[k].x); p[1] = __uint_as_float(pr[k].y);
                    p[2] = __uint_as_float(pr[k].z); p[3] = __uint_as_float(pr[k].w);
                }
                g[0] = __uint_as_float(gr[k].x << 16); g[1] = __uint_as_float(gr[k].x & 0xffff0000u);
                g[2] = __uint_as_float(gr[k].y << 16); g[3] = __uint_as_float(gr[k].y & 0xffff0000u);
                float2 m01 = make_float2(mr[k].x, mr[k].y), m23 = make_float2(mr[k].z, mr[k].w);
                float2 v01 = make_float2(vr[k].x, vr[k].y), v23 = make_float2(vr[k].z, vr[k].w);
                const float2 n01 = update2<PRECISE, P_BF16 && !PRECISE>(r, make_float2(p[0], p[1]), make_float2(g[0], g[1]), m01, v01);
                const float2 n23 = update2<PRECISE, P_BF16 && !PRECISE>(r, make_float2(p[2], p[3]), make_float2(g[2], g[3]), m23, v23);
                pn[0] = n01.x; pn[1] = n01.y; pn[2] = n23.x; pn[3] = n23.y;
                mr[k] = make_float4(m01.x, m01.y, m23.x, m23.y);
                vr[k] = make_float4(v01.x, v01.y, v23.x, v23.y);
                if (P_BF16) {
                    const __nv_bfloat162 lo = __floats2bfloat162_rn(pn[0], pn[1]);
                    const __nv_bfloat162 hi = __floats2bfloat162_rn(pn[2], pn[3]);
                    uint2 q;
                    q.x = *reinterpret_cast<const uint32_t*>(&lo);
                    q.y = *reinterpret_cast<const uint32_t*>(&hi);
                    *(uint2*)(pp + e0 * 2) = q;
                } else {
                    *(float4*)(pp + e0 * 4) = make_float4(pn[0], pn[1], pn[2], pn[3]);
                }
                *(float4*)(mp + e0) = mr[k];
                *(float4*)(vp + e0) = vr[k];
            }
        } else {
            for (int e = tid; e < len; e += kNT) {
                const float p = P_BF16 ? __uint_as_float((uint32_t)*(const unsigned short*)(pp + e * 2) << 16)
                                       : *(const float*)(pp + e * 4);
                const float g = g_f32 ? *(const float*)(gp + e * 4)
                                      : __uint_as_float((uint32_t)*(const unsigned short*)(gp + e * 2) << 16);
                float m = mp[e], v = vp[e];
                const float pn = update<PRECISE, P_BF16 && !PRECISE>(r, p, g, m, v);
                if (P_BF16) *(unsigned short*)(pp + e * 2) = __bfloat16_as_ushort(__float2bfloat16_rn(pn));
                else *(float*)(pp + e * 4) = pn;
                mp[e] = m;
                vp[e] = v;
            }
        }
    }
}

template <bool PRECISE, bool P_BF16>
int launch(const StepParams& p, int sm_count, cudaStream_t s) {
    static std::atomic<int> grid_of_device[kMaxDevices];   // racing host threads store the same value
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return LT_ERR_CUDA; }
    int full_grid = grid_of_device[dev].load(std::memory_order_acquire);
    if (full_grid == 0) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, adamw32_kernel<PRECISE, P_BF16>, kNT, 0) != cudaSuccess ||
            per_sm < 1) { cudaGetLastError(); return LT_ERR_CUDA; }
        full_grid = per_sm * sm_count;
        grid_of_device[dev].store(full_grid, std::memory_order_release);
    }
    const int grid = p.total_blocks < full_grid ? p.total_blocks : full_grid;
    adamw32_kernel<PRECISE, P_BF16><<<grid, kNT, 0, s>>>(p);
    return cudaGetLastError() == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

}  // namespace

__global__ void step_state_advance_kernel(lt_step_state* st, float lr, float beta1, float beta2, const double* sqnorm) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (sqnorm != nullptr && !isfinite(*sqnorm)) return;   // the coming step is skipped: it does not count
    const int64_t t = st->step + 1;
    const double bc1 = 1.0 - pow((double)beta1, (double)t);
    const double bc2 = 1.0 - pow((double)beta2, (double)t);
    st->step = t;
    st->step_size = (float)((double)lr / bc1);
    st->inv_sqrt_bc2 = (float)(1.0 / sqrt(bc2));
}

int launch_step_state_advance(lt_step_state* d_state, float lr, float beta1, float beta2, const double* d_sqnorm,
                              cudaStream_t s) {
    step_state_advance_kernel<<<1, 32, 0, s>>>(d_state, lr, beta1, beta2, d_sqnorm);
    return cudaGetLastError() == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

int launch_adamw32(const StepParams& p, int sm_count, cudaStream_t s) {
    if (p.param_bf16) return p.s.precise_param ? launch<true, true>(p, sm_count, s) : launch<false, true>(p, sm_count, s);
    return p.s.precise_param ? launch<true, false>(p, sm_count, s) : launch<false, false>(p, sm_count, s);
}

}  // namespace lt
