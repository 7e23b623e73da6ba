// S1: multi-tensor squared L2 norm of the gradients, finished on the device.
//
// Bound: HBM read bandwidth, 2 bytes per bf16 gradient element, read once. A work item is 128 KiB of
// one tensor's 16-byte-aligned span; a CTA of 1024 threads, one per SM, issues eight independent 16-byte
// streaming loads per thread per item and walks the items in a grid-stride loop, so each SM keeps 128 KiB of
// loads in flight (the kernel is bound by memory latency times bytes in flight: half as much is 9 % slower).
//
// Accuracy and reproducibility. Each thread converts its bf16 values to fp64 (exact), and adds their
// exact squares to an fp64 accumulator with one fused multiply-add each, so only the running fp64
// sum rounds. Per-CTA fp64 partials go to the workspace; the last CTA to arrive
// (an atomic ticket, not a wait) adds them in index order and accumulates the launch total into
// *out. Nothing depends on arrival order, so the result is bit-reproducible.
#include <mutex>

#include "lt_common.cuh"

namespace lt {

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// eight squares of one vector of bf16 added to an fp64 accumulator. A bf16 value converts to fp64
// exactly and its square has 16 significant bits, so every product is exact and only the running
// sum rounds (in fp64). (Summing the squares in fp32 first is biased: the addends have few
// significant bits, ties are frequent, and ties-to-even then always rounds the sum down.)
__device__ __forceinline__ double sq8_bf16(const uint4& v, double acc) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const double lo = (double)bf16_lo(w[i]), hi = (double)bf16_hi(w[i]);
        acc = fma(lo, lo, acc);
        acc = fma(hi, hi, acc);
    }
    return acc;
}

__device__ __forceinline__ double sq4_f32(const uint4& v) {
    const double a = (double)__uint_as_float(v.x), b = (double)__uint_as_float(v.y);
    const double c = (double)__uint_as_float(v.z), d = (double)__uint_as_float(v.w);
    return (a * a + b * b) + (c * c + d * d);
}

// elements of a vector that straddles the tensor's first or last byte, read one by one
__device__ __forceinline__ double sq_partial(const char* base, int64_t off, int64_t lo, int64_t hi, bool f32) {
    double acc = 0.0;
    if (f32) {
        for (int j = 0; j < 4; ++j) {
            const int64_t b = off + 4 * j;
            if (b >= lo && b + 4 <= hi) { const double x = (double)*(const float*)(base + b); acc += x * x; }
        }
    } else {
        for (int j = 0; j < 8; ++j) {
            const int64_t b = off + 2 * j;
            if (b >= lo && b + 2 <= hi) {
                const double x = (double)__uint_as_float((uint32_t)*(const unsigned short*)(base + b) << 16);
                acc += x * x;
            }
        }
    }
    return acc;
}

__global__ void __launch_bounds__(kNormThreads, kNormCtasPerSm) sqnorm_kernel(const __grid_constant__ NormParams P) {
    __shared__ double s_warp[kNormThreads / 32];
    __shared__ bool s_last;
    const int tid = threadIdx.x;
    double acc = 0.0;
    int t = 0;
    int item_begin = 0;
    for (int w = blockIdx.x; w < P.total_items; w += gridDim.x) {
        while (w >= P.t[t].item_end) { item_begin = P.t[t].item_end; ++t; }
        const NormDesc& d = P.t[t];
        const char* base = (const char*)d.base16;
        const int64_t lo = d.lead_f32 & 0xff;
        const bool f32 = (d.lead_f32 >> 8) != 0;
        const int64_t hi = d.span_bytes;
        const int64_t item_off = (int64_t)(w - item_begin) * kNormItemBytes;
        if (item_off >= lo && item_off + kNormItemBytes <= hi) {
            uint4 v[kNormVecPerThread];
#pragma unroll
            for (int k = 0; k < kNormVecPerThread; ++k)
                v[k] = ld_stream16(base + item_off + (int64_t)(k * kNormThreads + tid) * 16);
            if (!f32) {
#pragma unroll
                for (int k = 0; k < kNormVecPerThread; ++k) acc = sq8_bf16(v[k], acc);
            } else {
#pragma unroll
                for (int k = 0; k < kNormVecPerThread; ++k) acc += sq4_f32(v[k]);
            }
        } else {
#pragma unroll
            for (int k = 0; k < kNormVecPerThread; ++k) {
                const int64_t off = item_off + (int64_t)(k * kNormThreads + tid) * 16;
                if (off >= lo && off + 16 <= hi) {
                    const uint4 v = ld_stream16(base + off);
                    acc = f32 ? acc + sq4_f32(v) : sq8_bf16(v, acc);
                } else if (off + 16 > lo && off < hi) {
                    acc += sq_partial(base, off, lo, hi, f32);
                }
            }
        }
    }
    // CTA reduction in a fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) s_warp[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double s = 0.0;
        for (int i = 0; i < kNormThreads / 32; ++i) s += s_warp[i];
        P.partials[blockIdx.x] = s;
        __threadfence();
        const unsigned int ticket = atomicAdd(P.ticket, 1u);
        s_last = (ticket == gridDim.x - 1);
    }
    __syncthreads();
    if (s_last && tid < 32) {
        __threadfence();
        // lanes take partials i = lane, lane + 32, ... in order, then a fixed shuffle tree
        double s = 0.0;
        for (int i = tid; i < (int)gridDim.x; i += 32) s += __ldcg(&P.partials[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (tid == 0) {
            *P.out = *P.out + s;
            *P.ticket = 0u;
        }
    }
}

int validate_grads(const lt_tensor* t, int32_t n, int* live) {
    if (n < 0 || (n > 0 && t == nullptr)) return LT_ERR_INVALID_ARG;
    int cnt = 0;
    for (int32_t i = 0; i < n; ++i) {
        const lt_tensor& x = t[i];
        if (x.numel < 0) return LT_ERR_INVALID_ARG;
        if (x.numel > ((int64_t)1 << 38)) return LT_ERR_UNSUPPORTED;   // keeps per-launch item counts in int32
        if (x.numel == 0) continue;
        if ((x.grad_dtype != LT_F32 && x.grad_dtype != LT_BF16) || x.grad == nullptr) return LT_ERR_INVALID_ARG;
        if (((uintptr_t)x.grad % (x.grad_dtype == LT_F32 ? 4 : 2)) != 0) return LT_ERR_ALIGNMENT;
        ++cnt;
    }
    if (live) *live = cnt;
    return LT_OK;
}

void pack_norm(const lt_tensor* t, int32_t n, int32_t* i, NormParams* P) {
    int cnt = 0;
    int64_t items = 0;
    while (*i < n && cnt < kCap) {
        const lt_tensor& x = t[*i];
        if (x.numel == 0) { ++*i; continue; }
        // the kernel reads whole 16-byte vectors: the span starts at the address rounded down to 16 bytes
        const uintptr_t a = (uintptr_t)x.grad;
        const int lead = (int)(a & 15);
        const int64_t span = lead + x.numel * (x.grad_dtype == LT_F32 ? 4 : 2);
        const int64_t it = (span + kNormItemBytes - 1) / kNormItemBytes;
        if (items + it > 0x7fffffff) break;   // next launch; one tensor alone always fits (numel <= 2^38)
        NormDesc& d = P->t[cnt];
        d.base16 = (const void*)(a - lead);
        d.span_bytes = span;
        items += it;
        d.item_end = (int32_t)items;
        d.lead_f32 = lead | ((x.grad_dtype == LT_F32 ? 1 : 0) << 8);
        d.slot = *i;
        d.pad = 0;
        ++cnt; ++*i;
    }
    P->n = cnt;
    P->total_items = (int32_t)items;
}

int launch_sqnorm(const NormParams& p, int sm_count, cudaStream_t s) {
    int grid = kNormCtasPerSm * sm_count;
    if (grid > kNormMaxCtas) grid = kNormMaxCtas;
    if (grid > p.total_items) grid = p.total_items;
    if (grid < 1) grid = 1;
    sqnorm_kernel<<<grid, kNormThreads, 0, s>>>(p);
    if (cudaGetLastError() != cudaSuccess) return LT_ERR_CUDA;
    return LT_OK;
}

}  // namespace lt

// ---- per-tensor norms and skip bookkeeping -----------------------------------------------------------
namespace lt {

// Same item walk as sqnorm_kernel; a CTA flushes its running sum to the tensor's slot whenever the item
// it picks up belongs to another tensor (and at the end), so atomics are few.
__global__ void __launch_bounds__(kNormThreads, 2) sqnorm_per_tensor_kernel(const __grid_constant__ NormParams P) {
    __shared__ double s_warp[kNormThreads / 32];
    const int tid = threadIdx.x;
    double acc = 0.0;
    int t = 0, item_begin = 0, cur = -1;
    for (int w = blockIdx.x; ; w += gridDim.x) {
        const bool more = w < P.total_items;
        if (more) while (w >= P.t[t].item_end) { item_begin = P.t[t].item_end; ++t; }
        if (cur >= 0 && (!more || t != cur)) {      // flush the finished tensor's partial sum
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            __syncthreads();
            if ((tid & 31) == 0) s_warp[tid >> 5] = acc;
            __syncthreads();
            if (tid == 0) {
                double s = 0.0;
                for (int i = 0; i < kNormThreads / 32; ++i) s += s_warp[i];
                atomicAdd(&P.out[P.t[cur].slot], s);
            }
            acc = 0.0;
        }
        if (!more) break;
        cur = t;
        const NormDesc& d = P.t[t];
        const char* base = (const char*)d.base16;
        const int64_t lo = d.lead_f32 & 0xff;
        const bool f32 = (d.lead_f32 >> 8) != 0;
        const int64_t hi = d.span_bytes;
        const int64_t item_off = (int64_t)(w - item_begin) * kNormItemBytes;
#pragma unroll
        for (int k = 0; k < kNormVecPerThread; ++k) {
            const int64_t off = item_off + (int64_t)(k * kNormThreads + tid) * 16;
            if (off >= lo && off + 16 <= hi) {
                const uint4 v = ld_stream16(base + off);
                acc = f32 ? acc + sq4_f32(v) : sq8_bf16(v, acc);
            } else if (off + 16 > lo && off < hi) {
                acc += sq_partial(base, off, lo, hi, f32);
            }
        }
    }
}

__global__ void skip_count_kernel(const double* sqnorm, int32_t* count) {
    if (threadIdx.x == 0 && blockIdx.x == 0) *count = isfinite(*sqnorm) ? 0 : *count + 1;
}

}  // namespace lt

extern "C" int lt_grad_sqnorm_per_tensor(const lt_tensor* tensors, int32_t n, double* d_out, lt_stream stream) {
    using namespace lt;
    int rc = validate_grads(tensors, n, nullptr);
    if (rc != LT_OK) return rc;
    if (n > 0 && d_out == nullptr) return LT_ERR_INVALID_ARG;
    if (((uintptr_t)d_out & 7) != 0) return LT_ERR_ALIGNMENT;
    DeviceInfo* dev = nullptr;
    if ((rc = ensure_device((cudaStream_t)stream, &dev)) != LT_OK) return rc;
    NormParams P;
    P.ticket = nullptr; P.partials = nullptr; P.out = d_out;
    int32_t i = 0;
    while (i < n) {
        pack_norm(tensors, n, &i, &P);
        if (P.n == 0) continue;
        int grid = kNormCtasPerSm * dev->sm_count;
        if (grid > P.total_items) grid = P.total_items;
        sqnorm_per_tensor_kernel<<<grid, kNormThreads, 0, (cudaStream_t)stream>>>(P);
        if (cudaGetLastError() != cudaSuccess) return LT_ERR_CUDA;
    }
    return LT_OK;
}

extern "C" int lt_skip_count_update(const double* d_sqnorm, int32_t* d_skip_count, lt_stream stream) {
    if (!d_sqnorm || !d_skip_count) return LT_ERR_INVALID_ARG;
    if (((uintptr_t)d_sqnorm & 7) != 0 || ((uintptr_t)d_skip_count & 3) != 0) return LT_ERR_ALIGNMENT;
    lt::skip_count_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(d_sqnorm, d_skip_count);
    return cudaGetLastError() == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}

// ---- lt_grad_sqnorm_multi_noalloc ------------------------------------------------------------------
// Same kernel, scratch in a module-scope device array instead of a caller-supplied workspace.
namespace {

constexpr int kNoAllocMaxCtas = 512;                               // partial sums the array has room for
constexpr int kNoAllocScratchBytes = 256 + kNoAllocMaxCtas * 8;    // arrival counter + partials: 4352 bytes

// Every GPU that loads this library holds these 4352 bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// In host code `g_noalloc_scratch` is only a handle for the runtime, not a device address, so the
// address the kernel gets is asked for once per device (with that device current) and kept here.
std::mutex g_noalloc_mu;
void* g_noalloc_ptr[64] = {nullptr};

int noalloc_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return LT_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(g_noalloc_mu);
    if (g_noalloc_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return LT_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return LT_OK;
}

}  // namespace

extern "C" int lt_grad_sqnorm_multi_noalloc(const lt_tensor* tensors, int32_t n, double* d_sqnorm, lt_stream stream) {
    using namespace lt;
    int live = 0;
    int rc = validate_grads(tensors, n, &live);
    if (rc != LT_OK) return rc;
    if (d_sqnorm == nullptr) return LT_ERR_INVALID_ARG;
    if (((uintptr_t)d_sqnorm & 7) != 0) return LT_ERR_ALIGNMENT;
    if (live > LT_NOALLOC_MAX_TENSORS) return LT_ERR_WORKSPACE;   // beyond what one launch over the fixed scratch covers
    if (live == 0) return LT_OK;
    NormParams P;
    int32_t i = 0;
    pack_norm(tensors, n, &i, &P);
    while (i < n && tensors[i].numel == 0) ++i;
    if (i < n) return LT_ERR_UNSUPPORTED;     // 2^31 work items or more: not one launch (nothing has been touched yet)

    DeviceInfo* dev = nullptr;
    if ((rc = ensure_device((cudaStream_t)stream, &dev)) != LT_OK) return rc;
    void* scratch = nullptr;
    if ((rc = noalloc_scratch(&scratch)) != LT_OK) return rc;
    P.ticket = (unsigned int*)scratch;
    P.partials = (double*)((char*)scratch + 256);
    P.out = d_sqnorm;
    // the array keeps what the last call left: the arrival counter must start at zero
    if (cudaMemsetAsync(P.ticket, 0, 256, (cudaStream_t)stream) != cudaSuccess) { cudaGetLastError(); return LT_ERR_CUDA; }
    int grid = kNormCtasPerSm * dev->sm_count;
    if (grid > kNoAllocMaxCtas) grid = kNoAllocMaxCtas;
    if (grid > P.total_items) grid = P.total_items;
    sqnorm_kernel<<<grid, kNormThreads, 0, (cudaStream_t)stream>>>(P);
    return cudaGetLastError() == cudaSuccess ? LT_OK : LT_ERR_CUDA;
}
