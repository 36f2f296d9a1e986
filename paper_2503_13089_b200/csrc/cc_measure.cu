// Measurement aids: per-kernel event timing read-out and an FP32 FMA saturation kernel.
#include "cc_common.cuh"

namespace {

typedef unsigned long long ull;

// 8 independent FMA chains per thread, operands in registers only.
template <bool PACKED>
__global__ void __launch_bounds__(256) fma_peak_kernel(float* out, int iters, float seed) {
    float a = seed + threadIdx.x * 1e-6f, b = 0.999f;
    if (PACKED) {
        ull acc[8], av, bv;
        asm("mov.b64 %0, {%1, %2};" : "=l"(av) : "f"(a), "f"(a + 1e-3f));
        asm("mov.b64 %0, {%1, %2};" : "=l"(bv) : "f"(b), "f"(b));
#pragma unroll
        for (int k = 0; k < 8; ++k) asm("mov.b64 %0, {%1, %2};" : "=l"(acc[k]) : "f"(a * k), "f"(a + k));
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int k = 0; k < 8; ++k) asm volatile("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc[k]) : "l"(bv), "l"(av));
        }
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float lo, hi;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc[k]));
            s += lo + hi;
        }
        if (s == 12345.678f) out[0] = s;   // keeps the loop alive without a store in practice
    } else {
        float acc[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) acc[k] = a * k;
        for (int i = 0; i < iters; ++i) {
#pragma unroll
            for (int k = 0; k < 16; ++k) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(acc[k]) : "f"(b), "f"(a));
        }
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) s += acc[k];
        if (s == 12345.678f) out[0] = s;
    }
}

}  // namespace

extern "C" {

cc_status cc_profile_enable(cc_ctx* ctx, int on) {
    if (!ctx) return CC_ERR_NULL;
    if (on && !ctx->prof) {
        ctx->prof = new cc_prof_slot[CC_PROF_CAP];
        ctx->prof_used = ctx->prof_made = 0;
    }
    ctx->prof_on = on ? 1 : 0;
    return CC_OK;
}

cc_status cc_profile_read(cc_ctx* ctx, double* total_ms_host, int64_t* launches_host) {
    if (!ctx) return CC_ERR_NULL;
    double ms[CC_K_COUNT] = {0};
    int64_t n[CC_K_COUNT] = {0};
    cc_status s = CC_OK;
    for (int i = 0; i < ctx->prof_used; ++i) {
        cc_prof_slot& sl = ctx->prof[i];
        float t = 0.f;
        if (cudaEventSynchronize(sl.b) != cudaSuccess || cudaEventElapsedTime(&t, sl.a, sl.b) != cudaSuccess) {
            s = CC_ERR_CUDA;
            continue;
        }
        ms[sl.kind] += t;
        n[sl.kind] += 1;
    }
    ctx->prof_used = 0;
    for (int k = 0; k < CC_K_COUNT; ++k) {
        if (total_ms_host) total_ms_host[k] = ms[k];
        if (launches_host) launches_host[k] = n[k];
    }
    return s;
}

cc_status cc_measure_fp32_peak(cc_ctx* ctx, double* tflops_scalar_host, double* tflops_packed_host, void* stream) {
    if (!ctx) return CC_ERR_NULL;
    if (!ctx->ws) return CC_ERR_WORKSPACE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    float* out = reinterpret_cast<float*>(static_cast<char*>(ctx->ws) + 128);   // unused status words
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return CC_ERR_CUDA;
    const int blocks = ctx->sm_count * 8, iters = 20000;
    double res[2] = {0, 0};
    for (int packed = 0; packed < 2; ++packed) {
        for (int rep = 0; rep < 3; ++rep) {   // first repetition warms up; keep the best of the rest
            cudaEventRecord(a, st);
            if (packed) fma_peak_kernel<true><<<blocks, 256, 0, st>>>(out, iters, 1.0f);
            else fma_peak_kernel<false><<<blocks, 256, 0, st>>>(out, iters, 1.0f);
            ctx->launches++;
            cudaEventRecord(b, st);
            if (cudaEventSynchronize(b) != cudaSuccess) return CC_ERR_CUDA;
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            const double flops = 2.0 * 16.0 * (double)iters * 256.0 * (double)blocks;
            const double tf = flops / (ms * 1e-3) / 1e12;
            if (rep > 0 && tf > res[packed]) res[packed] = tf;
        }
    }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    if (tflops_scalar_host) *tflops_scalar_host = res[0];
    if (tflops_packed_host) *tflops_packed_host = res[1];
    return cudaGetLastError() == cudaSuccess ? CC_OK : CC_ERR_CUDA;
}

}  // extern "C"
