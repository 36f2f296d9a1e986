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

// Register-only loops of the FP32 minimum, the instruction the tensor-core E-step spends its ALU
// time on: 16 independent chains per thread.  MODE 0: two-input min.f32; 1: three-input min.f32
// (two new values per instruction); 2: both alternating.  One block per SM; every block reports its
// own cycle count (clock64 around the loop, after a block-wide barrier) and the SM it ran on.
template <int MODE>
__global__ void __launch_bounds__(512) min_rate_kernel(int iters, float seed, float* out, long long* cycles,
                                                       unsigned* smid) {
    float f[16];
    float a = seed + (float)threadIdx.x, b = seed * 3.0f + 1.0f;
#pragma unroll
    for (int c = 0; c < 16; ++c) f[c] = a * (float)(c + 1) + 1.0e6f;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            if (MODE == 0 || (MODE == 2 && (c & 1) == 0)) asm volatile("min.f32 %0, %0, %1;" : "+f"(f[c]) : "f"(a));
            else asm volatile("min.f32 %0, %0, %1, %2;" : "+f"(f[c]) : "f"(a), "f"(b));
        }
    }
    const long long t1 = clock64();
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < 16; ++c) s += f[c];
    if (s == 12345.678f) out[0] = s;
    if (threadIdx.x == 0) {
        cycles[blockIdx.x] = t1 - t0;
        unsigned id;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(id));
        smid[blockIdx.x] = id;
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

cc_status cc_measure_min_rate(cc_ctx* ctx, double* lane_instr_per_clk_per_sm_host, double* sm_mhz_host,
                              int32_t* distinct_sms_host, void* stream) {
    if (!ctx || !lane_instr_per_clk_per_sm_host) return CC_ERR_NULL;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    const int blocks = ctx->sm_count, threads = 512, iters = 8192;
    if (blocks > 1024) return CC_ERR_SHAPE;
    char* dev = nullptr;
    if (cudaMalloc(&dev, 256 + (size_t)blocks * 16) != cudaSuccess) return CC_ERR_CUDA;
    float* out = reinterpret_cast<float*>(dev);
    long long* cyc = reinterpret_cast<long long*>(dev + 256);
    unsigned* smid = reinterpret_cast<unsigned*>(dev + 256 + (size_t)blocks * 8);
    cudaEvent_t a, b;
    if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { cudaFree(dev); return CC_ERR_CUDA; }
    cc_status status = CC_OK;
    static long long h_cyc[1024];
    static unsigned h_sm[1024];
    double mhz_sum = 0.0;
    int distinct = 0;
    for (int mode = 0; mode < 3 && status == CC_OK; ++mode) {
        double best = 0.0;
        for (int rep = 0; rep < 3; ++rep) {   // first repetition warms up; keep the best of the rest
            cudaEventRecord(a, st);
            if (mode == 0) min_rate_kernel<0><<<blocks, threads, 0, st>>>(iters, 1.0f, out, cyc, smid);
            else if (mode == 1) min_rate_kernel<1><<<blocks, threads, 0, st>>>(iters, 1.0f, out, cyc, smid);
            else min_rate_kernel<2><<<blocks, threads, 0, st>>>(iters, 1.0f, out, cyc, smid);
            ctx->launches++;
            cudaEventRecord(b, st);
            if (cudaEventSynchronize(b) != cudaSuccess ||
                cudaMemcpy(h_cyc, cyc, sizeof(long long) * blocks, cudaMemcpyDeviceToHost) != cudaSuccess ||
                cudaMemcpy(h_sm, smid, sizeof(unsigned) * blocks, cudaMemcpyDeviceToHost) != cudaSuccess) {
                status = CC_ERR_CUDA;
                break;
            }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            // a block alone on its SM: lane-instructions of the block over its own cycle count; the
            // median over the blocks ignores an SM that had to run two of them
            double rate[1024];
            long long cmax = 0;
            for (int i = 0; i < blocks; ++i) {
                rate[i] = (double)threads * 16.0 * (double)iters / (double)(h_cyc[i] > 0 ? h_cyc[i] : 1);
                if (h_cyc[i] > cmax) cmax = h_cyc[i];
            }
            for (int i = 1; i < blocks; ++i) {   // insertion sort: at most a few hundred entries
                const double v = rate[i];
                int j = i - 1;
                while (j >= 0 && rate[j] > v) { rate[j + 1] = rate[j]; --j; }
                rate[j + 1] = v;
            }
            if (rep > 0 && rate[blocks / 2] > best) best = rate[blocks / 2];
            if (rep == 2) {
                mhz_sum += (double)cmax / ((double)ms * 1e3);   // cycles of the longest block over the launch's time
                if (mode == 0) {
                    bool seen[4096] = {};
                    for (int i = 0; i < blocks; ++i) if (h_sm[i] < 4096 && !seen[h_sm[i]]) { seen[h_sm[i]] = true; ++distinct; }
                }
            }
        }
        lane_instr_per_clk_per_sm_host[mode] = best;
    }
    if (sm_mhz_host) *sm_mhz_host = mhz_sum / 3.0;
    if (distinct_sms_host) *distinct_sms_host = distinct;
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    cudaFree(dev);
    if (status == CC_OK && cudaGetLastError() != cudaSuccess) status = CC_ERR_CUDA;
    return status;
}

}  // extern "C"
