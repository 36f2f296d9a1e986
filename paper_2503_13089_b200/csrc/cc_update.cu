// M-step of Section 3.1: per-cluster mean, exact and order-independent.
//
// Every finite FP16 value is an integer multiple of 2^-24, and those of magnitude >= 8 are
// multiples of 2^-7.  Each coordinate is therefore added as an INTEGER into one of two 64-bit
// accumulators per (cluster, dimension): |x| < 8 in units of 2^-24 (< 2^27 per term) and
// |x| >= 8 in units of 2^-7 (< 2^23 per term).  With N < 2^31 neither can overflow, integer
// addition is associative, and so the result does not depend on the order in which the points
// arrive: the kernel is deterministic without sorting the points first, the counts are exact
// integers, and the mean is rounded exactly once (sum -> double -> divide -> FP32).
// A cluster with no member keeps its previous centroid.
// The same property lets the Lloyd loop keep the sums between iterations and only move the points
// whose code changed (update_delta_kernel), and gives the gradient with respect to the codebook
// (the same sums without the division).
#include "cc_common.cuh"

namespace {

typedef unsigned long long ull;

__device__ __forceinline__ void add_coord(uint16_t h, ull* lo, ull* hi) {
    const float v = __half2float(__ushort_as_half(h));
    const unsigned e = (h >> 10) & 31u;
    if (e == 31u) return;                       // non-finite: reported by the E-step, skipped here
    if (e >= 18u) {                             // |v| >= 8: multiple of 2^-7
        const long long q = __float2ll_rn(v * 128.0f);
        atomicAdd(hi, (ull)q);
    } else if ((h & 0x7fffu) != 0u) {           // multiple of 2^-24
        const long long q = __float2ll_rn(v * 16777216.0f);
        atomicAdd(lo, (ull)q);
    }
}

template <int G>
__global__ void __launch_bounds__(256)
update_accumulate_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ idx, int K,
                         ull* __restrict__ sum_lo, ull* __restrict__ sum_hi, int* __restrict__ counts) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += (int64_t)gridDim.x * blockDim.x) {
        const int j = idx[i];
        if (j >= K) continue;
        atomicAdd(counts + j, 1);
        const uint16_t* row = X + i * G;
        uint16_t h[G];
        if constexpr (G % 8 == 0) {
#pragma unroll
            for (int v = 0; v < G / 8; ++v) {
                uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
                unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) { h[v * 8 + 2 * k] = w[k] & 0xffffu; h[v * 8 + 2 * k + 1] = w[k] >> 16; }
            }
        } else if constexpr (G % 4 == 0) {
#pragma unroll
            for (int v = 0; v < G / 4; ++v) {
                uint2 u = __ldg(reinterpret_cast<const uint2*>(row) + v);
                h[v * 4] = u.x & 0xffffu; h[v * 4 + 1] = u.x >> 16; h[v * 4 + 2] = u.y & 0xffffu; h[v * 4 + 3] = u.y >> 16;
            }
        } else {
#pragma unroll
            for (int t = 0; t < G; ++t) h[t] = __ldg(row + t);
        }
#pragma unroll
        for (int t = 0; t < G; ++t) add_coord(h[t], sum_lo + (int64_t)j * G + t, sum_hi + (int64_t)j * G + t);
    }
}

// M-step inside the Lloyd loop, from the second iteration on: the sums of the previous M-step are
// still in the workspace, so only the points whose code changed are moved, subtracted from their
// old cluster and added to the new one.  Integer sums make this bit-identical to summing all the
// points again.  idx_prev holds the codes the sums correspond to and is brought up to date.
template <int G>
__global__ void __launch_bounds__(256)
update_delta_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ idx,
                    uint16_t* __restrict__ idx_prev, int K, ull* __restrict__ sum_lo, ull* __restrict__ sum_hi,
                    int* __restrict__ counts) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += (int64_t)gridDim.x * blockDim.x) {
        const int jn = idx[i], jo = idx_prev[i];
        if (jn == jo || jn >= K || jo >= K) continue;
        idx_prev[i] = (uint16_t)jn;
        atomicAdd(counts + jn, 1);
        atomicSub(counts + jo, 1);
        const uint16_t* row = X + i * G;
#pragma unroll
        for (int t = 0; t < G; ++t) {
            const uint16_t h = __ldg(row + t);
            const float v = __half2float(__ushort_as_half(h));
            const unsigned e = (h >> 10) & 31u;
            if (e == 31u) continue;
            if (e >= 18u) {
                const long long q = __float2ll_rn(v * 128.0f);
                atomicAdd(sum_hi + (int64_t)jn * G + t, (ull)q);
                atomicAdd(sum_hi + (int64_t)jo * G + t, (ull)(-q));
            } else if ((h & 0x7fffu) != 0u) {
                const long long q = __float2ll_rn(v * 16777216.0f);
                atomicAdd(sum_lo + (int64_t)jn * G + t, (ull)q);
                atomicAdd(sum_lo + (int64_t)jo * G + t, (ull)(-q));
            }
        }
    }
}

__global__ void __launch_bounds__(256)
update_finish_kernel(const long long* __restrict__ sum_lo, const long long* __restrict__ sum_hi,
                     const int* __restrict__ counts, int K, int g, float* __restrict__ C) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= K * g) return;
    const int n = counts[e / g];
    if (n <= 0) return;   // empty cluster: previous centroid stays
    const double s = (double)sum_lo[e] * 5.9604644775390625e-8 + (double)sum_hi[e] * 0.0078125;
    C[e] = (float)(s / (double)n);
}

// Gradient with respect to the codebook: the exact integer sums as they are, rounded once to FP32.
__global__ void __launch_bounds__(256)
grad_finish_kernel(const long long* __restrict__ sum_lo, const long long* __restrict__ sum_hi, int n,
                   float* __restrict__ dC) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    dC[e] = (float)((double)sum_lo[e] * 5.9604644775390625e-8 + (double)sum_hi[e] * 0.0078125);
}

}  // namespace

#define CC_UPDATE_DISPATCH(g, CALL)                                                                           \
    switch (g) {                                                                                              \
        case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;   case 4: CALL(4); break;   \
        case 5: CALL(5); break;   case 6: CALL(6); break;   case 7: CALL(7); break;   case 8: CALL(8); break;   \
        case 9: CALL(9); break;   case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break; \
        case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break; case 16: CALL(16); break; \
        default: return cudaErrorInvalidValue;                                                                \
    }

namespace {

template <int G>
cudaError_t launch_accumulate(cc_ctx* ctx, const uint16_t* X, int64_t N, const uint16_t* idx, int K, ull* sum_lo,
                              ull* sum_hi, int32_t* counts, cudaStream_t st) {
    ProfScope ps(ctx, CC_K_UPDATE_ACCUM, st);
    int64_t blocks = (N + 255) / 256;
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    update_accumulate_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, K, sum_lo, sum_hi, counts);
    return cudaGetLastError();
}

}  // namespace

cudaError_t cc_launch_update(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g, const uint16_t* idx,
                             int K, float* C, int32_t* counts, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    ull* sum_lo = reinterpret_cast<ull*>(ws + L.sum_lo);
    ull* sum_hi = reinterpret_cast<ull*>(ws + L.sum_hi);
    cudaError_t e;
    // sum_lo and sum_hi are adjacent in the workspace
    if ((e = cudaMemsetAsync(sum_lo, 0, L.tmp_c - L.sum_lo, st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(counts, 0, sizeof(int32_t) * (size_t)K, st)) != cudaSuccess) return e;
    if (N > 0) {
#define CALL(G) e = launch_accumulate<G>(ctx, X, N, idx, K, sum_lo, sum_hi, counts, st)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
        if (e != cudaSuccess) return e;
    }
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                             reinterpret_cast<long long*>(sum_hi), counts, K, g, C);
    return cudaGetLastError();
}

// dC[j] = sum of dX[i] over idx[i] = j, with the M-step's exact accumulation (scratch counts in the
// workspace: the position list of the initialisation is free by then).
cudaError_t cc_launch_codebook_grad(cc_ctx* ctx, const WsLayout& L, const uint16_t* dX, int64_t N, int g,
                                    const uint16_t* idx, int K, float* dC, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    ull* sum_lo = reinterpret_cast<ull*>(ws + L.sum_lo);
    ull* sum_hi = reinterpret_cast<ull*>(ws + L.sum_hi);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.positions);
    cudaError_t e;
    if ((e = cudaMemsetAsync(sum_lo, 0, L.tmp_c - L.sum_lo, st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(counts, 0, sizeof(int32_t) * (size_t)K, st)) != cudaSuccess) return e;
    if (N > 0) {
#define CALL(G) e = launch_accumulate<G>(ctx, dX, N, idx, K, sum_lo, sum_hi, counts, st)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
        if (e != cudaSuccess) return e;
    }
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    grad_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                            reinterpret_cast<long long*>(sum_hi), K * g, dC);
    return cudaGetLastError();
}

// Incremental M-step (see update_delta_kernel): the workspace sums and `counts` must be those of
// the previous M-step on the same X, and idx_prev the codes they were computed from.
cudaError_t cc_launch_update_delta(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                   const uint16_t* idx, uint16_t* idx_prev, int K, float* C, int32_t* counts,
                                   cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    ull* sum_lo = reinterpret_cast<ull*>(ws + L.sum_lo);
    ull* sum_hi = reinterpret_cast<ull*>(ws + L.sum_hi);
    if (N > 0) {
        int64_t blocks = (N + 255) / 256;
        const int64_t cap = (int64_t)ctx->sm_count * 16;
        if (blocks > cap) blocks = cap;
        ProfScope ps(ctx, CC_K_UPDATE_ACCUM, st);
#define CALL(G) update_delta_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, idx_prev, K, sum_lo, sum_hi, counts)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
    }
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                             reinterpret_cast<long long*>(sum_hi), counts, K, g, C);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// M-step for callers that cannot allocate device memory: the integer sums live in a fixed array
// that is part of the loaded library image instead of a caller-provided workspace.
namespace {

constexpr int kStaticMaxDevices = 64;

// [0, CC_UPDATE_STATIC_MAX_KG): sums in units of 2^-24; [MAX_KG, 2*MAX_KG): sums in units of 2^-7.
static __device__ __align__(256) ull g_static_sums[2 * CC_UPDATE_STATIC_MAX_KG];

// Device address of g_static_sums on each device.  In host code the symbol's name is only a
// handle; the address a kernel may dereference comes from cudaGetSymbolAddress, asked once per
// device with that device current.
void* g_static_addr[kStaticMaxDevices] = {};

cudaError_t static_sums_address(int device, ull** out) {
    if (!g_static_addr[device]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_sums);
        if (e != cudaSuccess) return e;
        g_static_addr[device] = p;
    }
    *out = static_cast<ull*>(g_static_addr[device]);
    return cudaSuccess;
}

}  // namespace

extern "C" cc_status cc_update_static(int device, const uint16_t* X, int64_t N, int g, const uint16_t* idx, int K,
                                      float* C, int32_t* counts, void* stream) {
    if (!C || !counts || (N > 0 && (!X || !idx))) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (N < 0 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if ((int64_t)K * g > CC_UPDATE_STATIC_MAX_KG) return CC_ERR_STATIC_CAPACITY;
    if (device < 0 || device >= kStaticMaxDevices) return CC_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(C) & 15u)) return CC_ERR_ALIGN;
    if (cudaSetDevice(device) != cudaSuccess) return CC_ERR_CUDA;
    ull* sums = nullptr;
    if (static_sums_address(device, &sums) != cudaSuccess) return CC_ERR_CUDA;
    ull* sum_lo = sums;
    ull* sum_hi = sums + CC_UPDATE_STATIC_MAX_KG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t used = sizeof(ull) * (size_t)K * g;
    // the array still holds the previous call's sums
    if (cudaMemsetAsync(sum_lo, 0, used, st) != cudaSuccess) return CC_ERR_CUDA;
    if (cudaMemsetAsync(sum_hi, 0, used, st) != cudaSuccess) return CC_ERR_CUDA;
    if (cudaMemsetAsync(counts, 0, sizeof(int32_t) * (size_t)K, st) != cudaSuccess) return CC_ERR_CUDA;
    if (N > 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return CC_ERR_CUDA;
        int64_t blocks = (N + 255) / 256;
        const int64_t cap = (int64_t)sms * 16;
        if (blocks > cap) blocks = cap;
#define CALL(G)                                                                                               \
    update_accumulate_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, K, sum_lo, sum_hi, counts)
        switch (g) {
            case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;   case 4: CALL(4); break;
            case 5: CALL(5); break;   case 6: CALL(6); break;   case 7: CALL(7); break;   case 8: CALL(8); break;
            case 9: CALL(9); break;   case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;
            case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break; case 16: CALL(16); break;
            default: return CC_ERR_UNSUPPORTED_G;
        }
#undef CALL
    }
    update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                             reinterpret_cast<long long*>(sum_hi), counts, K, g, C);
    return cudaGetLastError() == cudaSuccess ? CC_OK : CC_ERR_CUDA;
}
