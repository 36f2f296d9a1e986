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
        int64_t blocks = (N + 255) / 256;
        const int64_t cap = (int64_t)ctx->sm_count * 16;
        if (blocks > cap) blocks = cap;
        ProfScope ps(ctx, CC_K_UPDATE_ACCUM, st);
#define CALL(G)                                                                                               \
    update_accumulate_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, K, sum_lo, sum_hi, counts)
        switch (g) {
            case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;   case 4: CALL(4); break;
            case 5: CALL(5); break;   case 6: CALL(6); break;   case 7: CALL(7); break;   case 8: CALL(8); break;
            case 9: CALL(9); break;   case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;
            case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break; case 16: CALL(16); break;
            default: return cudaErrorInvalidValue;
        }
#undef CALL
    }
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                             reinterpret_cast<long long*>(sum_hi), counts, K, g, C);
    return cudaGetLastError();
}
