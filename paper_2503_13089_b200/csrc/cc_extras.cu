// Options around the clustering path that the paper mentions or leaves to its k-means library:
// uniform quantisation of the stored codebook (Section 5.3, "Inference latency"), a cluster-splitting
// rule for empty clusters, and the gather of a subsampled training set.
#include <cuda_fp16.h>

#include "cc_common.cuh"

namespace {

// ---------------------------------------------------------------------------------------------
// Uniform symmetric quantisation of the FP16 codebook to b = 8 or 4 bits, one scale per codebook:
//   s = max|c| / (2^(b-1) - 1),  q = clamp(round-to-nearest-even(c / s), -2^(b-1), 2^(b-1) - 1),
// all in IEEE single precision (division and product correctly rounded).
__global__ void __launch_bounds__(256)
quant_absmax_kernel(const uint16_t* __restrict__ C16, int64_t n, unsigned* __restrict__ max_bits) {
    unsigned m = 0u;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        const unsigned a = C16[e] & 0x7fffu;          // |c| as a bit pattern: orders like the value
        if (a <= 0x7c00u) m = max(m, a);              // NaN patterns are ignored, Inf is kept
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m) atomicMax(max_bits, m);
}

__device__ __forceinline__ int quant_one(uint16_t h, float s, int L) {
    const float c = __half2float(__ushort_as_half(h));
    float r = rintf(__fdiv_rn(c, s));                 // ties to even
    r = fminf(fmaxf(r, -(float)(L + 1)), (float)L);
    return (int)r;
}

// One thread per output byte: one element (8 bits) or two (4 bits: element 2k in the low nibble).
__global__ void __launch_bounds__(256)
quant_apply_kernel(const uint16_t* __restrict__ C16, int64_t n, int bits, const unsigned* __restrict__ max_bits,
                   uint8_t* __restrict__ q, float* __restrict__ scale, uint16_t* __restrict__ deq) {
    const int L = (1 << (bits - 1)) - 1;
    const float maxabs = __half2float(__ushort_as_half((unsigned short)*max_bits));
    const float s = maxabs > 0.f ? __fdiv_rn(maxabs, (float)L) : 1.0f;
    const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) *scale = s;
    if (bits == 8) {
        if (b >= n) return;
        const int v = quant_one(C16[b], s, L);
        q[b] = (uint8_t)(int8_t)v;
        if (deq) deq[b] = __half_as_ushort(__float2half_rn(__fmul_rn((float)v, s)));
    } else {
        const int64_t e0 = 2 * b;
        if (e0 >= n) return;
        const int v0 = quant_one(C16[e0], s, L);
        const int v1 = (e0 + 1 < n) ? quant_one(C16[e0 + 1], s, L) : 0;
        q[b] = (uint8_t)((v0 & 0xF) | ((v1 & 0xF) << 4));
        if (deq) {
            deq[e0] = __half_as_ushort(__float2half_rn(__fmul_rn((float)v0, s)));
            if (e0 + 1 < n) deq[e0 + 1] = __half_as_ushort(__float2half_rn(__fmul_rn((float)v1, s)));
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Rows pos[0..n) of X (g halves each) copied to consecutive rows of `out`.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint16_t* __restrict__ X, int g, const unsigned* __restrict__ pos, int64_t n,
                   uint16_t* __restrict__ out) {
    const int64_t total = n * g;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / g;
        const int t = (int)(e - r * g);
        out[e] = __ldg(X + (int64_t)pos[r] * g + t);
    }
}

// ---------------------------------------------------------------------------------------------
// Second empty-cluster rule (the default keeps the centroid): after the means, every empty cluster e,
// in increasing order, takes over half of the most populated cluster d (largest working count, lowest
// index among equals; nothing happens once that count is below 2): c_e = c_d, then coordinate t of
// c_e is multiplied by 1 + 2^-10 and that of c_d by 1 - 2^-10 for even t, the other way round for odd
// t (FP32 products); working counts n_e = floor(n_d / 2), n_d -= n_e.  The member counts reported
// to the caller are not changed.
// One block: thread t owns a contiguous range of clusters and keeps the best (count, lowest index)
// of its range; an iteration is a block-wide maximum of those plus two range rescans.
constexpr int SPLIT_THREADS = 1024;

__device__ __forceinline__ unsigned long long split_key(int count, int index) {
    return ((unsigned long long)(unsigned)count << 32) | (unsigned long long)(0xffffffffu - (unsigned)index);
}

__global__ void __launch_bounds__(SPLIT_THREADS)
split_empty_kernel(float* __restrict__ C, int K, int g, const int* __restrict__ counts, int* __restrict__ work,
                   int* __restrict__ empties) {
    __shared__ int scan[SPLIT_THREADS];
    __shared__ unsigned long long wmax[SPLIT_THREADS / 32];
    __shared__ unsigned long long best_sh;
    const int tid = threadIdx.x;
    const int per = (K + SPLIT_THREADS - 1) / SPLIT_THREADS;
    const int lo = min(K, tid * per), hi = min(K, lo + per);
    int n_mine = 0;
    for (int j = lo; j < hi; ++j) {
        const int n = counts[j];
        work[j] = n;
        n_mine += (n == 0);
    }
    // exclusive scan of the per-thread numbers of empty clusters: the list comes out in index order
    scan[tid] = n_mine;
    __syncthreads();
    for (int o = 1; o < SPLIT_THREADS; o <<= 1) {
        const int v = (tid >= o) ? scan[tid - o] : 0;
        __syncthreads();
        scan[tid] += v;
        __syncthreads();
    }
    const int n_empty = scan[SPLIT_THREADS - 1];
    int at = scan[tid] - n_mine;
    for (int j = lo; j < hi; ++j)
        if (counts[j] == 0) empties[at++] = j;
    auto range_best = [&]() {
        unsigned long long b = 0ull;
        for (int j = lo; j < hi; ++j) {
            const unsigned long long k = split_key(work[j], j);
            b = k > b ? k : b;
        }
        return b;
    };
    unsigned long long mine = range_best();
    __syncthreads();
    const float up = 1.0f + 0.0009765625f, down = 1.0f - 0.0009765625f;
    for (int k = 0; k < n_empty; ++k) {
        unsigned long long b = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, b, o);
            b = other > b ? other : b;
        }
        if ((tid & 31) == 0) wmax[tid >> 5] = b;
        __syncthreads();
        if (tid < 32) {
            b = wmax[tid];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const unsigned long long other = __shfl_xor_sync(0xffffffffu, b, o);
                b = other > b ? other : b;
            }
            if (tid == 0) best_sh = b;
        }
        __syncthreads();
        const unsigned long long best = best_sh;
        const int n_d = (int)(best >> 32);
        const int d = (int)(0xffffffffu - (unsigned)(best & 0xffffffffull));
        if (n_d < 2) break;                           // the largest count only shrinks: nobody can donate any more
        const int e = empties[k];
        if (tid < g) {
            const float c = C[(int64_t)d * g + tid];
            C[(int64_t)e * g + tid] = __fmul_rn(c, (tid & 1) ? down : up);
            C[(int64_t)d * g + tid] = __fmul_rn(c, (tid & 1) ? up : down);
        }
        const int half = n_d / 2;
        if (d >= lo && d < hi) { work[d] = n_d - half; mine = range_best(); }
        if (e >= lo && e < hi) { work[e] = half; mine = range_best(); }
        __syncthreads();                              // best_sh and wmax are rewritten next round
    }
}

}  // namespace

cudaError_t cc_launch_quantize_codebook(cc_ctx* ctx, const uint16_t* C16, int64_t n, int bits, uint8_t* q, float* scale,
                                        uint16_t* deq, cudaStream_t st) {
    unsigned* max_bits = reinterpret_cast<unsigned*>(static_cast<char*>(ctx->ws) + 144);   // word 36 of the status block
    cudaError_t e = cudaMemsetAsync(max_bits, 0, sizeof(unsigned), st);
    if (e != cudaSuccess) return e;
    {
        ProfScope ps(ctx, CC_K_OTHER, st);
        int64_t blocks = (n + 255) / 256;
        if (blocks > 1024) blocks = 1024;
        quant_absmax_kernel<<<(unsigned)blocks, 256, 0, st>>>(C16, n, max_bits);
    }
    ProfScope ps(ctx, CC_K_OTHER, st);
    const int64_t bytes = bits == 8 ? n : (n + 1) / 2;
    quant_apply_kernel<<<(unsigned)((bytes + 255) / 256), 256, 0, st>>>(C16, n, bits, max_bits, q, scale, deq);
    return cudaGetLastError();
}

cudaError_t cc_launch_gather_rows(cc_ctx* ctx, const uint16_t* X, int g, const unsigned* pos_dev, int64_t n,
                                  uint16_t* out, cudaStream_t st) {
    ProfScope ps(ctx, CC_K_OTHER, st);
    int64_t blocks = (n * g + 255) / 256;
    const int64_t cap = (int64_t)ctx->sm_count * 16;
    if (blocks > cap) blocks = cap;
    gather_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(X, g, pos_dev, n, out);
    return cudaGetLastError();
}

cudaError_t cc_launch_split_empty(cc_ctx* ctx, const WsLayout& L, float* C, int K, int g, const int32_t* counts,
                                  cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    split_empty_kernel<<<1, SPLIT_THREADS, 0, st>>>(C, K, g, counts, reinterpret_cast<int*>(ws + L.count_copies),
                                                   reinterpret_cast<int*>(ws + L.positions));
    return cudaGetLastError();
}
