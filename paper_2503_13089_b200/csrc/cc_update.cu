// M-step of Section 3.1: per-cluster mean, exact and order-independent.
//
// Every finite FP16 value is an integer multiple of 2^-24, and those of magnitude >= 8 are
// multiples of 2^-7.  Each coordinate is therefore added as an INTEGER into one of two 64-bit
// accumulators per (cluster, dimension): |x| < 8 in units of 2^-24 (< 2^27 per term) and
// |x| >= 8 in units of 2^-7 (< 2^23 per term).  With N < 2^31 neither can overflow, integer
// addition is associative, and so the result does not depend on the order in which the points
// arrive: the kernel is deterministic without sorting the points first and the counts are exact
// integers.  The mean is formed as the CPU oracle forms it: the integer sums go to double (exact
// while a sum stays below 2^53 units of 2^-24, i.e. |sum| < 2^29: more than 8000 values of the
// largest FP16 magnitude in one cluster, or 5 * 10^8 of magnitude 1), are divided by the count in
// double and the quotient is rounded to FP32.
// A cluster with no member keeps its previous centroid.
// The same property lets the Lloyd loop keep the sums between iterations and only move the points
// whose code changed (update_delta_kernel), and gives the gradient with respect to the codebook
// (the same sums without the division).
#include "cc_common.cuh"
#include "cc_assign_shared.cuh"

namespace {

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

// One lane per coordinate: the G reductions of a point go to G adjacent 64-bit words (one 32-byte
// sector at G = 4, one 128-byte line at G = 16), so a warp's reduction instruction touches 32 / G
// sectors instead of 32.  With few clusters the same words are hit by many points at once and the
// reductions queue up in L2; the sums are then kept in R copies (copy = block % R, one after the
// other, `copy_elems` words apart; the counts likewise, K apart) which the finish kernel adds up.
template <int G>
__global__ void __launch_bounds__(256)
update_accumulate_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ idx, int K,
                         ull* __restrict__ sum_lo, ull* __restrict__ sum_hi, int* __restrict__ counts, int R) {
    const int copy = (int)(blockIdx.x % (unsigned)R);
    sum_lo += (int64_t)copy * K * G;
    sum_hi += (int64_t)copy * K * G;
    counts += (int64_t)copy * K;
    const int64_t total = N * G;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    constexpr int EB = 4;                            // elements per thread and round: their loads are issued together
    for (int64_t e0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e0 < total; e0 += EB * stride) {
        int jj[EB];
        uint16_t hh[EB];
#pragma unroll
        for (int p = 0; p < EB; ++p) {
            const int64_t e = e0 + p * stride;
            jj[p] = (e < total) ? (int)__ldg(idx + e / G) : K;
            hh[p] = (e < total) ? __ldg(X + e) : (uint16_t)0;
        }
#pragma unroll
        for (int p = 0; p < EB; ++p) {
            const int64_t e = e0 + p * stride;
            const int j = jj[p];
            if (j >= K) continue;
            const int t = (int)(e % G);
            if (t == 0) atomicAdd(counts + j, 1);
            add_coord(hh[p], sum_lo + (int64_t)j * G + t, sum_hi + (int64_t)j * G + t);
        }
    }
}

// M-step over all points for codebooks whose accumulators fit one SM's shared memory (K (8 g + 4) bytes
// within 196 KB: K = 4096 at g = 4): every thread block keeps a private copy of all sums and counts in
// shared memory, so that a point costs shared-memory atomics instead of two reduction requests to L2
// (which is what bounds update_accumulate_kernel: the path from the SMs to L2 takes about one such
// request per two clocks and SM), and adds its copy to the global 64-bit accumulators at the end.
// Exact and order-independent as before: coordinate values in units of 2^-24 are added as 32-bit words
// with carry into a second word; the words are biased by 2^27 per addend so that every addend is
// non-negative and a carry is rare (the bias, count * 2^27, is taken off when the block adds its sums to
// the global accumulators).  Values of magnitude >= 8 are rare and go straight to the global accumulator
// in units of 2^-7.
// Measured and not kept: the same kernel for larger codebooks with the clusters cut into ranges that fit
// shared memory, every block scanning the codes of a slice of the points for those inside its range
// (compacted through a per-warp queue).  Every code is then inspected once per range, and on a B200 that
// cost more than it saved: g = 4, K = 65536 (12 ranges), 58.7 M points 1.87 ms against 0.91 ms with L2
// reductions, 16.7 M points 0.54 against 0.26 ms.
constexpr int UP_THREADS = 1024;
constexpr int UP_SMEM = 196 * 1024;

template <int G>
__global__ void __launch_bounds__(UP_THREADS, 1)
update_private_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ idx, int K,
                      ull* __restrict__ sum_lo, ull* __restrict__ sum_hi, int* __restrict__ counts) {
    extern __shared__ uint32_t up_sm[];
    // coordinate-major (word t K + j): at step t a warp's 32 points hit banks j mod 32, spread over all
    // banks, where the cluster-major order would confine them to the banks t mod G
    uint32_t* lo32 = up_sm;                          // G x K: low words of the biased sums
    uint32_t* hi32 = lo32 + (size_t)K * G;           // G x K: carries
    uint32_t* cnt = hi32 + (size_t)K * G;            // K
    for (int e = threadIdx.x; e < K * (2 * G + 1); e += UP_THREADS) up_sm[e] = 0u;
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * UP_THREADS;
    constexpr int PB = (G <= 8) ? 4 : 2;             // points per thread and round: their loads are issued together
    for (int64_t i0 = (int64_t)blockIdx.x * UP_THREADS + threadIdx.x; i0 < N; i0 += PB * stride) {
        unsigned jj[PB];
        float xx[PB][G];
#pragma unroll
        for (int p = 0; p < PB; ++p) {
            const int64_t i = i0 + p * stride;
            bool nf = false;
            jj[p] = (i < N) ? (unsigned)__ldg(idx + i) : 0xffffffffu;
            load_point<G>(X, i, N, xx[p], nf);
        }
#pragma unroll
        for (int p = 0; p < PB; ++p) {
            const unsigned j = jj[p];
            if (j >= (unsigned)K) continue;
            atomicAdd(cnt + j, 1u);
#pragma unroll
            for (int t = 0; t < G; ++t) {
                const float v = xx[p][t];
                uint32_t q = 1u << 27;               // the bias alone: a skipped or coarse value adds nothing else
                if (fabsf(v) >= 8.0f) {
                    if (fabsf(v) <= 65504.0f)        // finite: multiple of 2^-7, straight to the global accumulator
                        atomicAdd(sum_hi + (int64_t)j * G + t, (ull)__float2ll_rn(v * 128.0f));
                } else if (v == v) {
                    q += (uint32_t)__float2int_rn(v * 16777216.0f);      // |.| < 2^27
                }
                const uint32_t old = atomicAdd(lo32 + t * K + j, q);
                if (old + q < old) atomicAdd(hi32 + t * K + j, 1u);      // carry out of the low word
            }
        }
    }
    __syncthreads();
    // add this block's sums to the global accumulators (cluster-major): one reduction per touched word
    for (int e = threadIdx.x; e < K * G; e += UP_THREADS) {
        const int j = e / G, t = e - j * G;
        const uint32_t c = cnt[j];
        if (c == 0u) continue;
        const ull v = (((ull)hi32[t * K + j] << 32) | (ull)lo32[t * K + j]) - ((ull)c << 27);
        if (v) atomicAdd(sum_lo + e, v);
    }
    for (int j = threadIdx.x; j < K; j += UP_THREADS)
        if (cnt[j]) atomicAdd(counts + j, (int)cnt[j]);
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

// Adds up the R copies of the sums and counts, leaves the totals in copy 0 and in `counts` (the
// incremental M-step continues from those), and writes the means.  With R = 1, count_copies is
// `counts` itself.
__global__ void __launch_bounds__(256)
update_finish_kernel(long long* __restrict__ sum_lo, long long* __restrict__ sum_hi, const int* count_copies,
                     int* counts, int K, int g, int R, float* __restrict__ C) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    const int KG = K * g;
    if (e >= KG) return;
    const int j = e / g;
    long long lo = sum_lo[e], hi = sum_hi[e];
    int n = count_copies[j];
    if (R > 1) {
        for (int r = 1; r < R; ++r) {
            lo += sum_lo[(int64_t)r * KG + e];
            hi += sum_hi[(int64_t)r * KG + e];
            n += count_copies[(int64_t)r * K + j];
        }
        sum_lo[e] = lo;
        sum_hi[e] = hi;
        if (e == j * g) counts[j] = n;
    }
    if (n <= 0) return;   // empty cluster: previous centroid stays
    const double s = (double)lo * 5.9604644775390625e-8 + (double)hi * 0.0078125;
    C[e] = (float)(s / (double)n);
}

// Gradient with respect to the codebook: the exact integer sums as they are, rounded once to FP32.
__global__ void __launch_bounds__(256)
grad_finish_kernel(const long long* __restrict__ sum_lo, const long long* __restrict__ sum_hi, int n, int R,
                   float* __restrict__ dC) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    long long lo = 0, hi = 0;
    for (int r = 0; r < R; ++r) {
        lo += sum_lo[(int64_t)r * n + e];
        hi += sum_hi[(int64_t)r * n + e];
    }
    dC[e] = (float)((double)lo * 5.9604644775390625e-8 + (double)hi * 0.0078125);
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
cudaError_t launch_accumulate(int sm_count, const uint16_t* X, int64_t N, const uint16_t* idx, int K, ull* sum_lo,
                              ull* sum_hi, int32_t* counts, int R, cudaStream_t st) {
    int64_t blocks = (N * G + 255) / 256;
    const int64_t cap = (int64_t)sm_count * 16;
    if (blocks > cap) blocks = cap;
    update_accumulate_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, K, sum_lo, sum_hi, counts, R);
    return cudaGetLastError();
}

// The shared-memory kernel is used where all accumulators fit one SM and the point reductions it saves
// outnumber the words every block adds to the global accumulators at its end.
bool use_private(int64_t N, int K, int g, int sm_count) {
    if ((size_t)K * (8 * (size_t)g + 4) > (size_t)UP_SMEM) return false;
    return N >= 3 * (int64_t)sm_count * K;
}

template <int G>
cudaError_t launch_private(cc_ctx* ctx, const uint16_t* X, int64_t N, const uint16_t* idx, int K, ull* sum_lo, ull* sum_hi,
                           int32_t* counts, cudaStream_t st) {
    static bool attr_dev[64] = {};
    bool& attr = attr_dev[ctx->device & 63];
    if (!attr) {
        const cudaError_t e = cudaFuncSetAttribute(update_private_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, UP_SMEM);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    const size_t smem = (size_t)K * (8 * (size_t)G + 4);
    update_private_kernel<G><<<ctx->sm_count, UP_THREADS, smem, st>>>(X, N, idx, K, sum_lo, sum_hi, counts);
    return cudaGetLastError();
}

// Clears the R copies of the sums and counts and accumulates all points (R comes back as 1 when the
// shared-memory kernel ran: it keeps a single copy).  *count_copies is where the (copies of the)
// counts were accumulated: the caller's array when R = 1.
cudaError_t accumulate_all(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g, const uint16_t* idx,
                           int K, int32_t* counts, int& R, int32_t** count_copies, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    ull* sum_lo = reinterpret_cast<ull*>(ws + L.sum_lo);
    ull* sum_hi = reinterpret_cast<ull*>(ws + L.sum_hi);
    if (N > 0 && use_private(N, K, g, ctx->sm_count)) {
        // one copy of the accumulators; the blocks add their shared-memory sums to it
        R = 1;
        *count_copies = counts;
        const size_t words = sizeof(ull) * (size_t)K * g;
        cudaError_t e;
        if ((e = cudaMemsetAsync(sum_lo, 0, words, st)) != cudaSuccess) return e;
        if ((e = cudaMemsetAsync(sum_hi, 0, words, st)) != cudaSuccess) return e;
        if ((e = cudaMemsetAsync(counts, 0, sizeof(int32_t) * (size_t)K, st)) != cudaSuccess) return e;
        ProfScope ps(ctx, CC_K_UPDATE_ACCUM, st);
#define CALL(G) e = launch_private<G>(ctx, X, N, idx, K, sum_lo, sum_hi, counts, st)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
        return e;
    }
    int32_t* cc = R > 1 ? reinterpret_cast<int32_t*>(ws + L.count_copies) : counts;
    *count_copies = cc;
    const size_t used = sizeof(ull) * (size_t)K * g * R;
    cudaError_t e;
    if ((e = cudaMemsetAsync(sum_lo, 0, used, st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(sum_hi, 0, used, st)) != cudaSuccess) return e;
    if ((e = cudaMemsetAsync(cc, 0, sizeof(int32_t) * (size_t)K * R, st)) != cudaSuccess) return e;
    if (N > 0) {
        ProfScope ps(ctx, CC_K_UPDATE_ACCUM, st);
#define CALL(G) e = launch_accumulate<G>(ctx->sm_count, X, N, idx, K, sum_lo, sum_hi, cc, R, st)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
    }
    return e;
}

}  // namespace

cudaError_t cc_launch_update(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g, const uint16_t* idx,
                             int K, float* C, int32_t* counts, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    int R = cc_sum_copies(K, g);
    int32_t* count_copies = nullptr;
    const cudaError_t e = accumulate_all(ctx, L, X, N, g, idx, K, counts, R, &count_copies, st);
    if (e != cudaSuccess) return e;
    {
        ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
        update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(ws + L.sum_lo),
                                                                 reinterpret_cast<long long*>(ws + L.sum_hi),
                                                                 count_copies, counts, K, g, R, C);
    }
    if (ctx->empty_rule == CC_EMPTY_SPLIT_LARGEST) return cc_launch_split_empty(ctx, L, C, K, g, counts, st);
    return cudaGetLastError();
}

// dC[j] = sum of dX[i] over idx[i] = j, with the M-step's exact accumulation (scratch counts in the
// workspace: the position list of the initialisation is free by then).
cudaError_t cc_launch_codebook_grad(cc_ctx* ctx, const WsLayout& L, const uint16_t* dX, int64_t N, int g,
                                    const uint16_t* idx, int K, float* dC, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    int32_t* counts = reinterpret_cast<int32_t*>(ws + L.positions);
    int R = cc_sum_copies(K, g);
    int32_t* count_copies = nullptr;
    const cudaError_t e = accumulate_all(ctx, L, dX, N, g, idx, K, counts, R, &count_copies, st);
    if (e != cudaSuccess) return e;
    ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
    grad_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(ws + L.sum_lo),
                                                           reinterpret_cast<long long*>(ws + L.sum_hi), K * g, R, dC);
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
        ProfScope ps(ctx, CC_K_UPDATE_DELTA, st);
#define CALL(G) update_delta_kernel<G><<<(unsigned)blocks, 256, 0, st>>>(X, N, idx, idx_prev, K, sum_lo, sum_hi, counts)
        CC_UPDATE_DISPATCH(g, CALL)
#undef CALL
    }
    {
        ProfScope ps(ctx, CC_K_UPDATE_FINISH, st);
        update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                                 reinterpret_cast<long long*>(sum_hi), counts, counts, K,
                                                                 g, 1, C);
    }
    if (ctx->empty_rule == CC_EMPTY_SPLIT_LARGEST) return cc_launch_split_empty(ctx, L, C, K, g, counts, st);
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
        cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_accumulate<G>(sms, X, N, idx, K, sum_lo, sum_hi, counts, 1, st)
        switch (g) {
            case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;   case 4: CALL(4); break;
            case 5: CALL(5); break;   case 6: CALL(6); break;   case 7: CALL(7); break;   case 8: CALL(8); break;
            case 9: CALL(9); break;   case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;
            case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break; case 16: CALL(16); break;
            default: return CC_ERR_UNSUPPORTED_G;
        }
#undef CALL
        if (e != cudaSuccess) return CC_ERR_CUDA;
    }
    update_finish_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long*>(sum_lo),
                                                             reinterpret_cast<long long*>(sum_hi), counts, counts, K, g,
                                                             1, C);
    return cudaGetLastError() == cudaSuccess ? CC_OK : CC_ERR_CUDA;
}
