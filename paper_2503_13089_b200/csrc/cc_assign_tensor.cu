// E-step of Section 3.1 on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
// The score matrix S = ||c||^2 - 2 x.c of a tile of 128 points x 256 centroids is one dense
// contraction  S = A . B^T  with
//     A row (point i)    = [ x , x (, x) , 1 , 1 , 1 , 0.. ]
//     B row (centroid j) = [ m1, m2 (, m3), q1, q2, q3, 0.. ],   m = -2c = m1 + m2 (+ m3),
// where the FP32 centroid is split into TF32 pieces (three pieces = exact, two pieces = 2^-22
// relative) and q1 + q2 + q3 is ||c||^2 (computed in FP64) to 33 bits.  FP16 points are exact in
// TF32.  `tcgen05.mma.kind::tf32` accumulates in FP32 in tensor memory; operands sit in shared
// memory in the canonical K-major layout without swizzle (8-row x 16-byte core matrices).
//
// One CTA keeps NA tiles of 128 points (the A operand) resident in shared memory and streams the
// whole staged codebook (B tiles of 256 centroids, written by the prep kernel in the exact
// shared-memory image so that one 1-D bulk copy fetches a tile) through a 2-stage ring.
// Warp roles: 8 epilogue warps (warp w reads TMEM lanes 32*(w%4).., columns 128*(w/4)..),
// one copy warp, one MMA warp (a single thread issues the MMAs).  The epilogue only takes the
// running minimum of each 64-centroid chunk (3-input min) and keeps best / second-best chunk
// minimum and the best chunk id per point; the index inside the chunk, the distance and the
// near-tie flag are computed afterwards by the finish kernel, exactly as in the FP32 path.
// Nothing N x K is ever written to memory.
//
// Every wait on an mbarrier is bounded (clock based); on a time-out the CTA raises the status
// bit CC_DEV_TIMEOUT, stops issuing work, and still releases its tensor memory.
#include "cc_common.cuh"
#include "cc_assign_shared.cuh"

namespace {

constexpr int TM = 128;            // points per MMA = TMEM lanes
constexpr int TN = 256;            // centroids per MMA = TMEM columns of one accumulator
constexpr int TCHUNK = 64;         // centroids per tracked minimum
constexpr int EPI_WARPS = 8;
constexpr int TC_THREADS = (EPI_WARPS + 2) * 32;
constexpr int STAGES = 2;
constexpr long long WAIT_LIMIT = 4000000000LL;   // clock cycles (about 2 s)

template <int G> struct TcCfg {
    static constexpr int SPLIT = (G <= 4) ? 3 : 2;                 // TF32 pieces of each centroid value
    static constexpr int KD = (SPLIT * G + 3 + 7) / 8 * 8;          // contraction length, multiple of 8
    static constexpr int A_TILE = TM * KD * 4;                      // bytes
    static constexpr int B_TILE = TN * KD * 4;
    // resident point tiles / TMEM accumulators: small g runs two CTAs per SM with one accumulator
    // each, large g one CTA per SM with two accumulators
    static constexpr int NA = (G <= 4) ? 8 : 4;
    static constexpr int SLOTS = (G <= 8) ? 1 : 2;
    static constexpr int MIN_BLOCKS = (G <= 8) ? 2 : 1;
    static constexpr int SMEM = NA * A_TILE + STAGES * B_TILE + 256;
    // rounding model of the scan: 2^-24 units of (2||c||^2 + ||x||^2); see the finish kernel
    static constexpr int ERR_UNITS = (SPLIT == 3) ? 16 : 40;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Offset (in floats) of element (row r, k) of an R-row operand in the canonical K-major layout.
__device__ __forceinline__ int canon_off(int r, int k, int R) {
    return (k >> 2) * (R * 4) + (r >> 3) * 32 + (r & 7) * 4 + (k & 3);
}

__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;   // between the two core matrices along K
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;   // between 8-row groups
    d |= (uint64_t)1 << 46;                             // descriptor version of sm_100
    return d;                                           // layout type 0: no swizzle
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false when the CTA is aborting (this or another waiter timed out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (unsigned spin = 1;; ++spin) {
        if (mbar_try(bar, parity)) return true;
        if ((spin & 255u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_LIMIT) { *abort_flag = 1; return false; }
        }
    }
}

__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ float tf32_trunc(float f) { return __uint_as_float(__float_as_uint(f) & 0xffffe000u); }
__device__ __forceinline__ float tf32_round(float f) {
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(f));
    return __uint_as_float(u & 0xffffe000u);
}

// Staged B operand: tile b holds centroids 256b .. 256b+255 in the canonical layout, KD floats per
// centroid: SPLIT x G pieces of m = -2c, three pieces of ||c||^2, zeros.  One thread writes four
// consecutive k of one centroid (16 bytes).
template <int G>
__global__ void prep_tensor_kernel(const float* __restrict__ C, int K, int Kpad, float* __restrict__ gB) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, SPLIT = Cfg::SPLIT;
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= Kpad * (KD / 4)) return;
    const int j = e / (KD / 4), kc = e - j * (KD / 4);
    float out[4];
    float q[3] = {kBig, 0.f, 0.f};
    if (j < K) {
        double s = 0.0;
#pragma unroll
        for (int t = 0; t < G; ++t) { const double c = (double)C[(int64_t)j * G + t]; s += c * c; }
        q[0] = tf32_trunc((float)s);
        const double r1 = s - (double)q[0];
        q[1] = tf32_trunc((float)r1);
        q[2] = tf32_round((float)(r1 - (double)q[1]));
    } else {
        q[0] = tf32_trunc(kBig);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int k = kc * 4 + u;
        float v = 0.f;
        if (k < SPLIT * G) {
            if (j < K) {
                const int piece = k / G, t = k - piece * G;
                const float m = -2.0f * C[(int64_t)j * G + t];
                const float m1 = tf32_trunc(m);
                const float r1 = m - m1;                       // exact in FP32
                if (piece == 0) v = m1;
                else if (SPLIT == 2) v = tf32_round(r1);
                else {
                    const float m2 = tf32_trunc(r1);
                    v = (piece == 1) ? m2 : (r1 - m2);         // at most 2 bits left: exact in TF32
                }
            }
        } else if (k < SPLIT * G + 3) {
            v = q[k - SPLIT * G];
        }
        out[u] = v;
    }
    const int tile = j / TN, jr = j - tile * TN;
    float* dst = gB + (int64_t)tile * (TN * KD) + canon_off(jr, kc * 4, TN);
    *reinterpret_cast<float4*>(dst) = make_float4(out[0], out[1], out[2], out[3]);
}

#define TMEM_LD32(v, taddr)                                                                                      \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                       \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                       \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                      \
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),  \
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]),      \
                   "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]),    \
                   "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]),    \
                   "=r"(v[29]), "=r"(v[30]), "=r"(v[31])                                                         \
                 : "r"(taddr))
// The loaded registers are only valid after the wait; naming them as in/out operands keeps the
// compiler from moving their uses above it.
#define TMEM_WAIT32(v)                                                                                           \
    asm volatile("tcgen05.wait::ld.sync.aligned;"                                                                \
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),  \
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]),      \
                   "+r"(v[15]), "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]),    \
                   "+r"(v[22]), "+r"(v[23]), "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]),    \
                   "+r"(v[29]), "+r"(v[30]), "+r"(v[31])                                                         \
                 :: "memory")

template <int G>
__global__ void __launch_bounds__(TC_THREADS, TcCfg<G>::MIN_BLOCKS)
assign_tensor_kernel(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ gB, int n_btiles,
                     float2* __restrict__ tstate, unsigned* __restrict__ status) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, NA = Cfg::NA, SLOTS = Cfg::SLOTS, SPLIT = Cfg::SPLIT;
    constexpr int A_FLOATS = TM * KD, B_FLOATS = TN * KD;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    float* sA = reinterpret_cast<float*>(smem_raw);                       // NA tiles
    float* sB = sA + NA * A_FLOATS;                                       // STAGES tiles
    uint64_t* bars = reinterpret_cast<uint64_t*>(sB + STAGES * B_FLOATS); // b_full, b_empty, t_full, t_empty
    uint64_t* b_full = bars, *b_empty = bars + STAGES, *t_full = bars + 2 * STAGES, *t_empty = bars + 2 * STAGES + SLOTS;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2 * SLOTS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t base = (int64_t)blockIdx.x * (NA * TM);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_empty + s)));
        }
        for (int s = 0; s < SLOTS; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(t_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(t_empty + s)), "r"(EPI_WARPS));
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // ---- A operand: [x repeated SPLIT times, 1, 1, 1, 0..] per point, written 16 bytes at a time
    bool nonfinite = false;
    for (int e = tid; e < NA * TM; e += TC_THREADS) {
        float x[G];
        load_point<G>(X, base + e, N, x, nonfinite);
        float* tile = sA + (e / TM) * A_FLOATS;
        const int r = e % TM;
#pragma unroll
        for (int kc = 0; kc < KD / 4; ++kc) {
            float v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int k = kc * 4 + u;
                v[u] = (k < SPLIT * G) ? x[k % G] : (k < SPLIT * G + 3 ? 1.0f : 0.0f);
            }
            *reinterpret_cast<float4*>(tile + canon_off(r, kc * 4, TM)) = make_float4(v[0], v[1], v[2], v[3]);
        }
    }
    if (nonfinite) atomicOr(status, CC_DEV_NONFINITE);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> async proxy (MMA)
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(SLOTS * TN));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp == EPI_WARPS) {
        // ------------------------------------------------------------ copy warp: B tiles -> ring
        if (lane == 0) {
            int issued = 0;
            for (int b = 0; b < n_btiles; ++b) {
                const int st = b % STAGES;
                if (!mbar_wait(smem_u32(b_empty + st), ((b / STAGES) & 1) ^ 1, abort_flag)) break;
                const uint32_t bar = smem_u32(b_full + st);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(Cfg::B_TILE) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(sB + st * B_FLOATS)), "l"(gB + (int64_t)b * B_FLOATS), "r"(Cfg::B_TILE), "r"(bar)
                             : "memory");
                issued = b + 1;
            }
            if (*abort_flag) {   // let the copies in flight land before the CTA exits (bounded)
                for (int b = (issued > STAGES ? issued - STAGES : 0); b < issued; ++b) {
                    const long long t0 = clock64();
                    while (!mbar_try(smem_u32(b_full + b % STAGES), (b / STAGES) & 1) && clock64() - t0 < WAIT_LIMIT) {}
                }
            }
        }
    } else if (warp == EPI_WARPS + 1) {
        // ------------------------------------------------------------ MMA warp: one thread issues
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
            bool ok = true;
            for (int b = 0; b < n_btiles && ok; ++b) {
                const int st = b % STAGES;
                ok = mbar_wait(smem_u32(b_full + st), (b / STAGES) & 1, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t bBase = smem_u32(sB + st * B_FLOATS);
                for (int a = 0; a < NA; ++a) {
                    const int q = b * NA + a, slot = q % SLOTS;
                    ok = mbar_wait(smem_u32(t_empty + slot), ((q / SLOTS) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t aBase = smem_u32(sA + a * A_FLOATS);
                    const uint32_t d = tmem + slot * TN;
#pragma unroll
                    for (int s = 0; s < KD / 8; ++s) {
                        const uint64_t da = make_desc(aBase + s * 2 * (TM * 16), TM * 16, 128);
                        const uint64_t db = make_desc(bBase + s * 2 * (TN * 16), TN * 16, 128);
                        const uint32_t acc = s > 0 ? 1u : 0u;
                        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                                     ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
                    }
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(smem_u32(t_full + slot)) : "memory");
                }
                if (ok)   // the ring stage may be refilled once these MMAs have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(smem_u32(b_empty + st)) : "memory");
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3, half = warp >> 2;
        float b1[NA], b2[NA];
        int bc[NA];
#pragma unroll
        for (int a = 0; a < NA; ++a) { b1[a] = INFINITY; b2[a] = INFINITY; bc[a] = half * 2; }
        bool ok = true;
        for (int b = 0; b < n_btiles && ok; ++b) {
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                if (!ok) continue;
                const int q = b * NA + a, slot = q % SLOTS;
                ok = mbar_wait(smem_u32(t_full + slot), (q / SLOTS) & 1, abort_flag);
                if (!ok) continue;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t t0 = tmem + ((uint32_t)(quarter * 32) << 16) + slot * TN + half * (TN / 2);
#pragma unroll
                for (int c = 0; c < (TN / 2) / TCHUNK; ++c) {
                    float m0 = INFINITY, m1 = INFINITY, m2 = INFINITY, m3 = INFINITY;
#pragma unroll
                    for (int l = 0; l < TCHUNK / 32; ++l) {
                        uint32_t v[32];
                        TMEM_LD32(v, t0 + c * TCHUNK + l * 32);
                        TMEM_WAIT32(v);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            m0 = min3(m0, __uint_as_float(v[8 * u + 0]), __uint_as_float(v[8 * u + 1]));
                            m1 = min3(m1, __uint_as_float(v[8 * u + 2]), __uint_as_float(v[8 * u + 3]));
                            m2 = min3(m2, __uint_as_float(v[8 * u + 4]), __uint_as_float(v[8 * u + 5]));
                            m3 = min3(m3, __uint_as_float(v[8 * u + 6]), __uint_as_float(v[8 * u + 7]));
                        }
                    }
                    const float m = fminf(min3(m0, m1, m2), m3);
                    const int chunk_id = b * (TN / TCHUNK) + half * ((TN / 2) / TCHUNK) + c;
                    const bool better = m < b1[a];
                    b2[a] = better ? b1[a] : fminf(b2[a], m);
                    bc[a] = better ? chunk_id : bc[a];
                    b1[a] = better ? m : b1[a];
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0)
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(t_empty + slot)) : "memory");
            }
        }
        // ---- merge the two column halves of each point (through the A region, no longer read by
        //      any MMA: the last accumulator was complete before its epilogue started) and store
        asm volatile("bar.sync 1, %0;" ::"r"(EPI_WARPS * 32));
        float* merge = sA;   // [NA][TM][3]
        const int r = quarter * 32 + lane;
        if (half == 1) {
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                merge[(a * TM + r) * 3 + 0] = b1[a];
                merge[(a * TM + r) * 3 + 1] = b2[a];
                merge[(a * TM + r) * 3 + 2] = __int_as_float(bc[a]);
            }
        }
        asm volatile("bar.sync 1, %0;" ::"r"(EPI_WARPS * 32));
        if (half == 0 && ok && !*abort_flag) {
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                const int64_t i = base + a * TM + r;
                if (i >= N) continue;
                const float o1 = merge[(a * TM + r) * 3 + 0], o2 = merge[(a * TM + r) * 3 + 1];
                const int oc = __float_as_int(merge[(a * TM + r) * 3 + 2]);
                float second;
                int chunk;
                if (o1 < b1[a] || (o1 == b1[a] && oc < bc[a])) { chunk = oc; second = fminf(o2, b1[a]); }
                else { chunk = bc[a]; second = fminf(b2[a], o1); }
                tstate[i] = make_float2(second, __int_as_float(chunk));
            }
        }
    }
    if (*abort_flag && lane == 0) atomicOr(status, CC_DEV_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(SLOTS * TN));
}

// Finish: index inside the winning chunk, distance, near-tie flag (shared with the FP32 path).
template <int G>
__global__ void __launch_bounds__(256)
finish_tensor_kernel(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ C, int K,
                     const float4* __restrict__ prep, const float2* __restrict__ tstate, uint16_t* __restrict__ idx,
                     float* __restrict__ dist, unsigned* __restrict__ status, unsigned* __restrict__ flagged) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const float2 t = tstate[i];
    finish_point<G, TCHUNK>(X, N, C, K, prep, i, __float_as_int(t.y), t.x, (double)TcCfg<G>::ERR_UNITS, idx, dist,
                            status, flagged);
}

template <int G>
cudaError_t launch_tensor(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, const float* C, int K,
                          uint16_t* idx, float* dist, cudaStream_t st) {
    using Cfg = TcCfg<G>;
    char* ws = static_cast<char*>(ctx->ws);
    unsigned* status = reinterpret_cast<unsigned*>(ws + L.status);
    float* gB = reinterpret_cast<float*>(ws + L.tensor);
    float2* tstate = reinterpret_cast<float2*>(ws + L.tstate);
    const int Kpad = (int)cc_align_up((size_t)K, TN);
    cudaError_t e = cc_launch_prep_ffma(ctx, L, G, C, K, st);   // staged codebook of the finish kernel; resets the flag counter
    if (e != cudaSuccess) return e;
    {
        ProfScope ps(ctx, CC_K_ASSIGN_PREP, st);
        const int n = Kpad * (Cfg::KD / 4);
        prep_tensor_kernel<G><<<(n + 255) / 256, 256, 0, st>>>(C, K, Kpad, gB);
    }
    if (N > 0) {
        static bool attr_set = false;
        if (!attr_set) {
            e = cudaFuncSetAttribute(assign_tensor_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
            if (e != cudaSuccess) return e;
            attr_set = true;
        }
        const int64_t per_block = (int64_t)Cfg::NA * TM;
        const int64_t blocks = (N + per_block - 1) / per_block;
        {
            ProfScope ps(ctx, CC_K_ASSIGN_MAIN, st);
            assign_tensor_kernel<G><<<(unsigned)blocks, TC_THREADS, Cfg::SMEM, st>>>(X, N, gB, Kpad / TN, tstate, status);
        }
        {
            ProfScope ps(ctx, CC_K_ASSIGN_FINISH, st);
            finish_tensor_kernel<G><<<(unsigned)((N + 255) / 256), 256, 0, st>>>(
                X, N, C, K, reinterpret_cast<const float4*>(ws + L.cprep), tstate, idx, dist, status,
                reinterpret_cast<unsigned*>(ws + L.flagged));
        }
    }
    return cudaGetLastError();
}

}  // namespace

bool cc_tensor_path_supported(int g, int K) {
    (void)K;
    return g == 4 || g == 8 || g == 16;
}

cudaError_t cc_launch_assign_tensor(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                    const float* C, int K, uint16_t* idx, float* dist, double* objective,
                                    int64_t* n_resolved, cudaStream_t st) {
    cudaError_t e;
    switch (g) {
        case 4: e = launch_tensor<4>(ctx, L, X, N, C, K, idx, dist, st); break;
        case 8: e = launch_tensor<8>(ctx, L, X, N, C, K, idx, dist, st); break;
        case 16: e = launch_tensor<16>(ctx, L, X, N, C, K, idx, dist, st); break;
        default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
    return cc_launch_assign_tail(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, st);
}
