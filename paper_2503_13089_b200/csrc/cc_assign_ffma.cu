// E-step of Section 3.1 on the FP32 FMA pipes, plus the exact second stage and the
// objective sum that both E-step paths share.
//
// Fast stage.  For point x and centroid c the comparison score is
//     s = ||c||^2 - 2 x.c        (||x||^2 is the same for every centroid and dropped)
// computed as one FMA chain  s = fma(x_{g-1}, m_{g-1}, ... fma(x_0, m_0, csq))  with m = -2c and
// csq = ||c||^2 staged once per call.  Each thread keeps P points in registers and walks the staged
// codebook through shared memory; every shared-memory value is read by the whole warp at once (a
// broadcast).  For g <= 4 the FMAs are the packed two-wide form over pairs of centroids.  Only the running MINIMUM of the scores is kept
// in the inner loop (one 3-input min per two scores); the minimum is tracked per chunk of CHUNK
// centroids, together with the best and second-best chunk minima, and the winning chunk is
// rescanned once per point at the end to recover the index and the runner-up inside it.
//
// Exactness.  |s_computed - s| <= gamma_{g+1} (2||c||^2 + ||x||^2) with gamma_n ~ n 2^-24.  For any
// centroid at least as close as the fast winner b, ||c||^2 <= 2||x||^2 + 2 d_b^2, so if the gap
// between the two smallest computed scores exceeds 2 gamma (5||x||^2 + 4 d_b^2) the fast winner is
// the true nearest centroid.  Otherwise the point is appended to a list and decided again by the
// exact stage (FP64, direct form, lowest index on ties).  The N x K matrix is never stored.
#include <float.h>

#include "cc_common.cuh"
#include "cc_assign_shared.cuh"

namespace {

__device__ __forceinline__ ull pack2(float lo, float hi) {
    ull r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(ull v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// Two FP32 FMAs in one instruction (sm_100 packed form); each lane rounds like fma.rn.f32.
__device__ __forceinline__ ull fma2(ull a, ull b, ull c) {
    ull d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

constexpr int kThreads = 256;

// Per-g tiling.  PACKED: two-wide FMAs over pairs of centroids (each point's coordinates are held
// twice in a 64-bit register pair); otherwise scalar FMAs and twice as many points per thread.
// Either way a thread's points cost at most 64 registers.  A shared-memory load is a broadcast,
// but it still returns 512 bytes per warp, so the number of points per thread is what keeps the
// load pipe below the FMA pipes.
template <int G> struct FfmaCfg {
    static constexpr bool PACKED = (G <= 4);
    static constexpr int P_RAW = PACKED ? 32 / G : 64 / G;
    static constexpr int P = P_RAW > 16 ? 16 : (P_RAW < 4 ? 4 : (P_RAW & ~1));   // points per thread
    static constexpr int TILE = (G <= 4) ? 1024 : (G <= 8) ? 512 : 256;          // centroids per smem tile
    static constexpr int CHUNK = 32;                                             // centroids per tracked minimum
    static constexpr int ROW4 = G + 1;                                           // float4 per 4 centroids
    static constexpr int MIN_BLOCKS = (G <= 4) ? 2 : 1;                          // resident blocks per SM aimed at
};

// Staged codebook: for each group of four centroids j..j+3, G float4 {m_{j,t} .. m_{j+3,t}}
// (t = 0..G-1, m = -2c) followed by {csq_j .. csq_{j+3}}.  Centroids K..Kpad-1 are padding that
// can never win.
template <int G>
__global__ void prep_ffma_kernel(const float* __restrict__ C, int K, int Kpad, float4* __restrict__ prep,
                                 unsigned* __restrict__ status) {
    int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q == 0) {  // reset the flagged-point counter of this E-step
        *reinterpret_cast<ull*>(status + 2) = 0ull;
    }
    if (q >= Kpad / 4) return;
    float m[4][G], csq[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        int j = 4 * q + h;
        if (j < K) {
            double s = 0.0;
#pragma unroll
            for (int t = 0; t < G; ++t) {
                float c = C[(int64_t)j * G + t];
                m[h][t] = -2.0f * c;
                s += (double)c * (double)c;
            }
            csq[h] = (float)s;
        } else {
#pragma unroll
            for (int t = 0; t < G; ++t) m[h][t] = 0.f;
            csq[h] = kBig;
        }
    }
    float4* out = prep + (int64_t)q * (G + 1);
#pragma unroll
    for (int t = 0; t < G; ++t) out[t] = make_float4(m[0][t], m[1][t], m[2][t], m[3][t]);
    out[G] = make_float4(csq[0], csq[1], csq[2], csq[3]);
}

template <int G>
__global__ void __launch_bounds__(kThreads, FfmaCfg<G>::MIN_BLOCKS)
assign_ffma_kernel(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ C, int K, int Kpad,
                   const float4* __restrict__ prep, uint16_t* __restrict__ idx, float* __restrict__ dist,
                   unsigned* __restrict__ status, unsigned* __restrict__ flagged) {
    using Cfg = FfmaCfg<G>;
    constexpr int P = Cfg::P, TILE = Cfg::TILE, CHUNK = Cfg::CHUNK, ROW4 = Cfg::ROW4;
    constexpr bool PACKED = Cfg::PACKED;
    constexpr int TILE4 = TILE / 4 * ROW4;   // float4 per tile
    constexpr int STASH4 = P * kThreads * 2 * 4 / 32;   // float4 per buffer needed by the final stash
    constexpr int BUF4 = TILE4 > STASH4 ? TILE4 : STASH4;
    static_assert(2 * BUF4 * 16 <= 48 * 1024, "static shared memory limit");
    __shared__ float4 tiles[2][BUF4];

    const int tid = threadIdx.x;
    const int64_t base = (int64_t)blockIdx.x * (kThreads * P);

    // ---- points of this thread: point p is row base + p*kThreads + tid
    constexpr int XW = PACKED ? 2 : 1;
    float xs[P][G];          // scalar mode operands (also the source of the packed copies)
    ull xd[PACKED ? P : 1][PACKED ? G : 1];
    bool nonfinite = false;
#pragma unroll
    for (int p = 0; p < P; ++p) {
        load_point<G>(X, base + (int64_t)p * kThreads + tid, N, xs[p], nonfinite);
        if constexpr (PACKED) {
#pragma unroll
            for (int t = 0; t < G; ++t) xd[p][t] = pack2(xs[p][t], xs[p][t]);
        }
    }
    (void)XW;
    if (nonfinite) atomicOr(status, CC_DEV_NONFINITE);

    float b1[P], b2[P];
    int bc[P];
#pragma unroll
    for (int p = 0; p < P; ++p) { b1[p] = INFINITY; b2[p] = INFINITY; bc[p] = 0; }

    const int n_tiles = Kpad / TILE;
    for (int e = tid; e < TILE4; e += kThreads) cp_async16(&tiles[0][e], prep + e);
    cp_async_commit();

    for (int tile = 0; tile < n_tiles; ++tile) {
        cp_async_wait_all();
        __syncthreads();   // tile `tile` has landed for everyone; buffer (tile+1)&1 is free again
        if (tile + 1 < n_tiles) {
            const float4* src = prep + (int64_t)(tile + 1) * TILE4;
            float4* dst = tiles[(tile + 1) & 1];
            for (int e = tid; e < TILE4; e += kThreads) cp_async16(dst + e, src + e);
            cp_async_commit();
        }
        const float4* tbuf = tiles[tile & 1];
#pragma unroll 1
        for (int c = 0; c < TILE / CHUNK; ++c) {
            float m[P];
#pragma unroll
            for (int p = 0; p < P; ++p) m[p] = INFINITY;
            const float4* cp = tbuf + c * (CHUNK / 4) * ROW4;
#pragma unroll 2
            for (int q = 0; q < CHUNK / 4; ++q) {
                const float4* row = cp + q * ROW4;
                const float4 cs = row[G];
                if constexpr (PACKED) {
                    float4 mv[G];
#pragma unroll
                    for (int t = 0; t < G; ++t) mv[t] = row[t];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {          // centroids (j, j+1), then (j+2, j+3)
                        ull acc[P];
                        const ull cs2 = h ? pack2(cs.z, cs.w) : pack2(cs.x, cs.y);
#pragma unroll
                        for (int t = 0; t < G; ++t) {
                            const ull m2 = h ? pack2(mv[t].z, mv[t].w) : pack2(mv[t].x, mv[t].y);
#pragma unroll
                            for (int p = 0; p < P; ++p) acc[p] = fma2(xd[p][t], m2, t == 0 ? cs2 : acc[p]);
                        }
#pragma unroll
                        for (int p = 0; p < P; ++p) {
                            float a0, a1;
                            unpack2(acc[p], a0, a1);
                            m[p] = min3(m[p], a0, a1);
                        }
                    }
                } else {
                    float mv[G][4];
#pragma unroll
                    for (int t = 0; t < G; ++t) {
                        const float4 v = row[t];
                        mv[t][0] = v.x; mv[t][1] = v.y; mv[t][2] = v.z; mv[t][3] = v.w;
                    }
                    const float csv[4] = {cs.x, cs.y, cs.z, cs.w};
#pragma unroll
                    for (int h = 0; h < 2; ++h) {          // two centroids at a time
                        float a0[P], a1[P];
#pragma unroll
                        for (int t = 0; t < G; ++t) {
#pragma unroll
                            for (int p = 0; p < P; ++p) {
                                a0[p] = fmaf(xs[p][t], mv[t][2 * h], t == 0 ? csv[2 * h] : a0[p]);
                                a1[p] = fmaf(xs[p][t], mv[t][2 * h + 1], t == 0 ? csv[2 * h + 1] : a1[p]);
                            }
                        }
#pragma unroll
                        for (int p = 0; p < P; ++p) m[p] = min3(m[p], a0[p], a1[p]);
                    }
                }
            }
            const int chunk_id = tile * (TILE / CHUNK) + c;
#pragma unroll
            for (int p = 0; p < P; ++p) {
                const bool better = m[p] < b1[p];
                b2[p] = better ? b1[p] : fminf(b2[p], m[p]);
                bc[p] = better ? chunk_id : bc[p];
                b1[p] = better ? m[p] : b1[p];
            }
        }
    }
    __syncthreads();   // everyone is done with the tile buffers: reuse them as a stash

    float* stash = reinterpret_cast<float*>(&tiles[0][0]);
#pragma unroll
    for (int p = 0; p < P; ++p) {
        stash[(0 * P + p) * kThreads + tid] = b2[p];
        stash[(1 * P + p) * kThreads + tid] = __int_as_float(bc[p]);
    }
    // (each thread reads back only what it wrote: no barrier needed)

#pragma unroll 1
    for (int p = 0; p < P; ++p) {
        const int64_t i = base + (int64_t)p * kThreads + tid;
        if (i >= N) continue;
        const float second_other = stash[(0 * P + p) * kThreads + tid];
        const int chunk = __float_as_int(stash[(1 * P + p) * kThreads + tid]);
        finish_point<G, CHUNK>(X, N, C, K, prep, i, chunk, second_other, (double)(G + 2), idx, dist, status, flagged);
    }
}

// ---------------------------------------------------------------------------------------------
// Exact stage.  Every flagged point is scanned against every centroid again, the codebook being
// cut into S slices so that (point, slice) items fill the GPU whether few or many points are
// flagged (S is derived on the device from the number of flagged points; consecutive threads take
// consecutive points of the same slice, so a warp reads each centroid once for 32 points).
// A cheap FP32 direct-form distance (relative error <= (g+2) 2^-24, no cancellation) screens the
// candidates; those within 2^-18 of the best FP64 distance so far are recomputed in FP64 (sub,
// mul, add, in dimension order, no FMA contraction) and the pair (distance, index) is minimised
// lexicographically.  Each item starts from the fast stage's winner, writes its slice's result to
// scratch, and a second kernel merges the S results of a point (one warp per point).
struct ResolveEntry { double D; int j; int pad; };

__device__ __forceinline__ int resolve_slices(ull F, ull total_threads, int K, int64_t cap_entries) {
    ull S = (2 * total_threads + F - 1) / F;
    ull smax = (ull)(K >= 16 ? K / 8 : 1);
    if (smax > 256) smax = 256;
    const ull by_cap = (ull)cap_entries / F;
    if (smax > by_cap) smax = by_cap;
    if (S > smax) S = smax;
    return S < 1 ? 1 : (int)S;
}

template <int G>
__device__ __forceinline__ void load_centroid(const float* __restrict__ C, int j, float* c) {
    const float* row = C + (int64_t)j * G;
    if constexpr (G % 4 == 0) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            const float4 u = __ldg(reinterpret_cast<const float4*>(row) + v);
            c[4 * v] = u.x; c[4 * v + 1] = u.y; c[4 * v + 2] = u.z; c[4 * v + 3] = u.w;
        }
    } else {
#pragma unroll
        for (int t = 0; t < G; ++t) c[t] = __ldg(row + t);
    }
}

template <int G>
__global__ void __launch_bounds__(128)
resolve_scan_kernel(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ C, int K,
                    const unsigned* __restrict__ status, const unsigned* __restrict__ flagged,
                    ResolveEntry* __restrict__ scratch, int64_t cap_entries, uint16_t* __restrict__ idx,
                    float* __restrict__ dist) {
    ull F = *reinterpret_cast<const ull*>(status + 2);
    if (F > (ull)N) F = (ull)N;
    if (F == 0) return;
    const ull total_threads = (ull)gridDim.x * blockDim.x;
    const int S = resolve_slices(F, total_threads, K, cap_entries);
    const int L = (K + S - 1) / S;
    const ull items = F * (ull)S;
    for (ull item = (ull)blockIdx.x * blockDim.x + threadIdx.x; item < items; item += total_threads) {
        const int sl = (int)(item / F);
        const ull f = item - (ull)sl * F;
        const int64_t i = flagged[f];
        float x[G];
        bool nf = false;
        load_point<G>(X, i, N, x, nf);
        int jb = idx[i];
        double Db = 0.0;
#pragma unroll
        for (int t = 0; t < G; ++t) {
            const double df = __dsub_rn((double)x[t], (double)__ldg(C + (int64_t)jb * G + t));
            Db = __dadd_rn(Db, __dmul_rn(df, df));
        }
        float bound = __double2float_ru(Db * (1.0 + 3.814697265625e-6));
        const int j_end = (sl + 1) * L < K ? (sl + 1) * L : K;
        // four centroids per round: their screening distances are independent chains, and only a round that
        // holds a candidate looks closer
        int j = sl * L;
        for (; j + 4 <= j_end; j += 4) {
            float dq[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float c[G];
                load_centroid<G>(C, j + q, c);
                dq[q] = 0.f;
#pragma unroll
                for (int t = 0; t < G; ++t) { const float df = x[t] - c[t]; dq[q] = fmaf(df, df, dq[q]); }
            }
            if (fminf(fminf(dq[0], dq[1]), fminf(dq[2], dq[3])) > bound) continue;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (dq[q] <= bound) {
                    float c[G];
                    load_centroid<G>(C, j + q, c);
                    double d = 0.0;
#pragma unroll
                    for (int t = 0; t < G; ++t) {
                        const double df = __dsub_rn((double)x[t], (double)c[t]);
                        d = __dadd_rn(d, __dmul_rn(df, df));
                    }
                    if (d < Db || (d == Db && j + q < jb)) {
                        Db = d; jb = j + q;
                        bound = __double2float_ru(Db * (1.0 + 3.814697265625e-6));
                    }
                }
            }
        }
        for (; j < j_end; ++j) {
            float c[G];
            load_centroid<G>(C, j, c);
            float dh = 0.f;
#pragma unroll
            for (int t = 0; t < G; ++t) { const float df = x[t] - c[t]; dh = fmaf(df, df, dh); }
            if (dh <= bound) {
                double d = 0.0;
#pragma unroll
                for (int t = 0; t < G; ++t) {
                    const double df = __dsub_rn((double)x[t], (double)c[t]);
                    d = __dadd_rn(d, __dmul_rn(df, df));
                }
                if (d < Db || (d == Db && j < jb)) {
                    Db = d; jb = j;
                    bound = __double2float_ru(Db * (1.0 + 3.814697265625e-6));
                }
            }
        }
        if (S == 1) {            // one item per point: nothing to merge
            idx[i] = (uint16_t)jb;
            dist[i] = (float)Db;
        } else {
            ResolveEntry e;
            e.D = Db; e.j = jb; e.pad = 0;
            scratch[(ull)sl * F + f] = e;
        }
    }
}

__global__ void __launch_bounds__(128)
resolve_merge_kernel(int64_t N, int K, const unsigned* __restrict__ status, const unsigned* __restrict__ flagged,
                     const ResolveEntry* __restrict__ scratch, int64_t cap_entries, ull scan_threads,
                     uint16_t* __restrict__ idx, float* __restrict__ dist) {
    ull F = *reinterpret_cast<const ull*>(status + 2);
    if (F > (ull)N) F = (ull)N;
    if (F == 0) return;
    const int S = resolve_slices(F, scan_threads, K, cap_entries);
    if (S == 1) return;
    const int lane = threadIdx.x & 31;
    const ull n_warps = ((ull)gridDim.x * blockDim.x) >> 5;
    for (ull f = ((ull)blockIdx.x * blockDim.x + threadIdx.x) >> 5; f < F; f += n_warps) {
        double Db = INFINITY;
        int jb = 0x7fffffff;
        for (int sl = lane; sl < S; sl += 32) {
            const ResolveEntry e = scratch[(ull)sl * F + f];
            if (e.D < Db || (e.D == Db && e.j < jb)) { Db = e.D; jb = e.j; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double Do = __shfl_xor_sync(0xffffffffu, Db, o);
            const int jo = __shfl_xor_sync(0xffffffffu, jb, o);
            if (Do < Db || (Do == Db && jo < jb)) { Db = Do; jb = jo; }
        }
        if (lane == 0) {
            const int64_t i = flagged[f];
            idx[i] = (uint16_t)jb;
            dist[i] = (float)Db;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Objective: sum of dist in FP64 with a fixed summation tree (same bits on every run).
__device__ __forceinline__ double block_sum(double v, double* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    if (l == 0) sh[w] = v;
    __syncthreads();
    double r = 0.0;
    if (w == 0) {
        r = (l < (blockDim.x >> 5)) ? sh[l] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r += __shfl_down_sync(0xffffffffu, r, o);
    }
    return r;   // valid in thread 0
}

// One kernel: every block writes the FP64 sum of its slice of dist; the block that finishes last
// (a ticket in status word 8, left at zero again) adds the partial sums in a fixed order, so the
// result does not depend on which block that is.
__global__ void __launch_bounds__(256)
objective_kernel(const float* __restrict__ dist, int64_t N, double* __restrict__ partials, unsigned* __restrict__ status,
                 double* __restrict__ objective, int64_t* __restrict__ n_resolved) {
    __shared__ double sh[8];
    __shared__ bool last;
    const int64_t per = (N + gridDim.x - 1) / gridDim.x;
    const int64_t lo = (int64_t)blockIdx.x * per;
    const int64_t hi = (lo + per < N) ? lo + per : N;
    double acc = 0.0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) acc += (double)dist[i];
    const double r = block_sum(acc, sh);
    if (threadIdx.x == 0) {
        partials[blockIdx.x] = r;
        __threadfence();
        last = atomicAdd(status + 8, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!last) return;
    __threadfence();
    double tot = 0.0;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += blockDim.x) tot += __ldcg(partials + i);
    const double t = block_sum(tot, sh);
    if (threadIdx.x == 0) {
        if (objective) *objective = t;
        if (n_resolved) *n_resolved = (int64_t)*reinterpret_cast<const ull*>(status + 2);
        status[8] = 0u;
    }
}

template <int G>
cudaError_t launch_prep(cc_ctx* ctx, const WsLayout& L, const float* C, int K, cudaStream_t st);

template <int G>
cudaError_t launch_ffma(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, const float* C, int K,
                        uint16_t* idx, float* dist, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    unsigned* status = reinterpret_cast<unsigned*>(ws + L.status);
    float4* prep = reinterpret_cast<float4*>(ws + L.cprep);
    unsigned* flagged = reinterpret_cast<unsigned*>(ws + L.flagged);
    const int Kpad = (int)cc_align_up((size_t)K, CC_KPAD);
    launch_prep<G>(ctx, L, C, K, st);
    if (N > 0) {
        const int64_t per_block = (int64_t)kThreads * FfmaCfg<G>::P;
        const int64_t blocks = (N + per_block - 1) / per_block;
        ProfScope ps(ctx, CC_K_ASSIGN_MAIN, st);
        assign_ffma_kernel<G><<<(unsigned)blocks, kThreads, 0, st>>>(X, N, C, K, Kpad, prep, idx, dist, status,
                                                                     flagged);
    }
    return cudaGetLastError();
}

template <int G>
cudaError_t launch_tail(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, const float* C, int K,
                        uint16_t* idx, float* dist, double* objective, int64_t* n_resolved, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    unsigned* status = reinterpret_cast<unsigned*>(ws + L.status);
    unsigned* flagged = reinterpret_cast<unsigned*>(ws + L.flagged);
    double* partials = reinterpret_cast<double*>(ws + L.partials);
    if (N > 0) {
        // scratch of the exact stage: the tensor scan's per-point state, free again by now
        ResolveEntry* scratch = reinterpret_cast<ResolveEntry*>(ws + L.tstate);
        const int64_t cap_entries = N / 2 > 0 ? N / 2 : 1;
        const int blocks = ctx->sm_count * 16;
        {
            ProfScope ps(ctx, CC_K_RESOLVE, st);
            resolve_scan_kernel<G><<<blocks, 128, 0, st>>>(X, N, C, K, status, flagged, scratch, cap_entries, idx, dist);
        }
        ProfScope ps(ctx, CC_K_RESOLVE, st);
        resolve_merge_kernel<<<blocks, 128, 0, st>>>(N, K, status, flagged, scratch, cap_entries, (ull)blocks * 128, idx, dist);
    }
    if (objective || n_resolved) {
        int blocks = (int)((N + 4095) / 4096);
        if (blocks > CC_OBJ_BLOCKS) blocks = CC_OBJ_BLOCKS;
        if (blocks < 1) blocks = 1;
        ProfScope ps(ctx, CC_K_OBJECTIVE, st);
        objective_kernel<<<blocks, 256, 0, st>>>(dist, N, partials, status, objective, n_resolved);
    }
    return cudaGetLastError();
}

template <int G>
cudaError_t launch_prep(cc_ctx* ctx, const WsLayout& L, const float* C, int K, cudaStream_t st) {
    char* ws = static_cast<char*>(ctx->ws);
    const int Kpad = (int)cc_align_up((size_t)K, CC_KPAD);
    ProfScope ps(ctx, CC_K_ASSIGN_PREP, st);
    prep_ffma_kernel<G><<<(Kpad / 4 + 127) / 128, 128, 0, st>>>(C, K, Kpad, reinterpret_cast<float4*>(ws + L.cprep),
                                                                reinterpret_cast<unsigned*>(ws + L.status));
    return cudaGetLastError();
}

}  // namespace

#define CC_DISPATCH_G(g, CALL)                                                                      \
    switch (g) {                                                                                    \
        case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;                 \
        case 4: CALL(4); break;   case 5: CALL(5); break;   case 6: CALL(6); break;                 \
        case 7: CALL(7); break;   case 8: CALL(8); break;   case 9: CALL(9); break;                 \
        case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;               \
        case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break;               \
        case 16: CALL(16); break;                                                                   \
        default: return cudaErrorInvalidValue;                                                      \
    }

cudaError_t cc_launch_assign_tail(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                  const float* C, int K, uint16_t* idx, float* dist, double* objective,
                                  int64_t* n_resolved, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_tail<G>(ctx, L, X, N, C, K, idx, dist, objective, n_resolved, st)
    CC_DISPATCH_G(g, CALL)
#undef CALL
    return e;
}

cudaError_t cc_launch_assign_ffma(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                  const float* C, int K, uint16_t* idx, float* dist, double* objective,
                                  int64_t* n_resolved, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_ffma<G>(ctx, L, X, N, C, K, idx, dist, st)
    CC_DISPATCH_G(g, CALL)
#undef CALL
    if (e != cudaSuccess) return e;
    return cc_launch_assign_tail(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, st);
}

cudaError_t cc_launch_prep_ffma(cc_ctx* ctx, const WsLayout& L, int g, const float* C, int K, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_prep<G>(ctx, L, C, K, st)
    CC_DISPATCH_G(g, CALL)
#undef CALL
    return e;
}
