// E-step of Section 3.1 on the 5th-generation tensor cores (tcgen05, accumulators in TMEM).
//
// The score matrix  S s_ij = S (||c_j||^2 - 2 x_i.c_j)  of a tile of 128 points x 256 centroids is
// one dense FP16 contraction  A . B^T  with FP32 accumulation:
//     A row (point i)    = [ x , x (, x) , 2^15, 2^6, 2^-3, 2^-12, 0.. ]
//     B row (centroid j) = [ h1, h2 (, h3), p1 , p2 , p3  , p4   , 0.. ]
// x is FP16 data and therefore exact.  S is a power of two chosen per call so that
// |S m| < 2^15 and S ||c||^2 < 2^30 for every centroid (m = -2c); S m = h1 + h2 + h3 is the FP32
// value cut into FP16 pieces (each piece is the FP16 rounding of what is left), and
// S ||c||^2 (from FP64) = 2^15 p1 + 2^6 p2 + 2^-3 p3 + 2^-12 p4 likewise.  Scaling by a power of
// two changes neither the order of the scores nor their rounding.  Where it shortens the contraction
// (g = 5, 6, 7: 16 columns; g = 10..15: 32) or is needed to fit 48 columns (g = 16), m is cut into two
// pieces only (relative residue 2^-22); for g = 7 and 15 the norm is cut into two pieces as well,
// S ||c||^2 = 2^e p1 + 2^(e-11) p2 with e fitted to the largest norm of the call.
//
// Subnormal pieces are never emitted: the tensor core adds the products of one instruction after
// aligning them by the operands' exponent FIELDS, so a subnormal piece next to the constant 2^15
// widens the alignment window and costs the other addends their low bits (measured: an absolute
// error of 2^-22 in scaled units).  A piece below 2^-14 is written as zero instead and the next,
// finer piece picks the residue up; what is lost in the end is below 2^-14 per coordinate of S m
// and below 2^-26 on S ||c||^2, and the near-tie test accounts for both.  Subnormal coordinates
// of x itself are multiplied exactly (measured) but count with magnitude 2^-14 in that test.
//
// One CTA keeps up to NA tiles of 128 points (the A operand) resident in shared memory and
// streams the staged codebook (B tiles of 256 centroids, written by the prep kernel as the exact
// shared-memory image so that one bulk copy fetches a tile) through a ring.  Warp roles:
// 16 epilogue warps (warp e reads TMEM lanes 32 (e % 4).., columns 64 (e / 4)..), one copy warp,
// one MMA warp (a single thread issues the MMAs).  Two accumulators of 256 columns alternate, so
// the tensor core fills one while the epilogue drains the other; a warp releases its share of
// an accumulator as soon as its 64 columns are in registers.  The epilogue keeps, per point, the
// smallest and second-smallest 64-centroid chunk minimum and the id of the best chunk (one
// 3-input min per two scores); the index inside the chunk, the distance and the near-tie flag are
// computed afterwards by the finish kernel from FP32 data.  Nothing N x K is written to memory.
// Three instantiations share this structure: a persistent kernel (g <= 15: one CTA per SM walks over
// groups of NA point tiles while an extra warp builds the next group's A operand), a one-group-per-
// CTA kernel specialised for full groups (g = 16), and a generic one for the ragged rest and for
// small inputs.
//
// Every wait on an mbarrier is bounded (clock based); on a time-out the CTA raises the status
// bit CC_DEV_TIMEOUT, stops issuing work, and still releases its tensor memory.
#include <cuda_fp16.h>

#include "cc_common.cuh"
#include "cc_assign_shared.cuh"
#include "cc_tcgen05.cuh"

namespace {

constexpr int TM = 128;            // points per MMA = TMEM lanes
constexpr int TN = 256;            // centroids per MMA = TMEM columns of one accumulator
constexpr int TCHUNK = 64;         // centroids per tracked minimum = columns per epilogue warp
constexpr int EW = TN / TCHUNK;    // epilogue warps per TMEM lane quarter
constexpr int EPI_WARPS = 4 * EW;
constexpr int TC_THREADS = (EPI_WARPS + 2) * 32;
constexpr int SLOTS = 2;           // accumulators in TMEM
constexpr int NA = 8;              // resident point tiles per CTA
constexpr int LPP = 8;             // lanes per point in the finish kernel

template <int G> struct TcCfg {
    // FP16 pieces of each S m value (SPLIT) and of S ||c||^2 (NQ).  Default three and four; fewer
    // where that makes the contraction shorter or is needed to fit 48 columns:
    //   two pieces of m (relative residue 2^-22): g = 5, 6 (16 instead of 32 columns), g = 10..14 (32
    //   instead of 48), g = 16;
    //   two pieces of m and two of the norm: g = 7 (16 columns), g = 15 (32 columns).  The two norm
    //   pieces multiply constants 2^e and 2^(e-11) with e fitted to the largest norm of the call
    //   (norm_exponent), so that the residue is 2^-22 of the norm and a piece written as zero loses
    //   at most 2^(e-25).
    static constexpr int KD34 = (3 * G + 4 + 15) / 16 * 16, KD24 = (2 * G + 4 + 15) / 16 * 16,
                         KD22 = (2 * G + 2 + 15) / 16 * 16;
    static constexpr bool FULL3 = KD34 <= 48 && KD34 <= KD24 && KD34 <= KD22;
    static constexpr int SPLIT = FULL3 ? 3 : 2;
    static constexpr int NQ = (FULL3 || KD24 <= KD22) ? 4 : 2;
    static constexpr int KD = (SPLIT * G + NQ + 15) / 16 * 16;      // contraction length (halves)
    static constexpr int A_TILE = TM * KD * 2;                      // bytes
    static constexpr int B_TILE = TN * KD * 2;
    static constexpr int STAGES = (KD <= 16) ? 4 : 3;
    static constexpr int MERGE = (EW - 1) * NA * TM * 12;           // exchange of the column groups' results
    static constexpr int SMEM = NA * A_TILE + STAGES * B_TILE + MERGE + 256;
    // Rounding model of the accumulation, in units of 2^-24 S (2||c||^2 + ||x||^2).  Assumed of the
    // tensor core: one 16-column step forms the 16 products exactly, aligns them and the FP32
    // accumulator to the largest exponent among the 17 addends, keeps at least 24 bits below that
    // exponent of each addend (the rest is dropped), adds exactly and rounds or truncates the sum to
    // FP32.  Every addend and every partial sum is at most S (2||c||^2 + ||x||^2) in magnitude
    // (2|x_t c_t| <= x_t^2 + c_t^2), so a step errs by at most 17 + 2 = 19 units.  Measured on the
    // device: 2.3 / 3.4 / 4.2 units for one / two / three steps.  Cutting S m into two pieces instead
    // of three leaves a residue of 2^-22 |S m_t| per coordinate: 4 more units; two norm pieces
    // instead of four leave 2^-22 S ||c||^2: 4 more.
    static constexpr int ERR_UNITS = 19 * (KD / 16) + (SPLIT == 2 ? 4 : 0) + (NQ == 2 ? 4 : 0);
};

// Written by the range kernel / prep kernel, read by the finish kernel (workspace, 16 bytes).
struct TcParams {
    unsigned cmax_bits;   // max |c| (FP32 bits; non-negative floats order like unsigned integers)
    unsigned qmax_bits;   // max ||c||^2, rounded up
    float S, invS;
};

__device__ __forceinline__ float min3(float a, float b, float c) {
    float d;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ int floor_log2_bits(unsigned bits) { return (int)((bits >> 23) & 0xffu) - 127; }

// S = 2^k, the largest power of two with  S * 2 cmax < 2^15  and  S * qmax < 2^30  (k <= 40).
__device__ __forceinline__ float scale_from_range(unsigned cmax_bits, unsigned qmax_bits) {
    int k = 14 - (floor_log2_bits(cmax_bits) + 1);
    const int k2 = 29 - floor_log2_bits(qmax_bits);
    k = k < k2 ? k : k2;
    k = k < 40 ? k : 40;
    k = k > -120 ? k : -120;
    return __int_as_float((k + 127) << 23);
}

// Largest |c| and largest ||c||^2 of the codebook (params zeroed beforehand).
__global__ void __launch_bounds__(256)
tensor_range_kernel(const float* __restrict__ C, int K, int g, TcParams* __restrict__ params) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    float cm = 0.f, qm = 0.f;
    if (j < K) {
        double s = 0.0;
        for (int t = 0; t < g; ++t) {
            const float c = C[(int64_t)j * g + t];
            cm = fmaxf(cm, fabsf(c));
            s += (double)c * (double)c;
        }
        qm = __double2float_ru(s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
        qm = fmaxf(qm, __shfl_xor_sync(0xffffffffu, qm, o));
    }
    if ((threadIdx.x & 31) == 0) {
        atomicMax(&params->cmax_bits, __float_as_uint(cm));
        atomicMax(&params->qmax_bits, __float_as_uint(qm));
    }
}

// h, or zero when h is not a normal FP16 number (see the header comment).
__device__ __forceinline__ __half normal_or_zero(__half h) {
    return ((__half_as_ushort(h) & 0x7c00u) == 0u) ? __ushort_as_half((unsigned short)0) : h;
}

// Exponent e of the larger of the two norm constants (NQ = 2): the smallest with S qmax / 2^e < 2^15,
// kept within [-3, 15] so that 2^e and 2^(e-11) are normal FP16 numbers.
__device__ __forceinline__ int norm_exponent(float S, unsigned qmax_bits) {
    int e = floor_log2_bits(__float_as_uint(S)) + floor_log2_bits(qmax_bits) - 14;
    e = e < -3 ? -3 : e;
    return e > 15 ? 15 : e;
}

// Constants that multiply the norm pieces: 2^15, 2^6, 2^-3, 2^-12 (four pieces) or 2^e, 2^(e-11) (two).
template <int NQ>
__device__ __forceinline__ float qconst(int p, int e) {
    if constexpr (NQ == 2) return __int_as_float((e - 11 * p + 127) << 23);
    else return p == 0 ? 32768.0f : p == 1 ? 64.0f : p == 2 ? 0.125f : 0.000244140625f;
}

// Staged B operand: tile b holds centroids 256b .. 256b+255 in the canonical layout, KD halves per
// centroid: SPLIT x G pieces of S m, NQ pieces of S ||c||^2, zeros.  One thread writes eight
// consecutive columns of one centroid (16 bytes).  Centroids K .. Kpad-1 are padding with a score
// of 2^15 * 65504; should it ever beat a real score (only with extreme inputs) the gap test fails
// and the exact stage decides.
template <int G>
__global__ void __launch_bounds__(256)
prep_tensor_kernel(const float* __restrict__ C, int K, int Kpad, TcParams* __restrict__ params,
                   uint16_t* __restrict__ gB, float* __restrict__ rescan) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, SPLIT = Cfg::SPLIT, NQ = Cfg::NQ;
    const float S = scale_from_range(params->cmax_bits, params->qmax_bits);
    const int ne = norm_exponent(S, params->qmax_bits);
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e == 0) { params->S = S; params->invS = 1.0f / S; }
    if (e >= Kpad * (KD / 8)) return;
    const int j = e / (KD / 8), kc = e - j * (KD / 8);
    if (kc == 0 && rescan) {
        // FP32 table of the finish kernel, one block of (g+1) x 64 floats per 64-centroid chunk: for
        // coordinate t the 64 values m_{j,t} = -2 c_{j,t} of the chunk side by side, then the 64 squared
        // norms (a group of 8 lanes reads 128 contiguous bytes per load); padding can never win
        float* blk = rescan + (int64_t)(j / TCHUNK) * ((G + 1) * TCHUNK) + (j % TCHUNK);
        double s = 0.0;
#pragma unroll
        for (int t = 0; t < G; ++t) {
            const float c = (j < K) ? C[(int64_t)j * G + t] : 0.f;
            blk[t * TCHUNK] = -2.0f * c;
            s += (double)c * (double)c;
        }
        blk[G * TCHUNK] = (j < K) ? (float)s : kBig;
    }
    __half out[8];
    __half qp[NQ];
    bool need_q = false;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int k = kc * 8 + u;
        if (k >= SPLIT * G && k < SPLIT * G + NQ) need_q = true;
    }
    if (need_q) {
        if (j < K) {
            double s = 0.0;
#pragma unroll
            for (int t = 0; t < G; ++t) { const double c = (double)C[(int64_t)j * G + t]; s += c * c; }
            double R = s * (double)S;
#pragma unroll
            for (int p = 0; p < NQ; ++p) {
                const double a = (double)qconst<NQ>(p, ne);
                qp[p] = normal_or_zero(__double2half(R / a));   // division by a power of two: exact
                R -= (double)__half2float(qp[p]) * a;           // exact: cancels the leading bits of R
            }
        } else {
            qp[0] = __ushort_as_half((unsigned short)0x7bffu);   // 65504
#pragma unroll
            for (int p = 1; p < NQ; ++p) qp[p] = __ushort_as_half((unsigned short)0);
        }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int k = kc * 8 + u;
        __half v = __ushort_as_half((unsigned short)0);
        if (k < SPLIT * G) {
            if (j < K) {
                const int piece = k / G, t = k - piece * G;
                const float M = S * (-2.0f * C[(int64_t)j * G + t]);    // exact (powers of two)
                const __half h1 = normal_or_zero(__float2half_rn(M));
                const float r1 = M - __half2float(h1);                  // exact: at most 13 bits (or M itself)
                const __half h2 = normal_or_zero(__float2half_rn(r1));
                const float r2 = r1 - __half2float(h2);
                v = (piece == 0) ? h1 : (piece == 1) ? h2 : normal_or_zero(__float2half_rn(r2));
            }
        } else if (k < SPLIT * G + NQ) {
            v = qp[k - SPLIT * G];
        }
        out[u] = v;
    }
    const int tile = j / TN, jr = j - tile * TN;
    unsigned char* dst = reinterpret_cast<unsigned char*>(gB) + (int64_t)tile * Cfg::B_TILE + canon_bytes(jr, kc * 8, TN);
    uint4 w;
    w.x = (unsigned)__half_as_ushort(out[0]) | ((unsigned)__half_as_ushort(out[1]) << 16);
    w.y = (unsigned)__half_as_ushort(out[2]) | ((unsigned)__half_as_ushort(out[3]) << 16);
    w.z = (unsigned)__half_as_ushort(out[4]) | ((unsigned)__half_as_ushort(out[5]) << 16);
    w.w = (unsigned)__half_as_ushort(out[6]) | ((unsigned)__half_as_ushort(out[7]) << 16);
    *reinterpret_cast<uint4*>(dst) = w;
}

// A operand rows [x repeated SPLIT times, 2^15, 2^6, 2^-3, 2^-12, 0..] of points base + e,
// e = first, first + step, .. < count, into the tiles at sA (canonical layout, 16 bytes at a time).
template <int G>
__device__ __forceinline__ void build_a_rows(const uint16_t* __restrict__ X, int64_t N, int64_t base, int first,
                                             int step, int count, unsigned char* sA, bool& nonfinite,
                                             const TcParams* __restrict__ params) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, SPLIT = Cfg::SPLIT, NQ = Cfg::NQ;
    int ne = 0;                                  // only the two-piece norm has call-dependent constants
    if constexpr (NQ == 2) ne = norm_exponent(scale_from_range(params->cmax_bits, params->qmax_bits), params->qmax_bits);
    for (int e = first; e < count; e += step) {
        float x[G];
        load_point<G>(X, base + e, N, x, nonfinite);
        unsigned short h[KD];
#pragma unroll
        for (int k = 0; k < KD; ++k) {
            h[k] = (k < SPLIT * G) ? __half_as_ushort(__float2half_rn(x[k % G]))    // exact: x is FP16 data
                 : (k < SPLIT * G + NQ) ? __half_as_ushort(__float2half_rn(qconst<NQ>(k - SPLIT * G, ne)))
                 : (unsigned short)0;
        }
        unsigned char* tile = sA + (e / TM) * Cfg::A_TILE;
        const int r = e % TM;
#pragma unroll
        for (int kc = 0; kc < KD / 8; ++kc) {
            uint4 w;
            w.x = (unsigned)h[kc * 8 + 0] | ((unsigned)h[kc * 8 + 1] << 16);
            w.y = (unsigned)h[kc * 8 + 2] | ((unsigned)h[kc * 8 + 3] << 16);
            w.z = (unsigned)h[kc * 8 + 4] | ((unsigned)h[kc * 8 + 5] << 16);
            w.w = (unsigned)h[kc * 8 + 6] | ((unsigned)h[kc * 8 + 7] << 16);
            *reinterpret_cast<uint4*>(tile + canon_bytes(r, kc * 8, TM)) = w;
        }
    }
}

// The reduction of one 64-column chunk held in two 32-register halves: a tree of three-input
// minima (21 + 7 + 2 + 1, and one two-input minimum for the 64th value).  The first level takes
// three consecutive registers each, so that registers free up as the tree advances; measured 2 %
// faster than four running chains of the same 32 instructions, which also spilled.
__device__ __forceinline__ float chunk_min64(const uint32_t* v0, const uint32_t* v1) {
    auto val = [&](int i) { return __uint_as_float(i < 32 ? v0[i] : v1[i - 32]); };
    float t[21];
#pragma unroll
    for (int k = 0; k < 21; ++k) t[k] = min3(val(3 * k), val(3 * k + 1), val(3 * k + 2));
    float u[7];
#pragma unroll
    for (int j = 0; j < 7; ++j) u[j] = min3(t[3 * j], t[3 * j + 1], t[3 * j + 2]);
    const float w0 = min3(u[0], u[1], u[2]), w1 = min3(u[3], u[4], u[5]);
    return fminf(min3(w0, w1, u[6]), val(63));
}

// DUMP = true writes every score (divided by S) to `dump` (row stride dump_ld) instead of
// reducing them: a verification aid for the rounding model, used on small inputs only.
// FULL = true: every CTA of the launch holds exactly NA point tiles, which makes the accumulator
// slot and the barrier phase of tile (b, a) compile-time functions of a; the ragged rest of the
// points (and small inputs) go through FULL = false, starting at point tile `tile_offset`.
template <int G, bool DUMP, bool FULL>
__global__ void __launch_bounds__(TC_THREADS, 1)
assign_tensor_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ gB, int n_btiles,
                     int na_per_cta, int64_t tile_offset, const TcParams* __restrict__ params,
                     float2* __restrict__ tstate, unsigned* __restrict__ status, float* __restrict__ dump,
                     int64_t dump_ld) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, STAGES = Cfg::STAGES;
    constexpr int A_TILE = Cfg::A_TILE, B_TILE = Cfg::B_TILE;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* sA = smem_raw;                                   // NA tiles
    unsigned char* sB = sA + NA * A_TILE;                           // STAGES tiles
    float* merge = reinterpret_cast<float*>(sB + STAGES * B_TILE);  // [EW-1][NA][3][TM]: best, second, best chunk id
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(merge) + Cfg::MERGE);
    uint64_t* b_full = bars, *b_empty = bars + STAGES, *t_full = bars + 2 * STAGES, *t_empty = bars + 2 * STAGES + SLOTS;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 2 * SLOTS);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t tile0 = tile_offset + (int64_t)blockIdx.x * na_per_cta;   // first point tile of this CTA
    const int64_t n_tiles = (N + TM - 1) / TM;
    const int na = FULL ? NA : (int)((n_tiles - tile0 < na_per_cta) ? (n_tiles - tile0) : na_per_cta);
    const int64_t base = tile0 * TM;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_empty + s)));
        }
        for (int s = 0; s < SLOTS; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(t_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(t_empty + s)), "r"(EPI_WARPS * 32));
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    bool nonfinite = false;
    build_a_rows<G>(X, N, base, tid, TC_THREADS, na * TM, sA, nonfinite, params);
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
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(B_TILE) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(sB + st * B_TILE)),
                               "l"(reinterpret_cast<const unsigned char*>(gB) + (int64_t)b * B_TILE), "r"(B_TILE), "r"(bar)
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
            // kind::f16: D = F32 (bits 4-5 = 1), A = B = F16 (0), both K-major, N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc = (1u << 4) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
            // descriptors of the first tiles; the start-address field counts 16-byte units, so a
            // tile or a 16-column step further on is a plain addition
            const uint64_t descA0 = make_desc(smem_u32(sA), TM * 16, 128);
            const uint64_t descB0 = make_desc(smem_u32(sB), TN * 16, 128);
            bool ok = true;
            int q = 0;
            for (int b = 0; b < n_btiles && ok; ++b) {
                const int st = b % STAGES;
                ok = mbar_wait(smem_u32(b_full + st), (b / STAGES) & 1, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t descB = descB0 + (uint64_t)((st * B_TILE) >> 4);
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    if (a >= na) break;
                    // with NA = 8 tiles per codebook tile the slot and phase of tile (b, a) depend on a only
                    const int slot = FULL ? (a % SLOTS) : (q % SLOTS);
                    const uint32_t par = FULL ? ((a / SLOTS) & 1) : ((q / SLOTS) & 1);
                    ++q;
                    ok = mbar_wait(smem_u32(t_empty + slot), par ^ 1, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t descA = descA0 + (uint64_t)((a * A_TILE) >> 4);
                    const uint32_t d = tmem + slot * TN;
#pragma unroll
                    for (int s = 0; s < KD / 16; ++s) {
                        const uint64_t da = descA + (uint64_t)((s * 2 * (TM * 16)) >> 4);
                        const uint64_t db = descB + (uint64_t)((s * 2 * (TN * 16)) >> 4);
                        if (s == 0)
                            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                                         "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                         ::"r"(d), "l"(da), "l"(db), "r"(idesc) : "memory");
                        else
                            asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                                         "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                         ::"r"(d), "l"(da), "l"(db), "r"(idesc) : "memory");
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
        const int quarter = warp & 3, cg = warp >> 2;     // TMEM lane quarter, 64-column group
        const int r = quarter * 32 + lane;                // row of the point tile = TMEM lane
        const float invS = DUMP ? params->invS : 0.f;
        float b1[NA], b2[NA];
        int bc[NA];
#pragma unroll
        for (int a = 0; a < NA; ++a) { b1[a] = INFINITY; b2[a] = INFINITY; bc[a] = cg; }
        const uint32_t tbase = tmem + ((uint32_t)(quarter * 32) << 16) + cg * TCHUNK;
        uint32_t okw = 1u;
        int q = 0;
        int chunk_id = cg;                                // id of this warp's chunk in codebook tile b
        for (int b = 0; b < n_btiles && okw; ++b, chunk_id += EW) {
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                if (a >= na) continue;
                // A wait that gives up is only acted upon after the tiles of this round: once the abort
                // flag is up the remaining waits return at their next look at it, and reading an
                // accumulator that was never written or releasing it once more harms nothing.
                const int slot = FULL ? (a % SLOTS) : (q % SLOTS);
                const uint32_t par = FULL ? ((a / SLOTS) & 1) : ((q / SLOTS) & 1);
                mbar_wait_acc(smem_u32(t_full + slot), par, abort_flag, okw);
                ++q;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                uint32_t v0[32], v1[32];
                TMEM_LD32(v0, tbase + slot * TN);
                TMEM_LD32(v1, tbase + slot * TN + 32);
                TMEM_WAIT64(v0, v1);
                // the 64 columns are in registers: every lane hands back its own share of the
                // accumulator (the barrier counts 16 x 32 arrivals; no predicate, no warp synchronisation)
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(t_empty + slot)) : "memory");
                if constexpr (DUMP) {
                    const int64_t i = base + a * TM + r;
                    if (i < N) {
                        float* row = dump + i * dump_ld + (int64_t)b * TN + cg * TCHUNK;
#pragma unroll
                        for (int u = 0; u < 32; ++u) { row[u] = __uint_as_float(v0[u]) * invS; row[32 + u] = __uint_as_float(v1[u]) * invS; }
                    }
                } else {
                    const float m = chunk_min64(v0, v1);
                    const bool better = m < b1[a];
                    b2[a] = better ? b1[a] : fminf(b2[a], m);
                    bc[a] = better ? chunk_id : bc[a];
                    b1[a] = better ? m : b1[a];
                }
            }
        }
        if constexpr (!DUMP) {
            // ---- merge the EW column groups of each point (through shared memory) and store
            if (cg > 0) {
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    float* mrow = merge + (((cg - 1) * NA + a) * 3) * TM + r;
                    mrow[0] = b1[a]; mrow[TM] = b2[a]; mrow[2 * TM] = __int_as_float(bc[a]);
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(EPI_WARPS * 32));
            if (cg == 0 && okw && !*abort_flag) {
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    const int64_t i = base + a * TM + r;
                    if (a >= na || i >= N) continue;
                    float w1 = b1[a], w2 = b2[a];
                    int wc = bc[a];
#pragma unroll
                    for (int o = 0; o < EW - 1; ++o) {
                        const float* srow = merge + ((o * NA + a) * 3) * TM + r;
                        const float o1 = srow[0], o2 = srow[TM];
                        const int oc = __float_as_int(srow[2 * TM]);
                        if (o1 < w1) { w2 = fminf(w1, o2); w1 = o1; wc = oc; }     // equal minima: the gap is 0 and
                        else { w2 = fminf(w2, o1); }                                // the point goes to the exact stage
                    }
                    tstate[i] = make_float2(w2, __int_as_float(wc));
                }
            }
        }
    }
    if (*abort_flag && lane == 0) atomicOr(status, CC_DEV_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(SLOTS * TN));
}

// Persistent form of the scan for contraction lengths up to 32 columns (g <= 15): one CTA per SM walks
// over groups of NA point tiles (group = blockIdx.x, + gridDim.x, ..) and keeps TWO sets of A tiles
// in shared memory.  A 19th warp builds the next group's A operand while the current group is
// multiplied and reduced, so the tensor core and the epilogue never wait for a CTA to start or to
// drain: with few codebook tiles per group (K = 4096: 16) that start-up is a tenth of the time.
// Roles and barriers are those of assign_tensor_kernel plus a_full / a_empty per A buffer; every
// group has n_btiles * NA tiles, a multiple of four, so accumulator slot and phase stay
// compile-time functions of a.
constexpr int PERSIST_THREADS = TC_THREADS + 32;

template <int G> struct PersistCfg {
    using Cfg = TcCfg<G>;
    static constexpr bool OK = Cfg::KD <= 32;
    static constexpr int SMEM = 2 * NA * Cfg::A_TILE + Cfg::STAGES * Cfg::B_TILE + Cfg::MERGE + 256;
};

template <int G>
__global__ void __launch_bounds__(PERSIST_THREADS, 1)
assign_tensor_persistent_kernel(const uint16_t* __restrict__ X, int64_t N, const uint16_t* __restrict__ gB, int n_btiles,
                                int n_groups, const TcParams* __restrict__ params, float2* __restrict__ tstate,
                                unsigned* __restrict__ status) {
    using Cfg = TcCfg<G>;
    constexpr int KD = Cfg::KD, STAGES = Cfg::STAGES;
    constexpr int A_TILE = Cfg::A_TILE, B_TILE = Cfg::B_TILE, A_SET = NA * A_TILE;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* sA = smem_raw;                                   // 2 sets of NA tiles
    unsigned char* sB = sA + 2 * A_SET;                             // STAGES tiles
    float* merge = reinterpret_cast<float*>(sB + STAGES * B_TILE);  // [EW-1][NA][3][TM]
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(merge) + Cfg::MERGE);
    uint64_t* b_full = bars, *b_empty = bars + STAGES, *t_full = bars + 2 * STAGES, *t_empty = t_full + SLOTS;
    uint64_t* a_full = t_empty + SLOTS, *a_empty = a_full + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_empty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_iter = (n_groups - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // groups of this CTA

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(b_empty + s)));
        }
        for (int s = 0; s < SLOTS; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(t_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(t_empty + s)), "r"(EPI_WARPS * 32));
        }
        for (int s = 0; s < 2; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(a_full + s)));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(a_empty + s)));
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // first group's A operand: built by everybody
    bool nonfinite = false;
    build_a_rows<G>(X, N, (int64_t)blockIdx.x * (NA * TM), tid, PERSIST_THREADS, NA * TM, sA, nonfinite, params);
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
            int st = 0;
            uint32_t ph = 0;
            int in_flight_from = 0, total = 0;
            bool ok = true;
            for (int it = 0; it < n_iter && ok; ++it) {
                for (int b = 0; b < n_btiles; ++b) {
                    if (!mbar_wait(smem_u32(b_empty + st), ph ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t bar = smem_u32(b_full + st);
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(B_TILE) : "memory");
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(sB + st * B_TILE)),
                                   "l"(reinterpret_cast<const unsigned char*>(gB) + (int64_t)b * B_TILE), "r"(B_TILE), "r"(bar)
                                 : "memory");
                    ++total;
                    if (++st == STAGES) { st = 0; ph ^= 1; }
                }
            }
            if (*abort_flag) {   // let the copies in flight land before the CTA exits (bounded)
                in_flight_from = total > STAGES ? total - STAGES : 0;
                for (int c = in_flight_from; c < total; ++c) {
                    const long long t0 = clock64();
                    while (!mbar_try(smem_u32(b_full + c % STAGES), (c / STAGES) & 1) && clock64() - t0 < WAIT_LIMIT) {}
                }
            }
        }
    } else if (warp == EPI_WARPS + 1) {
        // ------------------------------------------------------------ MMA warp: one thread issues
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | ((uint32_t)(TN >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
            const uint64_t descA0 = make_desc(smem_u32(sA), TM * 16, 128);
            const uint64_t descB0 = make_desc(smem_u32(sB), TN * 16, 128);
            bool ok = true;
            int st = 0;
            uint32_t ph = 0;
            for (int it = 0; it < n_iter && ok; ++it) {
                const int buf = it & 1;
                if (it > 0) {      // the first set was built before the barrier above
                    ok = mbar_wait(smem_u32(a_full + buf), ((it - 1) >> 1) & 1, abort_flag);
                    if (!ok) break;
                }
                for (int b = 0; b < n_btiles && ok; ++b) {
                    ok = mbar_wait(smem_u32(b_full + st), ph, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t descB = descB0 + (uint64_t)((st * B_TILE) >> 4);
#pragma unroll
                    for (int a = 0; a < NA; ++a) {
                        const int slot = a % SLOTS;
                        ok = mbar_wait(smem_u32(t_empty + slot), (((a / SLOTS) & 1)) ^ 1, abort_flag);
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        const uint64_t descA = descA0 + (uint64_t)((buf * A_SET + a * A_TILE) >> 4);
                        const uint32_t d = tmem + slot * TN;
#pragma unroll
                        for (int s = 0; s < KD / 16; ++s) {
                            const uint64_t da = descA + (uint64_t)((s * 2 * (TM * 16)) >> 4);
                            const uint64_t db = descB + (uint64_t)((s * 2 * (TN * 16)) >> 4);
                            if (s == 0)
                                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                             ::"r"(d), "l"(da), "l"(db), "r"(idesc) : "memory");
                            else
                                asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                             ::"r"(d), "l"(da), "l"(db), "r"(idesc) : "memory");
                        }
                        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                     ::"r"(smem_u32(t_full + slot)) : "memory");
                    }
                    if (ok)   // the ring stage may be refilled once these MMAs have read it
                        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                     ::"r"(smem_u32(b_empty + st)) : "memory");
                    if (++st == STAGES) { st = 0; ph ^= 1; }
                }
                if (ok)       // this set of A tiles may be overwritten once the group's MMAs have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(smem_u32(a_empty + buf)) : "memory");
            }
        }
    } else if (warp == EPI_WARPS + 2) {
        // ------------------------------------------------------------ A-operand warp: next group's tiles
        bool ok = true;
        for (int it = 1; it < n_iter && ok; ++it) {
            const int buf = it & 1;
            if (it >= 2) {     // the set was last used by group it - 2
                ok = mbar_wait(smem_u32(a_empty + buf), ((it - 2) >> 1) & 1, abort_flag);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
            }
            const int64_t group = (int64_t)blockIdx.x + (int64_t)it * gridDim.x;
            build_a_rows<G>(X, N, group * (NA * TM), lane, 32, NA * TM, sA + buf * A_SET, nonfinite, params);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0)
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(a_full + buf)) : "memory");
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        const int quarter = warp & 3, cg = warp >> 2;     // TMEM lane quarter, 64-column group
        const int r = quarter * 32 + lane;                // row of the point tile = TMEM lane
        // the same value in all lanes, and visibly so (broadcast from lane 0): the accumulator address
        // can then live in a uniform register instead of being converted for every load
        const uint32_t tbase = __shfl_sync(0xffffffffu, tmem + ((uint32_t)(quarter * 32) << 16) + cg * TCHUNK, 0);
        bool ok = true;
        for (int it = 0; it < n_iter && ok; ++it) {
            float b1[NA], b2[NA];
            int bc[NA];
#pragma unroll
            for (int a = 0; a < NA; ++a) { b1[a] = INFINITY; b2[a] = INFINITY; bc[a] = cg; }
            int chunk_id = cg;
            uint32_t okw = 1u;
            for (int b = 0; b < n_btiles && okw; ++b, chunk_id += EW) {
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    // A wait that gives up is only acted upon after the eight tiles: once the abort flag
                    // is up the remaining waits return at their next look at it, and reading an
                    // accumulator that was never written or releasing it once more harms nothing.
                    const int slot = a % SLOTS;
                    mbar_wait_acc(smem_u32(t_full + slot), (a / SLOTS) & 1, abort_flag, okw);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    uint32_t v0[32], v1[32];
                    TMEM_LD32(v0, tbase + slot * TN);
                    TMEM_LD32(v1, tbase + slot * TN + 32);
                    TMEM_WAIT64(v0, v1);
                    // every lane hands back its own 32 x 64 share (the barrier counts 16 x 32 arrivals):
                    // no predicate, no warp synchronisation
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(t_empty + slot)) : "memory");
                    const float m = chunk_min64(v0, v1);
                    const bool better = m < b1[a];
                    b2[a] = better ? b1[a] : fminf(b2[a], m);
                    bc[a] = better ? chunk_id : bc[a];
                    b1[a] = better ? m : b1[a];
                }
            }
            ok = okw != 0u;
            // ---- merge the EW column groups of each point and store; the exchange area is reused by
            //      the next group, hence the second barrier
            if (cg > 0) {
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    float* mrow = merge + (((cg - 1) * NA + a) * 3) * TM + r;
                    mrow[0] = b1[a]; mrow[TM] = b2[a]; mrow[2 * TM] = __int_as_float(bc[a]);
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(EPI_WARPS * 32));
            if (cg == 0 && ok && !*abort_flag) {
                const int64_t base = ((int64_t)blockIdx.x + (int64_t)it * gridDim.x) * (NA * TM);
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    const int64_t i = base + a * TM + r;
                    if (i >= N) continue;
                    float w1 = b1[a], w2 = b2[a];
                    int wc = bc[a];
#pragma unroll
                    for (int o = 0; o < EW - 1; ++o) {
                        const float* srow = merge + ((o * NA + a) * 3) * TM + r;
                        const float o1 = srow[0], o2 = srow[TM];
                        const int oc = __float_as_int(srow[2 * TM]);
                        if (o1 < w1) { w2 = fminf(w1, o2); w1 = o1; wc = oc; }
                        else { w2 = fminf(w2, o1); }
                    }
                    tstate[i] = make_float2(w2, __int_as_float(wc));
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(EPI_WARPS * 32));
            ok = !*abort_flag;     // read after the barrier: the same answer in all sixteen warps
        }
    }
    if (nonfinite) atomicOr(status, CC_DEV_NONFINITE);
    if (*abort_flag && lane == 0) atomicOr(status, CC_DEV_TIMEOUT);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(SLOTS * TN));
}

// Finish, LPP = 8 lanes per point (four points per warp): lane k of a group recomputes the scores of
// centroids 4k .. 4k+3 and 32+4k .. 32+4k+3 (four consecutive centroids every 4 LPP) of the winning
// 64-centroid chunk with the FMA chain
// s = fma(x_{g-1}, m_{g-1}, ... fma(x_0, m_0, ||c||^2)), keeping its smallest score, its index and
// its runner-up; a butterfly over the group gives every lane the chunk's winner and runner-up.
// A group does this for eight points in turn and lane k keeps the k-th result, so that the rest
// runs once per 32 points with one point per lane: the squared distance to the winner in FP64
// (sub, mul, add in dimension order, no contraction), the near-tie test and the stores.  A scan whose scores are off by at most
//     E = ERR_UNITS 2^-24 (2||c||^2 + ||x||^2) + 2^-14 ||x||_1 / S + 2^-26 / S   (2^(e-25) / S with two norm pieces)
// (|x_t| counted as at least 2^-14) may misorder two scores closer than 2E; every centroid at
// least as close as the winner (distance d) has ||c|| <= ||x|| + d, hence 2||c||^2 + ||x||^2 <=
// 3||x||^2 + 4||x|| d + 2 d^2, so a point whose two smallest scores are closer than 2E with that
// substitution goes to the exact stage.
template <int G>
__global__ void __launch_bounds__(256)
finish_tensor_kernel(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ C, int K, int n_chunks,
                     const float* __restrict__ rescan, const float2* __restrict__ tstate,
                     const TcParams* __restrict__ params, uint16_t* __restrict__ idx, float* __restrict__ dist,
                     unsigned* __restrict__ status, unsigned* __restrict__ flagged) {
    const int k = threadIdx.x & (LPP - 1);
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t rounds = (N + n_warps * 32 - 1) / (n_warps * 32);  // the same for every lane of a warp
    const float invS = params->invS;
    // what the norm pieces may lose to a piece written as zero, in scaled units: 2^-26 with four
    // pieces, 2^(e-25) with two
    double norm_abs = 1.4901161193847656e-8;
    if constexpr (TcCfg<G>::NQ == 2)
        norm_abs = (double)__int_as_float((norm_exponent(params->S, params->qmax_bits) - 25 + 127) << 23);
    for (int64_t rd = 0; rd < rounds; ++rd) {
        // A warp takes 32 consecutive points per round: its four lane groups rescan eight points
        // each, one after the other, and lane l keeps what was found for point base + l, so that
        // the exact distance, the bound and the stores are done once for 32 points.
        const int64_t base = (rd * n_warps + warp0) * 32;
        // every lane loads its own point and scan result once (coalesced); the group then gets the
        // point it works on from the lane that owns it
        const int64_t i_raw = base + lane;
        const bool live = i_raw < N;
        const int64_t i = live ? i_raw : N - 1;
        float2 t_own = tstate[i];
        // The chunk id comes from the scan's output.  A scan CTA that gave up on a bounded wait has
        // written nothing there, so the word may hold anything: keep it inside the table (the call
        // then reports CC_ERR_DEVICE_TIMEOUT and its results are void, but nothing is read out of
        // bounds).
        t_own.y = __int_as_float(min(max(__float_as_int(t_own.y), 0), n_chunks - 1));
        float x_own[G];
        bool nf = false;
        load_point<G>(X, i, N, x_own, nf);
        float keep_s1 = 0.f, keep_s2 = 0.f;
        int keep_j = 0;
#pragma unroll 1
        for (int sub = 0; sub < LPP; ++sub) {
            const int src = (lane & ~(LPP - 1)) + sub;
            const int chunk = __shfl_sync(0xffffffffu, __float_as_int(t_own.y), src);
            float x[G];
#pragma unroll
            for (int u = 0; u < G; ++u) x[u] = __shfl_sync(0xffffffffu, x_own[u], src);
            const float4* blk = reinterpret_cast<const float4*>(rescan + (int64_t)chunk * ((G + 1) * TCHUNK)) + k;
            float s1 = INFINITY, s2 = INFINITY;
            int j1 = 4 * k;
#pragma unroll
            for (int hf = 0; hf < TCHUNK / 4 / LPP; ++hf) {
                const float4 cs = __ldg(blk + G * (TCHUNK / 4) + hf * LPP);
                float s[4] = {cs.x, cs.y, cs.z, cs.w};
#pragma unroll
                for (int u = 0; u < G; ++u) {
                    const float4 mv = __ldg(blk + u * (TCHUNK / 4) + hf * LPP);
                    s[0] = fmaf(x[u], mv.x, s[0]);
                    s[1] = fmaf(x[u], mv.y, s[1]);
                    s[2] = fmaf(x[u], mv.z, s[2]);
                    s[3] = fmaf(x[u], mv.w, s[3]);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool take = s[e] < s1;                 // ascending index: strict '<' keeps the lowest
                    s2 = take ? s1 : fminf(s2, s[e]);
                    j1 = take ? (hf * LPP + k) * 4 + e : j1;
                    s1 = take ? s[e] : s1;
                }
            }
#pragma unroll
            for (int o = LPP / 2; o > 0; o >>= 1) {
                const float os1 = __shfl_xor_sync(0xffffffffu, s1, o);
                const float os2 = __shfl_xor_sync(0xffffffffu, s2, o);
                const int oj = __shfl_xor_sync(0xffffffffu, j1, o);
                const bool take = os1 < s1 || (os1 == s1 && oj < j1);
                s2 = fminf(take ? s1 : os1, fminf(s2, os2));
                s1 = take ? os1 : s1;
                j1 = take ? oj : j1;
            }
            if (k == sub) {                   // this round's point is the lane's own
                keep_j = j1 + chunk * TCHUNK;
                keep_s1 = s1;
                keep_s2 = fminf(s2, t_own.x * invS);
            }
        }
        int j1 = keep_j;
        if (j1 >= K) j1 = K - 1;   // only reachable with non-finite input or after a time-out
        const float (&x)[G] = x_own;
        double D = 0.0;
        float A = 0.f, L1 = 0.f;
#pragma unroll
        for (int u = 0; u < G; ++u) {
            const double df = __dsub_rn((double)x[u], (double)__ldg(C + (int64_t)j1 * G + u));
            D = __dadd_rn(D, __dmul_rn(df, df));
            const float xf = fmaxf(fabsf(x[u]), 6.103515625e-5f);
            A = fmaf(xf, xf, A);
            L1 += fabsf(x[u]);
        }
        if (live) {
            idx[i] = (uint16_t)j1;
            dist[i] = (float)D;
            // A and L1 only feed the bound: FP32 is enough once they are rounded up a little
            // 2||c||^2 + ||x||^2 <= 2 (||x|| + d)^2 + ||x||^2 = 3||x||^2 + 4||x|| d + 2 d^2 for every centroid within d of x
            const double Au = (double)A * 1.0001;
            const double bound = 2.0 * ((double)TcCfg<G>::ERR_UNITS * 5.9604644775390625e-8 *
                                            (3.0 * Au + 4.0 * sqrt(Au * D) * 1.0000001 + 2.0 * D)
                                        + (double)invS * (6.103515625e-5 * (double)L1 * 1.0001 + norm_abs));
            if (!((double)keep_s2 - (double)keep_s1 > bound)) {
                const ull slot = atomicAdd(reinterpret_cast<ull*>(status + 2), 1ull);
                flagged[slot] = (unsigned)i;
            }
        }
    }
}

template <int G>
cudaError_t launch_tensor(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, const float* C, int K,
                          uint16_t* idx, float* dist, float* dump, int64_t dump_ld, const float2* scan_in,
                          cudaStream_t st) {
    using Cfg = TcCfg<G>;
    char* ws = static_cast<char*>(ctx->ws);
    unsigned* status = reinterpret_cast<unsigned*>(ws + L.status);
    TcParams* params = reinterpret_cast<TcParams*>(ws + L.status + 128);
    uint16_t* gB = reinterpret_cast<uint16_t*>(ws + L.tensor);
    float2* tstate = reinterpret_cast<float2*>(ws + L.tstate);
    if (scan_in) tstate = const_cast<float2*>(scan_in);   // finish only: the caller supplies the scan's output
    const int Kpad = (int)cc_align_up((size_t)K, TN);
    // FP32 rows of the finish kernel sit behind the FP16 operand image (at most 96 bytes per centroid)
    float* rescan = reinterpret_cast<float*>(ws + L.tensor + (size_t)Kpad * 96);
    cudaError_t e;
    // status words 2..3 (the flagged-point counter of this E-step) up to the range words: one memset
    // (the words in between are unused except the objective's ticket, which is zero between kernels)
    if ((e = cudaMemsetAsync(status + 2, 0, 120 + sizeof(TcParams), st)) != cudaSuccess) return e;
    {
        ProfScope ps(ctx, CC_K_ASSIGN_PREP, st);
        tensor_range_kernel<<<(K + 255) / 256, 256, 0, st>>>(C, K, G, params);
    }
    {
        ProfScope ps(ctx, CC_K_ASSIGN_PREP, st);
        const int n = Kpad * (Cfg::KD / 8);
        prep_tensor_kernel<G><<<(n + 255) / 256, 256, 0, st>>>(C, K, Kpad, params, gB, dump ? nullptr : rescan);
    }
    if (N > 0) {
        const int64_t n_tiles = (N + TM - 1) / TM;
        int64_t na_per_cta = (n_tiles + ctx->sm_count - 1) / ctx->sm_count;    // small inputs still use every SM
        if (na_per_cta > NA) na_per_cta = NA;
        // the opt-in to large dynamic shared memory is per device
        static bool attr_set_dev[64] = {};
        bool& attr_set = attr_set_dev[ctx->device & 63];
        if (!attr_set) {
            if ((e = cudaFuncSetAttribute(assign_tensor_kernel<G, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM)) != cudaSuccess) return e;
            if ((e = cudaFuncSetAttribute(assign_tensor_kernel<G, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM)) != cudaSuccess) return e;
            if ((e = cudaFuncSetAttribute(assign_tensor_kernel<G, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM)) != cudaSuccess) return e;
            attr_set = true;
        }
        if (dump) {
            const int64_t blocks = (n_tiles + na_per_cta - 1) / na_per_cta;
            ProfScope ps(ctx, CC_K_OTHER, st);
            assign_tensor_kernel<G, true, false><<<(unsigned)blocks, TC_THREADS, Cfg::SMEM, st>>>(
                X, N, gB, Kpad / TN, (int)na_per_cta, 0, params, tstate, status, dump, dump_ld);
            return cudaGetLastError();
        }
        if (!scan_in) {
            ProfScope ps(ctx, CC_K_ASSIGN_MAIN, st);
            // CTAs with a full set of NA point tiles, then the ragged rest
            const int64_t full_blocks = (na_per_cta == NA) ? n_tiles / NA : 0;
            if (PersistCfg<G>::OK && full_blocks >= 2 * (int64_t)ctx->sm_count && full_blocks < (1ll << 30)) {
                static bool attr_p_dev[64] = {};
                bool& attr_p = attr_p_dev[ctx->device & 63];
                if (!attr_p) {
                    if ((e = cudaFuncSetAttribute(assign_tensor_persistent_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, PersistCfg<G>::SMEM)) != cudaSuccess) return e;
                    attr_p = true;
                }
                assign_tensor_persistent_kernel<G><<<ctx->sm_count, PERSIST_THREADS, PersistCfg<G>::SMEM, st>>>(
                    X, N, gB, Kpad / TN, (int)full_blocks, params, tstate, status);
            } else if (full_blocks > 0)
                assign_tensor_kernel<G, false, true><<<(unsigned)full_blocks, TC_THREADS, Cfg::SMEM, st>>>(
                    X, N, gB, Kpad / TN, NA, 0, params, tstate, status, nullptr, 0);
            const int64_t rest_tiles = n_tiles - full_blocks * NA;
            if (rest_tiles > 0) {
                const int64_t blocks = (rest_tiles + na_per_cta - 1) / na_per_cta;
                assign_tensor_kernel<G, false, false><<<(unsigned)blocks, TC_THREADS, Cfg::SMEM, st>>>(
                    X, N, gB, Kpad / TN, (int)na_per_cta, full_blocks * NA, params, tstate, status, nullptr, 0);
            }
        }
        {
            ProfScope ps(ctx, CC_K_ASSIGN_FINISH, st);
            int64_t fblocks = (N + 255) / 256;            // a warp takes 32 points per round
            const int64_t cap = (int64_t)ctx->sm_count * 32;
            if (fblocks > cap) fblocks = cap;
            finish_tensor_kernel<G><<<(unsigned)fblocks, 256, 0, st>>>(
                X, N, C, K, Kpad / TCHUNK, rescan, tstate, params, idx, dist, status,
                reinterpret_cast<unsigned*>(ws + L.flagged));
        }
    }
    return cudaGetLastError();
}

#define CC_TENSOR_DISPATCH(g, CALL)                                                                 \
    switch (g) {                                                                                    \
        case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;                 \
        case 4: CALL(4); break;   case 5: CALL(5); break;   case 6: CALL(6); break;                 \
        case 7: CALL(7); break;   case 8: CALL(8); break;   case 9: CALL(9); break;                 \
        case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;               \
        case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break;               \
        case 16: CALL(16); break;                                                                   \
        default: return cudaErrorInvalidValue;                                                      \
    }

}  // namespace

bool cc_tensor_path_supported(int g, int K) {
    (void)K;
    return g >= 1 && g <= 16;
}

int cc_tensor_score_ld(int K) { return (int)cc_align_up((size_t)K, TN); }

cudaError_t cc_launch_assign_tensor(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                    const float* C, int K, uint16_t* idx, float* dist, double* objective,
                                    int64_t* n_resolved, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_tensor<G>(ctx, L, X, N, C, K, idx, dist, nullptr, 0, nullptr, st)
    CC_TENSOR_DISPATCH(g, CALL)
#undef CALL
    if (e != cudaSuccess) return e;
    return cc_launch_assign_tail(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, st);
}

// Self-test of the bounded wait: one warp (a) waits on a barrier whose phase thread 0 completes,
// (b) waits on a barrier that nobody ever arrives on, with the given clock limit, and (c) waits on
// it again with the abort flag up.  out: {result of a, result of b, abort flag after b, result of c};
// cycles: {duration of b, duration of c}.
__global__ void __launch_bounds__(32)
wait_selftest_kernel(long long limit, int* __restrict__ out, long long* __restrict__ cycles) {
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars)));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + 1)));
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars)) : "memory");
    uint32_t ok_a = 1u, ok_b = 1u, ok_c = 1u;
    mbar_wait_acc(smem_u32(bars), 0, abort_flag, ok_a, limit);
    const long long t0 = clock64();
    mbar_wait_acc(smem_u32(bars + 1), 0, abort_flag, ok_b, limit);
    const long long t1 = clock64();
    const int flag_after_b = *abort_flag;
    mbar_wait_acc(smem_u32(bars + 1), 0, abort_flag, ok_c, limit);
    const long long t2 = clock64();
    if (threadIdx.x == 0) {
        out[0] = (int)ok_a; out[1] = (int)ok_b; out[2] = flag_after_b; out[3] = (int)ok_c;
        cycles[0] = t1 - t0; cycles[1] = t2 - t1;
    }
}

cudaError_t cc_launch_wait_selftest(long long limit, int* out_dev, long long* cycles_dev, cudaStream_t st) {
    wait_selftest_kernel<<<1, 32, 0, st>>>(limit, out_dev, cycles_dev);
    return cudaGetLastError();
}

cudaError_t cc_launch_tensor_scores(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                    const float* C, int K, float* scores, cudaStream_t st) {
    cudaError_t e = cudaSuccess;
    const int64_t ld = cc_tensor_score_ld(K);
#define CALL(G) e = launch_tensor<G>(ctx, L, X, N, C, K, nullptr, nullptr, scores, ld, nullptr, st)
    CC_TENSOR_DISPATCH(g, CALL)
#undef CALL
    return e;
}

// Verification aid: staging + finish kernel on scan results supplied by the caller (no scan, no exact stage).
cudaError_t cc_launch_tensor_finish_only(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g,
                                         const float* C, int K, const void* scan, uint16_t* idx, float* dist,
                                         cudaStream_t st) {
    cudaError_t e = cudaSuccess;
#define CALL(G) e = launch_tensor<G>(ctx, L, X, N, C, K, idx, dist, nullptr, 0, static_cast<const float2*>(scan), st)
    CC_TENSOR_DISPATCH(g, CALL)
#undef CALL
    return e;
}
