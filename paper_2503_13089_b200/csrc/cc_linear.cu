// Forward of the compressed linear layer (appendix listing): out = x . weight (+ bias) with
// weight = codebook[code] viewed as (in_features, out_features + pad), the padded columns dropped.
// The decoded weight is never written to memory: the kernel gathers codebook rows straight into the
// shared-memory operand of a tcgen05 GEMM.
//
// The product is computed transposed, out^T = weight^T . x^T, so that the WEIGHT is the 128-row
// operand of the MMA (128 out_features per CTA) and the tokens are its N dimension (16..256 columns,
// FP32 accumulators in TMEM).  A batch of a few tokens then costs a narrow MMA instead of a padded
// 128-row one, and the weight -- the large operand -- is gathered exactly once per token block.
//
// Per stage of 64 in_features the producer warps build
//   A: 128 out_features x 64 in_features, FP16, canonical K-major layout without swizzle.  One work
//      item = 8 consecutive in_features x one code group (g consecutive out_features): 8 codes, 8
//      codebook rows, transposed in registers into g rows of 16 bytes.
//   B: NT tokens x 64 in_features of x (16-byte copies).
// A ring of STAGES such stages feeds one MMA-issuing thread (4 MMAs of K = 16 per stage).  Each stage
// belongs to its own four producer warps, so the gathers of four stages (codes, then codebook rows:
// two dependent trips to L2) are in flight at once.  Full / empty
// mbarriers, every wait bounded by a clock limit (a wait that runs out raises CC_DEV_TIMEOUT, the
// CTA stops issuing work, skips its stores and still frees its tensor memory).
// With few tokens and few 128-row tiles the in_features are split across CTAs (split-K): every split
// writes its partial sums to scratch and a second kernel adds them in a fixed order, so the result
// does not depend on scheduling.
#include <cuda_fp16.h>

#include "cc_common.cuh"
#include "cc_tcgen05.cuh"

namespace {

constexpr int LM = 128;                 // out_features per CTA = MMA M = TMEM lanes
constexpr int LKB = 64;                 // in_features per pipeline stage
constexpr int LSTAGES = 4;              // at most; two where the 4-bit table leaves room for no more wide tiles
constexpr int LPROD = 512;              // producer threads (16 warps); warps 0..3 also run the epilogue
constexpr int LTHREADS = LPROD + 32;    // + the MMA warp
constexpr int LNT_MAX = 256;            // tokens per CTA = MMA N
// Operand tiles in shared memory: the K-major no-swizzle layout of 8 x 16-byte core matrices, with the two
// strides of the descriptor chosen against bank conflicts of the producers' 16-byte stores.  Neighbouring
// lanes of an A-tile store hold neighbouring code groups, i.e. rows g apart in one column of core matrices:
// 144 instead of 128 bytes between 8-row groups puts row r at 16-byte slot 9 (r / 8) + r % 8, and the eight
// lanes of a store phase then fall into eight different slots mod 8 for g = 2, 4, 8 (two by two for g = 16;
// at 128 bytes they all shared one or two).  Neighbouring lanes of a B-tile store hold neighbouring
// 8-column pieces of one token's row: 16 bytes more between the columns of core matrices does the same.
// Measured (4096 x 4096, g 4, K 65536): the B stride alone 0.772 -> 0.585 ms at 4096 tokens, 64 -> 50 us at
// 256; the A stride on top 35.7 -> 33.6 us at 64 tokens (87 -> 64 us at g = 8 on 8192 x 8192, 16 tokens) but
// 0.585 -> 0.807 ms at 4096 tokens, where the MMA's own reads of the wider-spaced A tile come to matter:
// the A tile is widened for token blocks of at most 64 only, and never beside the 4-bit table (no room).
__host__ __device__ constexpr int a_sbo(bool pad) { return pad ? 144 : 128; }
__host__ __device__ constexpr int a_lbo(bool pad) { return (LM / 8) * a_sbo(pad); }
__host__ __device__ constexpr int a_stage(bool pad) { return (LKB / 8) * a_lbo(pad); }   // bytes
__host__ __device__ constexpr int b_lbo(int nt) { return nt * 16 + 16; }
__host__ __device__ constexpr int b_stage_bytes(int nt) { return (LKB / 8) * b_lbo(nt); }
__device__ __forceinline__ int tile_off(int r, int kc, int lbo, int sbo) { return kc * lbo + (r >> 3) * sbo + (r & 7) * 16; }

// Row of G halves of the codebook as raw bit patterns.
template <int G>
__device__ __forceinline__ void load_code_row(const uint16_t* __restrict__ C16, int code, uint16_t* h) {
    const uint16_t* row = C16 + (int64_t)code * G;
    if constexpr (G % 8 == 0) {
#pragma unroll
        for (int v = 0; v < G / 8; ++v) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
            const unsigned w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) { h[v * 8 + 2 * k] = w[k] & 0xffffu; h[v * 8 + 2 * k + 1] = w[k] >> 16; }
        }
    } else if constexpr (G % 4 == 0) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            const uint2 u = __ldg(reinterpret_cast<const uint2*>(row) + v);
            h[v * 4] = u.x & 0xffffu; h[v * 4 + 1] = u.x >> 16; h[v * 4 + 2] = u.y & 0xffffu; h[v * 4 + 3] = u.y >> 16;
        }
    } else if constexpr (G % 2 == 0) {
#pragma unroll
        for (int v = 0; v < G / 2; ++v) {
            const unsigned u = __ldg(reinterpret_cast<const unsigned*>(row) + v);
            h[v * 2] = u & 0xffffu; h[v * 2 + 1] = u >> 16;
        }
    } else {
#pragma unroll
        for (int t = 0; t < G; ++t) h[t] = __ldg(row + t);
    }
}

// The same row as G / 2 32-bit words (even G).
template <int G>
__device__ __forceinline__ void load_code_row_words(const uint16_t* __restrict__ C16, int code, uint32_t* w) {
    const uint16_t* row = C16 + (int64_t)code * G;
    if constexpr (G % 8 == 0) {
#pragma unroll
        for (int v = 0; v < G / 8; ++v) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(row) + v);
            w[4 * v] = u.x; w[4 * v + 1] = u.y; w[4 * v + 2] = u.z; w[4 * v + 3] = u.w;
        }
    } else if constexpr (G % 4 == 0) {
#pragma unroll
        for (int v = 0; v < G / 4; ++v) {
            const uint2 u = __ldg(reinterpret_cast<const uint2*>(row) + v);
            w[2 * v] = u.x; w[2 * v + 1] = u.y;
        }
    } else {
#pragma unroll
        for (int v = 0; v < G / 2; ++v) w[v] = __ldg(reinterpret_cast<const unsigned*>(row) + v);
    }
}

// Quantised codebook (4 bits per value, two values per byte, low nibble first; Section 5.3): the whole
// table sits in shared memory, and a 256-entry table turns a byte into its two dequantised FP16 values
// (value = round-to-nearest-even FP16 of nibble * scale, the nibble a two's-complement number).
constexpr int LQ_TABLE_MAX = 128 * 1024;   // bytes of packed codebook that fit beside the stages
constexpr int LQ_BULK_PIECE = 32 * 1024;   // bytes per bulk copy of the table
constexpr int LQ_WIDE_FROM = 256;
constexpr int LQ_NT_MAX = 64;              // tokens per CTA when the table takes most of the shared memory

template <int G>
__device__ __forceinline__ void load_code_row_words_q(const unsigned char* __restrict__ qt,
                                                      const uint32_t* __restrict__ lut2, int code, uint32_t* w) {
    const unsigned char* row = qt + code * (G / 2);
#pragma unroll
    for (int v = 0; v < G / 2; ++v) w[v] = lut2[row[v]];
}

// blockIdx.x: tile of 128 out_features; blockIdx.y: block of NT tokens; blockIdx.z: split of the
// in_features (chunks_per_split stages each).  out: y itself (splits == 1) or this split's slab of
// partial sums, both M x d_out FP32 row-major.
// QUANT: the codebook is the packed 4-bit table `qtab` (K G / 2 bytes) with its scale instead of C16.
template <int G, bool QUANT, int STAGES>
__global__ void __launch_bounds__(LTHREADS, 1)
linear_forward_kernel(const uint16_t* __restrict__ x, int M, const uint16_t* __restrict__ C16,
                      const unsigned char* __restrict__ qtab, const float* __restrict__ qscale, int K,
                      const uint16_t* __restrict__ idx, int d_out, int d_in, int out_groups, int NT,
                      int a_pad, int tmem_cols, int chunks_per_split, float* __restrict__ out, int64_t split_stride,
                      const float* __restrict__ bias, unsigned* __restrict__ status, unsigned* __restrict__ arrived,
                      const float* __restrict__ bias_final, float* __restrict__ y_final) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int A_STAGE = a_stage(a_pad), A_LBO = a_lbo(a_pad), A_SBO = a_sbo(a_pad);
    const int b_stage = b_stage_bytes(NT), B_LBO = b_lbo(NT);
    unsigned char* sA = smem_raw;                                   // n_stages (2 or 4) tiles of 128 x 64
    constexpr int n_stages = STAGES, stage_threads = LPROD / STAGES;   // producer threads that fill one stage
    unsigned char* sB = sA + n_stages * A_STAGE;                    // n_stages tiles of NT x 64
    uint64_t* bars = reinterpret_cast<uint64_t*>(sB + n_stages * b_stage);
    uint64_t* full = bars, *empty = bars + LSTAGES, *acc_full = bars + 2 * LSTAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * LSTAGES + 1);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint64_t* qbar = bars + 16;                                                                  // QUANT only: the table has landed
    uint32_t* lut2 = reinterpret_cast<uint32_t*>(reinterpret_cast<unsigned char*>(bars) + 256);   // QUANT only
    unsigned char* qt = reinterpret_cast<unsigned char*>(lut2 + 256);                            // QUANT only

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int o0 = blockIdx.x * LM;
    const int m0 = blockIdx.y * NT;
    const int n_chunks_total = (d_in + LKB - 1) / LKB;
    const int chunk_first = blockIdx.z * chunks_per_split;
    int n_chunks = n_chunks_total - chunk_first;
    n_chunks = n_chunks < chunks_per_split ? n_chunks : chunks_per_split;
    if (n_chunks < 0) n_chunks = 0;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(full + s)), "r"(stage_threads));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(empty + s)));
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(acc_full)));
        if constexpr (QUANT) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(qbar)));
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if constexpr (QUANT) {
            // the packed codebook comes in as bulk copies (whole 16-byte pieces; the threads fetch the rest below)
            // while the CTA sets itself up; the producers wait for it before their first look-up
            const uint32_t bulk = (uint32_t)(K * (G / 2)) & ~15u, bar = smem_u32(qbar);
            if (bulk) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bulk) : "memory");
                for (uint32_t off = 0; off < bulk; off += LQ_BULK_PIECE) {
                    const uint32_t n = bulk - off < (uint32_t)LQ_BULK_PIECE ? bulk - off : (uint32_t)LQ_BULK_PIECE;
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(smem_u32(qt + off)), "l"(qtab + off), "r"(n), "r"(bar) : "memory");
                }
            } else {
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
            }
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(tmem_cols));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if constexpr (QUANT) {
        // the packed codebook and the byte -> two FP16 values table, once per CTA
        const float s = __ldg(qscale);
        if (tid < 256) {
            const int lo = ((tid & 15) ^ 8) - 8, hi = ((tid >> 4) ^ 8) - 8;     // sign-extended nibbles
            const unsigned a = __half_as_ushort(__float2half_rn(__fmul_rn((float)lo, s)));
            const unsigned b = __half_as_ushort(__float2half_rn(__fmul_rn((float)hi, s)));
            lut2[tid] = a | (b << 16);
        }
        const int bytes = K * (G / 2);
        for (int v = (bytes / 16) * 16 + tid; v < bytes; v += LTHREADS) qt[v] = __ldg(qtab + v);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp < LPROD / 32) {
        // ------------------------------------------------------------ producers
        // code groups that touch this tile of out_features
        const int grp_lo = o0 / G;
        int grp_hi = (o0 + LM - 1) / G;
        if (grp_hi > out_groups - 1) grp_hi = out_groups - 1;
        const int n_grp = grp_hi - grp_lo + 1;                      // >= 1: o0 < d_out <= out_groups * G
        const bool vec_x = (d_in % 8) == 0;
        bool ok = true;
        if constexpr (QUANT) ok = mbar_wait(smem_u32(qbar), 0, abort_flag);
        const int st = tid / stage_threads;                         // the stage this thread's group of warps fills
        const int ptid = tid - st * stage_threads;
        for (int c = st; c < n_chunks && ok; c += n_stages) {
            ok = mbar_wait(smem_u32(empty + st), ((c / n_stages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            unsigned char* tA = sA + st * A_STAGE;
            unsigned char* tB = sB + st * b_stage;
            const int i0 = (chunk_first + c) * LKB;
            // ---- A: gather, transpose, store.  item = (block of 8 in_features, code group)
            // IPT items per thread and pass: all their codes are requested first, then all their rows, so that a
            // pass costs two trips to L2 whatever IPT is (the rows of IPT items must fit the registers)
            constexpr int IPT = (G % 2 == 0 && G <= 8) ? 2 : 1;
            for (int item0 = ptid; item0 < (LKB / 8) * n_grp; item0 += IPT * stage_threads) {
                if constexpr (G % 2 == 0) {
                    // rows kept as 32-bit words (two out_features each): half the registers of a 16-bit copy
                    uint32_t v[IPT][8][G / 2];
                    int code[IPT][8];
                    int ibs[IPT], grps[IPT];
#pragma unroll
                    for (int q = 0; q < IPT; ++q) {
                        const int item = item0 + q * stage_threads;
                        const bool live = item < (LKB / 8) * n_grp;
                        ibs[q] = live ? item / n_grp : 0;
                        grps[q] = live ? grp_lo + (item - ibs[q] * n_grp) : -1;
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const int i = i0 + ibs[q] * 8 + u;
                            code[q][u] = (live && i < d_in) ? (int)__ldg(idx + (int64_t)i * out_groups + grps[q]) : -1;
                        }
                    }
#pragma unroll
                    for (int q = 0; q < IPT; ++q) {
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            if (code[q][u] >= 0) {
                                if constexpr (QUANT) load_code_row_words_q<G>(qt, lut2, code[q][u], v[q][u]);
                                else load_code_row_words<G>(C16, code[q][u], v[q][u]);
                            } else {
#pragma unroll
                                for (int t = 0; t < G / 2; ++t) v[q][u][t] = 0u;
                            }
                        }
                    }
#pragma unroll
                    for (int q = 0; q < IPT; ++q) {
                        if (grps[q] < 0) continue;
#pragma unroll
                        for (int t = 0; t < G; ++t) {
                            const int r = grps[q] * G + t - o0;     // row of the tile = out_feature - o0
                            if (r < 0 || r >= LM) continue;
                            const unsigned sel = (t & 1) ? 0x7632u : 0x5410u;   // high or low halves of two words
                            uint4 w;
                            w.x = __byte_perm(v[q][0][t / 2], v[q][1][t / 2], sel);
                            w.y = __byte_perm(v[q][2][t / 2], v[q][3][t / 2], sel);
                            w.z = __byte_perm(v[q][4][t / 2], v[q][5][t / 2], sel);
                            w.w = __byte_perm(v[q][6][t / 2], v[q][7][t / 2], sel);
                            *reinterpret_cast<uint4*>(tA + tile_off(r, ibs[q], A_LBO, A_SBO)) = w;
                        }
                    }
                } else {
                    const int ib = item0 / n_grp, grp = grp_lo + (item0 - (item0 / n_grp) * n_grp);
                    uint16_t v[8][G];
                    int code[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const int i = i0 + ib * 8 + u;
                        code[u] = (i < d_in) ? (int)__ldg(idx + (int64_t)i * out_groups + grp) : -1;
                    }
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (code[u] >= 0) {
                            load_code_row<G>(C16, code[u], v[u]);
                        } else {
#pragma unroll
                            for (int t = 0; t < G; ++t) v[u][t] = 0;
                        }
                    }
#pragma unroll
                    for (int t = 0; t < G; ++t) {
                        const int r = grp * G + t - o0;
                        if (r < 0 || r >= LM) continue;
                        uint4 w;
                        w.x = (unsigned)v[0][t] | ((unsigned)v[1][t] << 16);
                        w.y = (unsigned)v[2][t] | ((unsigned)v[3][t] << 16);
                        w.z = (unsigned)v[4][t] | ((unsigned)v[5][t] << 16);
                        w.w = (unsigned)v[6][t] | ((unsigned)v[7][t] << 16);
                        *reinterpret_cast<uint4*>(tA + tile_off(r, ib, A_LBO, A_SBO)) = w;
                    }
                }
            }
            // ---- B: the tokens' slice of x, 8 in_features (16 bytes) at a time, four loads in flight per thread
            const int n_b = NT * (LKB / 8);
            for (int item0 = ptid; item0 < n_b; item0 += 4 * stage_threads) {
                uint4 w[4];
#pragma unroll
                for (int u4 = 0; u4 < 4; ++u4) {
                    const int item = item0 + u4 * stage_threads;
                    const int kc = item % (LKB / 8), r = item / (LKB / 8);
                    const int m = m0 + r, i = i0 + kc * 8;
                    w[u4] = make_uint4(0u, 0u, 0u, 0u);
                    if (item < n_b && m < M && i < d_in) {
                        const uint16_t* src = x + (int64_t)m * d_in + i;
                        if (vec_x) {
                            w[u4] = __ldg(reinterpret_cast<const uint4*>(src));
                        } else {
                            unsigned short h[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u) h[u] = (i + u < d_in) ? __ldg(src + u) : (unsigned short)0;
                            w[u4].x = (unsigned)h[0] | ((unsigned)h[1] << 16);
                            w[u4].y = (unsigned)h[2] | ((unsigned)h[3] << 16);
                            w[u4].z = (unsigned)h[4] | ((unsigned)h[5] << 16);
                            w[u4].w = (unsigned)h[6] | ((unsigned)h[7] << 16);
                        }
                    }
                }
#pragma unroll
                for (int u4 = 0; u4 < 4; ++u4) {
                    const int item = item0 + u4 * stage_threads;
                    if (item < n_b) {
                        const int kc = item % (LKB / 8), r = item / (LKB / 8);
                        *reinterpret_cast<uint4*>(tB + tile_off(r, kc, B_LBO, 128)) = w[u4];
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> async proxy (MMA)
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(full + st)) : "memory");
        }
        // ------------------------------------------------------------ epilogue (warps 0..3)
        if (warp < 4) {
            ok = ok && mbar_wait(smem_u32(acc_full), 0, abort_flag);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int o = o0 + warp * 32 + lane;                    // TMEM lane = out_feature of the tile
            float* dst = out + (int64_t)blockIdx.z * split_stride;
            const float b = (bias && o < d_out) ? __ldg(bias + o) : 0.f;
            for (int cb = 0; cb < NT; cb += 32) {
                uint32_t v[32];
                TMEM_LD32(v, tmem + ((uint32_t)(warp * 32) << 16) + cb);
                TMEM_WAIT32(v);
                if (ok && !*abort_flag && o < d_out) {
#pragma unroll
                    for (int u = 0; u < 32; ++u) {
                        const int m = m0 + cb + u;
                        if (cb + u < NT && m < M)                   // 32 lanes write 32 consecutive out_features
                            dst[(int64_t)m * d_out + o] = (n_chunks > 0 ? __uint_as_float(v[u]) : 0.f) + b;
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ MMA warp: one thread issues
        if (lane == 0) {
            // kind::f16: D = F32 (bits 4-5 = 1), A = B = F16 (0), both K-major, N >> 3 at bit 17, M >> 4 at bit 24
            const int mma_n = NT < LNT_MAX ? NT : LNT_MAX;          // 512 tokens per CTA are two MMAs of 256 columns
            const uint32_t idesc = (1u << 4) | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(LM >> 4) << 24);
            const uint64_t descA0 = make_desc(smem_u32(sA), A_LBO, A_SBO);
            const uint64_t descB0 = make_desc(smem_u32(sB), B_LBO, 128);
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int st = c % n_stages;
                ok = mbar_wait(smem_u32(full + st), (c / n_stages) & 1, abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t descA = descA0 + (uint64_t)((st * A_STAGE) >> 4);
                const uint64_t descB = descB0 + (uint64_t)((st * b_stage) >> 4);
                for (int nb = 0; nb * mma_n < NT; ++nb) {
#pragma unroll
                    for (int s = 0; s < LKB / 16; ++s) {
                        const uint64_t da = descA + (uint64_t)((s * 2 * A_LBO) >> 4);
                        const uint64_t db = descB + (uint64_t)((s * 2 * B_LBO + nb * mma_n * 16) >> 4);   // 8-row groups are 128 bytes apart
                        const uint32_t acc = (c > 0 || s > 0) ? 1u : 0u;
                        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                     ::"r"(tmem + (uint32_t)(nb * mma_n)), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
                    }
                }
                // the stage may be refilled once these MMAs have read it
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(smem_u32(empty + st)) : "memory");
            }
            if (ok)
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(smem_u32(acc_full)) : "memory");
            else
                *abort_flag = 1;   // the epilogue's wait on acc_full returns at its next look at the flag
        }
    }
    // ---- split in_features: the CTA that finishes last among the splits of this tile adds the slabs, in split
    // order (the same bits whichever CTA that is), and the bias, with all its threads; it leaves the counter at
    // zero for the next call.  Every CTA counts itself, also one that gave up, so that the counter returns to zero.
    if (arrived) {
        __shared__ int last;
        unsigned* cnt = arrived + blockIdx.y * gridDim.x + blockIdx.x;
        __threadfence();                                            // this thread's slab stores before the count
        __syncthreads();
        if (tid == 0) last = atomicAdd(cnt, 1u) == gridDim.z - 1;
        __syncthreads();
        if (last) {
            __threadfence();
            const int m_end = (M - m0) < NT ? (M - m0) : NT;
            for (int e = tid; e < m_end * LM; e += LTHREADS) {
                const int mm = e / LM, o = o0 + (e - mm * LM);
                if (o >= d_out) continue;
                const float* src = out + (int64_t)(m0 + mm) * d_out + o;
                float sum = bias_final ? __ldg(bias_final + o) : 0.f;
                unsigned k = 0;
                for (; k + 4 <= gridDim.z; k += 4) {                // four loads in flight, added in split order
                    float pv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) pv[u] = __ldcg(src + (int64_t)(k + u) * split_stride);
#pragma unroll
                    for (int u = 0; u < 4; ++u) sum += pv[u];
                }
                for (; k < gridDim.z; ++k) sum += __ldcg(src + (int64_t)k * split_stride);
                y_final[(int64_t)(m0 + mm) * d_out + o] = sum;
            }
            if (tid == 0) *cnt = 0u;
        }
    }
    if (*abort_flag && lane == 0) atomicOr(status, CC_DEV_TIMEOUT);
    if constexpr (QUANT) {
        if (*abort_flag && tid == 0) {   // let the table's copies land before the CTA gives its shared memory back (bounded)
            const long long t0 = clock64();
            while (!mbar_try(smem_u32(qbar), 0) && clock64() - t0 < WAIT_LIMIT) {}
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols));
}

// y[m][o] = bias[o] + sum over the splits, in split order.
__global__ void __launch_bounds__(256)
linear_reduce_kernel(const float* __restrict__ partial, int splits, int64_t n, int d_out, const float* __restrict__ bias,
                     float* __restrict__ y) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
        float s = bias ? __ldg(bias + (int)(e % d_out)) : 0.f;
        for (int k = 0; k < splits; ++k) s += partial[(int64_t)k * n + e];
        y[e] = s;
    }
}

// ---- A handful of tokens (M <= 4; M <= 2 for g > 8) on the 4-bit codebook: no tensor core.  With so few columns the MMA
// idles and the tensor kernel's time is its producers' instructions; here a thread owns one code group (g
// out_features), walks down the in_features of its CTA's slice, looks each code up in the packed table in
// shared memory (one load of g / 2 bytes, then one load per 4-bit level from a 16-entry FP32 table, whose
// entries lie in 16 different banks: no conflicts whatever the levels) and adds x times the g values
// to M x g FP32 accumulators.  A product of two FP16 values is exact in FP32, so only the additions round.
// CTA = 64 code groups x 16 interleaved sub-slices of the in_features; the sixteen partial sums meet in
// shared memory in a fixed order, and the CTA writes its slab of partial sums (y itself when the layer
// needs a single slice per block of code groups); the slabs are added in slice order by the CTA that
// finishes last, or by linear_reduce_kernel: the same bits on every call.
// blockIdx.x: block of 64 code groups; blockIdx.y: slice of rows_per_split in_features.
constexpr int LG_THREADS = 1024, LG_GRPS = 64, LG_SUB = 16, LG_ROWS_MAX = 1024, LG_M_MAX = 4;

template <int G>
__device__ __forceinline__ void gemv_levels(const unsigned char* row, unsigned (&lv)[G]) {
    if constexpr (G == 4) {
        const unsigned w = *reinterpret_cast<const uint16_t*>(row);
#pragma unroll
        for (int t = 0; t < 4; ++t) lv[t] = (w >> (4 * t)) & 15u;
    } else if constexpr (G == 8) {
        const unsigned w = *reinterpret_cast<const unsigned*>(row);
#pragma unroll
        for (int t = 0; t < 8; ++t) lv[t] = (w >> (4 * t)) & 15u;
    } else if constexpr (G == 16) {
        const uint2 w = *reinterpret_cast<const uint2*>(row);
#pragma unroll
        for (int t = 0; t < 8; ++t) { lv[t] = (w.x >> (4 * t)) & 15u; lv[8 + t] = (w.y >> (4 * t)) & 15u; }
    } else {
#pragma unroll
        for (int b = 0; b < G / 2; ++b) { const unsigned w = row[b]; lv[2 * b] = w & 15u; lv[2 * b + 1] = w >> 4; }
    }
}

template <int G, int MT>
__global__ void __launch_bounds__(LG_THREADS, 1)
linear_gemv_q4_kernel(const uint16_t* __restrict__ x, int M, const unsigned char* __restrict__ qtab,
                      const float* __restrict__ qscale, int K, const uint16_t* __restrict__ idx, int d_out, int d_in,
                      int out_groups, int rows_per_split, float* __restrict__ out, int64_t split_stride,
                      unsigned* __restrict__ status, unsigned* __restrict__ arrived, const float* __restrict__ bias,
                      float* __restrict__ y, int direct) {
    extern __shared__ __align__(16) unsigned char gv_smem[];
    uint64_t* qbar = reinterpret_cast<uint64_t*>(gv_smem);                       // the table has landed
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gv_smem + 8);
    float* lut16 = reinterpret_cast<float*>(gv_smem + 64);                       // level -> value
    float* xs = reinterpret_cast<float*>(gv_smem + 128);                         // [row][MT]
    unsigned char* qt = gv_smem + 128 + ((size_t)rows_per_split * MT * 4 + 15) / 16 * 16;   // packed table, later the exchange area
    const int tid = threadIdx.x, gl = tid % LG_GRPS, sub = tid / LG_GRPS;
    const int i0 = blockIdx.y * rows_per_split;
    int rows = d_in - i0;
    rows = rows < rows_per_split ? rows : rows_per_split;
    const int bytes = K * (G / 2);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(qbar)));
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const uint32_t bulk = (uint32_t)bytes & ~15u, bar = smem_u32(qbar);
        if (bulk) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bulk) : "memory");
            for (uint32_t off = 0; off < bulk; off += LQ_BULK_PIECE) {
                const uint32_t n = bulk - off < (uint32_t)LQ_BULK_PIECE ? bulk - off : (uint32_t)LQ_BULK_PIECE;
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(smem_u32(qt + off)), "l"(qtab + off), "r"(n), "r"(bar) : "memory");
            }
        } else {
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
        }
    }
    for (int v = (bytes / 16) * 16 + tid; v < bytes; v += LG_THREADS) qt[v] = __ldg(qtab + v);
    if (tid < 16) {
        const int level = (tid ^ 8) - 8;                                         // sign-extended
        lut16[tid] = __half2float(__float2half_rn(__fmul_rn((float)level, __ldg(qscale))));   // the quantiser's own value
    }
    for (int e = tid; e < rows * MT; e += LG_THREADS) {
        const int r = e / MT, m = e - r * MT;
        xs[e] = (m < M) ? __half2float(__ushort_as_half(__ldg(x + (int64_t)m * d_in + i0 + r))) : 0.f;
    }
    __syncthreads();
    bool ok = true, waited = false;                        // the first codes are requested before the wait for the table

    const int grp = blockIdx.x * LG_GRPS + gl;
    const bool live = grp < out_groups;
    float acc[MT][G];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int t = 0; t < G; ++t) acc[m][t] = 0.f;
    const unsigned kmax = (unsigned)K - 1u;
    if (live) {
        const uint16_t* col = idx + (int64_t)i0 * out_groups + grp;
        constexpr int RB = 4;                                                    // rows whose codes are requested together
        for (int r0 = sub; r0 < rows; r0 += RB * LG_SUB) {
            unsigned code[RB];
#pragma unroll
            for (int u = 0; u < RB; ++u) {
                const int r = r0 + u * LG_SUB;
                code[u] = (r < rows) ? (unsigned)__ldg(col + (int64_t)r * out_groups) : 0u;
            }
            if (!waited) {
                ok = mbar_wait(smem_u32(qbar), 0, abort_flag);
                waited = true;
                if (!ok) break;
            }
#pragma unroll
            for (int u = 0; u < RB; ++u) {
                const int r = r0 + u * LG_SUB;
                if (r >= rows) break;
                unsigned lv[G];
                gemv_levels<G>(qt + (size_t)min(code[u], kmax) * (G / 2), lv);   // a code beyond the codebook must not leave it
                float xv[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) xv[m] = xs[r * MT + m];
#pragma unroll
                for (int t = 0; t < G; ++t) {
                    const float c = lut16[lv[t]];
#pragma unroll
                    for (int m = 0; m < MT; ++m) acc[m][t] = fmaf(xv[m], c, acc[m][t]);
                }
            }
        }
    }
    if (!waited) ok = mbar_wait(smem_u32(qbar), 0, abort_flag);   // nobody writes over the table's place before it has landed
    // ---- the sub-slices meet, one token at a time (the exchange area takes the table's place)
    __syncthreads();
    float* red = reinterpret_cast<float*>(qt);                                   // [LG_SUB - 1][G][LG_GRPS]
    float* dst = out + (int64_t)blockIdx.y * split_stride;
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        if (sub > 0) {
#pragma unroll
            for (int t = 0; t < G; ++t) red[((sub - 1) * G + t) * LG_GRPS + gl] = acc[m][t];
        }
        __syncthreads();
        if (sub == 0 && m < M && grp < out_groups && !*abort_flag) {
#pragma unroll
            for (int t = 0; t < G; ++t) {
                float s = acc[m][t];
#pragma unroll
                for (int q = 0; q < LG_SUB - 1; ++q) s += red[(q * G + t) * LG_GRPS + gl];
                const int o = grp * G + t;
                if (o < d_out) dst[(int64_t)m * d_out + o] = (direct && bias) ? s + __ldg(bias + o) : s;
            }
        }
        __syncthreads();
    }
    if (*abort_flag && tid == 0) {
        atomicOr(status, CC_DEV_TIMEOUT);
        const long long t0 = clock64();                                          // let the table's copies land (bounded)
        while (!mbar_try(smem_u32(qbar), 0) && clock64() - t0 < WAIT_LIMIT) {}
    }
    // ---- the CTA that finishes last among the slices of this block of code groups adds the slabs, in slice
    // order (the same bits whichever CTA that is), and the bias; it leaves the counter at zero for the next call.
    // Every CTA counts itself, also one that gave up, so that the counter always returns to zero.
    if (arrived) {
        __shared__ int last;
        __threadfence();                                                         // this thread's slab stores before the count
        __syncthreads();
        if (tid == 0) last = atomicAdd(arrived + blockIdx.x, 1u) == gridDim.y - 1;
        __syncthreads();
        if (last) {
            __threadfence();
            const int o_lo = blockIdx.x * LG_GRPS * G;
            int width = d_out - o_lo;
            width = width < LG_GRPS * G ? width : LG_GRPS * G;
            for (int e = tid; e < M * width; e += LG_THREADS) {
                const int m = e / width, o = o_lo + (e - m * width);
                const float* src = out + (int64_t)m * d_out + o;
                float sum = bias ? __ldg(bias + o) : 0.f;
                unsigned k = 0;
                for (; k + 8 <= gridDim.y; k += 8) {                             // eight loads in flight, added in slice order
                    float v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = __ldcg(src + (int64_t)(k + u) * split_stride);
#pragma unroll
                    for (int u = 0; u < 8; ++u) sum += v[u];
                }
                for (; k < gridDim.y; ++k) sum += __ldcg(src + (int64_t)k * split_stride);
                y[(int64_t)m * d_out + o] = sum;
            }
            if (tid == 0) arrived[blockIdx.x] = 0u;
        }
    }
}

struct GemvPlan { int o_blocks, splits, rows_per_split; };

GemvPlan gemv_plan(int64_t d_in, int out_groups, int sm_count) {
    GemvPlan p;
    p.o_blocks = (out_groups + LG_GRPS - 1) / LG_GRPS;
    int splits = sm_count / p.o_blocks;                                          // one CTA per SM where the shape allows
    if (splits < 1) splits = 1;
    if ((int64_t)splits * 16 > d_in) splits = (int)((d_in + 15) / 16);           // at least 16 in_features per CTA
    int64_t rows = (d_in + splits - 1) / splits;
    if (rows > LG_ROWS_MAX) rows = LG_ROWS_MAX;
    p.rows_per_split = (int)rows;
    p.splits = (int)((d_in + rows - 1) / rows);
    return p;
}

size_t gemv_smem(int g, int K, int rows, int mt) {
    size_t tail = (size_t)K * (g / 2);
    const size_t red = (size_t)(LG_SUB - 1) * g * LG_GRPS * 4;
    if (tail < red) tail = red;
    return 128 + ((size_t)rows * mt * 4 + 15) / 16 * 16 + (tail + 15) / 16 * 16;
}

struct LinearPlan { int NT, a_pad, stages, tmem_cols, o_tiles, tok_blocks, splits, chunks_per_split; size_t smem; };

// nt_max: tokens per CTA (256, or 64 with a quantised codebook in shared memory); table_bytes: that codebook.
LinearPlan linear_plan(int64_t M, int64_t d_out, int64_t d_in, int sm_count, int nt_max = LNT_MAX, size_t table_bytes = 0,
                       int g = 4) {
    LinearPlan p;
    const int64_t mt = M < nt_max ? M : nt_max;
    p.NT = (int)((mt + 15) / 16 * 16);
    // FP16 codebook with rows of at most 8 bytes, many tokens: the gathers of the weight tile bound a stage, so
    // one tile serves 512 tokens (two MMAs of 256 columns, all 512 TMEM columns) and the pipeline has two stages
    // of that size: 4096 x 4096, g 4, 4096 tokens 0.571 -> 0.464 ms.  With 16-byte rows (g = 8) there are half as
    // many gathers per weight and the coarser grid costs more than the reuse saves (1.62 -> 1.70 ms on 8192 x 8192).
    const bool wide = table_bytes == 0 && nt_max == LNT_MAX && M >= 2 * LNT_MAX && g <= 4;
    if (wide) p.NT = 2 * LNT_MAX;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.NT) p.tmem_cols *= 2;
    p.o_tiles = (int)((d_out + LM - 1) / LM);
    p.tok_blocks = (int)((M + p.NT - 1) / p.NT);
    const int chunks = (int)((d_in + LKB - 1) / LKB);
    int splits = sm_count / (p.o_tiles * p.tok_blocks);             // fill the SMs when there are few tiles
    if (splits > chunks / 4) splits = chunks / 4;                   // at least four stages of work per CTA
    if (splits < 1) splits = 1;
    p.chunks_per_split = (chunks + splits - 1) / splits;
    p.splits = (chunks + p.chunks_per_split - 1) / p.chunks_per_split;
    p.a_pad = (table_bytes == 0 && p.NT <= 64) ? 1 : 0;
    p.stages = (wide || (table_bytes != 0 && p.NT > LQ_NT_MAX)) ? 2 : LSTAGES;
    p.smem = (size_t)p.stages * (a_stage(p.a_pad) + (size_t)b_stage_bytes(p.NT)) + 256;
    if (table_bytes) p.smem += 1024 + (table_bytes + 15) / 16 * 16;
    return p;
}

}  // namespace

size_t cc_linear_scratch_bytes(int64_t M, int64_t d_out, int64_t d_in, int sm_count) {
    // enough for either form of the codebook: the quantised one takes narrower token blocks and may split more
    const LinearPlan p = linear_plan(M, d_out, d_in, sm_count);     // g <= 4: the shape with the fewest CTAs, hence the most splits
    const LinearPlan q = linear_plan(M, d_out, d_in, sm_count, LQ_NT_MAX, 16);
    int splits = p.splits > q.splits ? p.splits : q.splits;
    if (splits < 2) splits = 0;    // a single CTA per tile writes y itself
    if (M <= LG_M_MAX) {
        // the few-token kernel of the quantised codebook always goes through its slabs; the most slices come
        // with the fewest blocks of code groups, i.e. at g = 16
        const GemvPlan v = gemv_plan(d_in, (int)((d_out + 15) / 16), sm_count);
        if (v.splits > splits) splits = v.splits;
    }
    return CC_STATUS_BYTES + (size_t)splits * (size_t)M * (size_t)d_out * 4;
}

int cc_linear_q_table_max(void) { return LQ_TABLE_MAX; }

#define CC_LINEAR_DISPATCH(g, CALL)                                                                 \
    switch (g) {                                                                                    \
        case 1: CALL(1); break;   case 2: CALL(2); break;   case 3: CALL(3); break;                 \
        case 4: CALL(4); break;   case 5: CALL(5); break;   case 6: CALL(6); break;                 \
        case 7: CALL(7); break;   case 8: CALL(8); break;   case 9: CALL(9); break;                 \
        case 10: CALL(10); break; case 11: CALL(11); break; case 12: CALL(12); break;               \
        case 13: CALL(13); break; case 14: CALL(14); break; case 15: CALL(15); break;               \
        case 16: CALL(16); break;                                                                   \
        default: return cudaErrorInvalidValue;                                                      \
    }

namespace {

template <int G, bool QUANT, int STAGES>
cudaError_t launch_linear_s(cc_ctx* ctx, const LinearPlan& p, const uint16_t* x, int M, const uint16_t* C16,
                            const unsigned char* qtab, const float* qscale, int K, const uint16_t* idx, int d_out, int d_in,
                            int out_groups, float* out, int64_t split_stride, const float* bias, unsigned* status,
                            unsigned* arrived, const float* bias_final, float* y_final, cudaStream_t st) {
    static bool attr_dev[64] = {};
    bool& have = attr_dev[ctx->device & 63];
    if (!have) {
        // the largest shape of each kind: four stages of 64 tokens or two of 256 beside the table; four stages of
        // 256 tokens or two of 512 without it
        const int max_smem = QUANT ? (STAGES == 2 ? (int)(2 * (a_stage(false) + b_stage_bytes(LNT_MAX)) + 256 + 1024 + LQ_TABLE_MAX)
                                                  : (int)(LSTAGES * (a_stage(false) + b_stage_bytes(LQ_NT_MAX)) + 256 + 1024 + LQ_TABLE_MAX))
                                   : (STAGES == 2 ? (int)(2 * (a_stage(false) + b_stage_bytes(2 * LNT_MAX)) + 256)
                                                  : (int)(LSTAGES * (a_stage(true) + b_stage_bytes(LNT_MAX)) + 256));
        const cudaError_t e = cudaFuncSetAttribute(linear_forward_kernel<G, QUANT, STAGES>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
        if (e != cudaSuccess) return e;
        have = true;
    }
    const dim3 grid(p.o_tiles, p.tok_blocks, p.splits);
    linear_forward_kernel<G, QUANT, STAGES><<<grid, LTHREADS, p.smem, st>>>(x, M, C16, qtab, qscale, K, idx, d_out, d_in,
                                                                            out_groups, p.NT, p.a_pad, p.tmem_cols,
                                                                            p.chunks_per_split, out, split_stride, bias, status, arrived,
                                                                            bias_final, y_final);
    return cudaGetLastError();
}

// Two stages exist where the plan can ask for them: beside the 4-bit table, and for rows of at most 8 bytes.
template <int G, bool QUANT>
cudaError_t launch_linear(cc_ctx* ctx, const LinearPlan& p, const uint16_t* x, int M, const uint16_t* C16,
                          const unsigned char* qtab, const float* qscale, int K, const uint16_t* idx, int d_out, int d_in,
                          int out_groups, float* out, int64_t split_stride, const float* bias, unsigned* status,
                          unsigned* arrived, const float* bias_final, float* y_final, cudaStream_t st) {
    if constexpr (QUANT || G <= 4) {
        if (p.stages == 2)
            return launch_linear_s<G, QUANT, 2>(ctx, p, x, M, C16, qtab, qscale, K, idx, d_out, d_in, out_groups, out,
                                                split_stride, bias, status, arrived, bias_final, y_final, st);
    }
    if (p.stages != LSTAGES) return cudaErrorInvalidValue;
    return launch_linear_s<G, QUANT, LSTAGES>(ctx, p, x, M, C16, qtab, qscale, K, idx, d_out, d_in, out_groups, out,
                                              split_stride, bias, status, arrived, bias_final, y_final, st);
}

}  // namespace

namespace {

template <int G, int MT>
cudaError_t launch_gemv(cc_ctx* ctx, const GemvPlan& p, const uint16_t* x, int M, const unsigned char* qtab,
                        const float* qscale, int K, const uint16_t* idx, int d_out, int d_in, int out_groups, float* out,
                        int64_t split_stride, unsigned* status, unsigned* arrived, const float* bias, float* y,
                        cudaStream_t st) {
    static bool attr_dev[64] = {};
    bool& have = attr_dev[ctx->device & 63];
    if (!have) {
        const cudaError_t e = cudaFuncSetAttribute(linear_gemv_q4_kernel<G, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)gemv_smem(G, LQ_TABLE_MAX / (G / 2), LG_ROWS_MAX, MT));
        if (e != cudaSuccess) return e;
        have = true;
    }
    const dim3 grid(p.o_blocks, p.splits);
    linear_gemv_q4_kernel<G, MT><<<grid, LG_THREADS, gemv_smem(G, K, p.rows_per_split, MT), st>>>(
        x, M, qtab, qscale, K, idx, d_out, d_in, out_groups, p.rows_per_split, out, split_stride, status, arrived, bias, y, p.splits == 1);
    return cudaGetLastError();
}

// Tokens padded to 1, 2 or 4 (from 8 on the tensor kernel is as fast); M x g accumulators must fit the
// registers of 1024 threads per SM.
constexpr int gemv_tokens(int g) { return g <= 8 ? 4 : 2; }

template <int G>
cudaError_t launch_gemv_m(cc_ctx* ctx, const GemvPlan& p, const uint16_t* x, int M, const unsigned char* qtab,
                          const float* qscale, int K, const uint16_t* idx, int d_out, int d_in, int out_groups, float* out,
                          int64_t split_stride, unsigned* status, unsigned* arrived, const float* bias, float* y,
                          cudaStream_t st) {
    if (M == 1) return launch_gemv<G, 1>(ctx, p, x, M, qtab, qscale, K, idx, d_out, d_in, out_groups, out, split_stride, status, arrived, bias, y, st);
    if (M == 2) return launch_gemv<G, 2>(ctx, p, x, M, qtab, qscale, K, idx, d_out, d_in, out_groups, out, split_stride, status, arrived, bias, y, st);
    if constexpr (gemv_tokens(G) >= 4) {
        if (M <= 4) return launch_gemv<G, 4>(ctx, p, x, M, qtab, qscale, K, idx, d_out, d_in, out_groups, out, split_stride, status, arrived, bias, y, st);
    }
    if constexpr (gemv_tokens(G) >= 8) {
        if (M <= 8) return launch_gemv<G, 8>(ctx, p, x, M, qtab, qscale, K, idx, d_out, d_in, out_groups, out, split_stride, status, arrived, bias, y, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

// qtab == nullptr: FP16 codebook C16; otherwise the packed 4-bit codebook with its scale (even g only).
cudaError_t cc_launch_linear_forward(cc_ctx* ctx, const uint16_t* x, int64_t M, const uint16_t* C16,
                                     const unsigned char* qtab, const float* qscale, int K, int g, const uint16_t* idx,
                                     int64_t d_out, int64_t d_in, const float* bias, float* y, cudaStream_t st) {
    // beside the table: token blocks of 64 with four stages, or, from LQ_WIDE_FROM tokens on, of 256 with two
    const LinearPlan p = qtab ? linear_plan(M, d_out, d_in, ctx->sm_count, M >= LQ_WIDE_FROM ? LNT_MAX : LQ_NT_MAX, (size_t)K * (g / 2))
                              : linear_plan(M, d_out, d_in, ctx->sm_count, LNT_MAX, 0, g);
    char* ws = static_cast<char*>(ctx->ws);
    unsigned* status = reinterpret_cast<unsigned*>(ws);
    float* partial = reinterpret_cast<float*>(ws + CC_STATUS_BYTES);
    const int out_groups = (int)((d_out + g - 1) / g);
    const int64_t n = M * d_out;
    cudaError_t e = cudaSuccess;
    if (qtab && M <= gemv_tokens(g)) {
        // a handful of tokens: the shared-memory look-up kernel, then the same reduction (it also adds the bias)
        const GemvPlan v = gemv_plan(d_in, out_groups, ctx->sm_count);
        unsigned* arrived = nullptr;
        {
            ProfScope ps(ctx, CC_K_LINEAR, st);
            // counters of the finished slices: the words of the status block kept for this (zero since
            // cc_set_workspace, put back to zero by the kernel); with more blocks than counters the reduction
            // is a kernel of its own
            arrived = (v.splits > 1 && v.o_blocks <= CC_ARRIVAL_COUNTERS) ? status + CC_ARRIVAL_WORD : nullptr;
            float* slabs = v.splits == 1 ? y : partial;          // a single slice writes y (and the bias) itself
#define CALL(G) e = launch_gemv_m<G>(ctx, v, x, (int)M, qtab, qscale, K, idx, (int)d_out, (int)d_in, out_groups, slabs, n, status, arrived, bias, y, st)
            switch (g) {
                case 2: CALL(2); break;   case 4: CALL(4); break;   case 6: CALL(6); break;   case 8: CALL(8); break;
                case 10: CALL(10); break; case 12: CALL(12); break; case 14: CALL(14); break; case 16: CALL(16); break;
                default: return cudaErrorInvalidValue;
            }
#undef CALL
        }
        if (e != cudaSuccess || arrived || v.splits == 1) return e;
        ProfScope ps(ctx, CC_K_LINEAR_REDUCE, st);
        int64_t blocks = (n + 255) / 256;
        const int64_t cap = (int64_t)ctx->sm_count * 8;
        if (blocks > cap) blocks = cap;
        linear_reduce_kernel<<<(unsigned)blocks, 256, 0, st>>>(partial, v.splits, n, (int)d_out, bias, y);
        return cudaGetLastError();
    }
    bool fused = false;
    {
        ProfScope ps(ctx, CC_K_LINEAR, st);
        float* out = p.splits > 1 ? partial : y;
        const float* b = p.splits > 1 ? nullptr : bias;
        // split in_features: up to 16 tokens the last CTA of a tile adds the slabs (one launch: 33.5 against 38 us
        // at one token, 36 against 38 at 16; at 64 tokens the lone CTA's tail costs more than the second launch:
        // 44 against 40 us), if the status block has a counter for every tile; else the reduction is a kernel of its own
        fused = p.splits > 1 && M <= 16 && (int64_t)p.o_tiles * p.tok_blocks <= CC_ARRIVAL_COUNTERS;
        unsigned* arrived = fused ? status + CC_ARRIVAL_WORD : nullptr;
        if (qtab) {
#define CALL(G) e = launch_linear<G, true>(ctx, p, x, (int)M, nullptr, qtab, qscale, K, idx, (int)d_out, (int)d_in, out_groups, out, n, b, status, arrived, bias, y, st)
            switch (g) {
                case 2: CALL(2); break;   case 4: CALL(4); break;   case 6: CALL(6); break;   case 8: CALL(8); break;
                case 10: CALL(10); break; case 12: CALL(12); break; case 14: CALL(14); break; case 16: CALL(16); break;
                default: return cudaErrorInvalidValue;
            }
#undef CALL
        } else {
#define CALL(G) e = launch_linear<G, false>(ctx, p, x, (int)M, C16, nullptr, nullptr, K, idx, (int)d_out, (int)d_in, out_groups, out, n, b, status, arrived, bias, y, st)
            CC_LINEAR_DISPATCH(g, CALL)
#undef CALL
        }
    }
    if (e != cudaSuccess) return e;
    if (p.splits > 1 && !fused) {
        ProfScope ps(ctx, CC_K_LINEAR_REDUCE, st);
        int64_t blocks = (n + 255) / 256;
        const int64_t cap = (int64_t)ctx->sm_count * 8;
        if (blocks > cap) blocks = cap;
        linear_reduce_kernel<<<(unsigned)blocks, 256, 0, st>>>(partial, p.splits, n, (int)d_out, bias, y);
        e = cudaGetLastError();
    }
    return e;
}
