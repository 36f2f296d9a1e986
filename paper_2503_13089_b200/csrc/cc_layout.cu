// Data-movement kernels: cutting W into sub-vectors (Section 3.1 footnote / appendix listing),
// the codebook gather that rebuilds W (Section 3.1, "codebook[code]" in the listing), the
// initial-codebook gather and the FP32 -> FP16 codebook export (Section 3.2).
#include "cc_common.cuh"

namespace {

constexpr int TD = 64;   // transpose tile edge (elements)

// PAPER_T reshape is a 2-D transpose with zero padding: X viewed as d_in x out_pad holds W^T.
// 64 x 64 tiles go through shared memory so that both the reads (along d_in) and the writes
// (along out_pad) are contiguous.
__global__ void __launch_bounds__(256)
reshape_transpose_kernel(const uint16_t* __restrict__ W, int64_t d_out, int64_t d_in, int64_t out_pad,
                         uint16_t* __restrict__ X) {
    __shared__ uint16_t tile[TD][TD + 2];
    const int64_t i0 = (int64_t)blockIdx.x * TD, o0 = (int64_t)blockIdx.y * TD;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    for (int r = ty; r < TD; r += 4) {          // r: out_feature within the tile, tx: in_feature
        const int64_t o = o0 + r, i = i0 + tx;
        tile[r][tx] = (o < d_out && i < d_in) ? W[o * d_in + i] : (uint16_t)0;
    }
    __syncthreads();
    for (int r = ty; r < TD; r += 4) {          // r: in_feature within the tile, tx: out_feature
        const int64_t i = i0 + r, o = o0 + tx;
        if (i < d_in && o < out_pad) X[i * out_pad + o] = tile[tx][r];
    }
}

// ---- 16-byte versions of the two transposing kernels (taken when every row is a whole number of
// 8-element groups).  A 64 x 64 tile goes through shared memory as 32-bit words (two elements),
// row r at word offset 33 r + 4 (r / 32): with that stride both the row-wise writes (four words per
// thread) and the column-wise reads (one word from each of eight rows) touch 32 different banks
// per warp.  A thread of the second phase reads eight words, i.e. a 8 x 2 block, and writes two
// 16-byte vectors into two adjacent output rows.
constexpr int TILE_WORDS = TD * 33 + 4;

__device__ __forceinline__ int tile_row(int r) { return r * 33 + (r >> 5) * 4; }

__device__ __forceinline__ void tile_put8(unsigned* tile, int r, int c, uint4 v) {
    unsigned* dst = tile + tile_row(r) + 4 * c;
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
}

// Elements [8c+k][2rp] (k = 0..7) into `even`, [8c+k][2rp+1] into `odd`.
__device__ __forceinline__ void tile_column8x2(const unsigned* tile, int c, int rp, uint4& even, uint4& odd) {
    unsigned w[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) w[k] = tile[tile_row(8 * c + k) + rp];
    even.x = __byte_perm(w[0], w[1], 0x5410); odd.x = __byte_perm(w[0], w[1], 0x7632);
    even.y = __byte_perm(w[2], w[3], 0x5410); odd.y = __byte_perm(w[2], w[3], 0x7632);
    even.z = __byte_perm(w[4], w[5], 0x5410); odd.z = __byte_perm(w[4], w[5], 0x7632);
    even.w = __byte_perm(w[6], w[7], 0x5410); odd.w = __byte_perm(w[6], w[7], 0x7632);
}

// PAPER_T reshape; needs d_in % 8 == 0 and out_pad % 8 == 0.
__global__ void __launch_bounds__(256)
reshape_transpose_vec_kernel(const uint16_t* __restrict__ W, int64_t d_out, int64_t d_in, int64_t out_pad,
                             uint16_t* __restrict__ X) {
    __shared__ unsigned tile[TILE_WORDS];
    const int64_t i0 = (int64_t)blockIdx.x * TD, o0 = (int64_t)blockIdx.y * TD;
    const int c = threadIdx.x & 7, r0 = threadIdx.x >> 3;
#pragma unroll
    for (int p = 0; p < 2; ++p) {               // rows: out_features, vectors along in_features
        const int r = r0 + 32 * p;
        const int64_t o = o0 + r, i = i0 + 8 * c;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (o < d_out && i < d_in) v = __ldg(reinterpret_cast<const uint4*>(W + o * d_in + i));
        tile_put8(tile, r, c, v);
    }
    __syncthreads();
    {                                           // rows: in_features 2 r0, 2 r0 + 1, vectors along out_features
        uint4 even, odd;
        tile_column8x2(tile, c, r0, even, odd);
        const int64_t i = i0 + 2 * r0, o = o0 + 8 * c;
        if (o < out_pad) {
            if (i < d_in) *reinterpret_cast<uint4*>(X + i * out_pad + o) = even;
            if (i + 1 < d_in) *reinterpret_cast<uint4*>(X + (i + 1) * out_pad + o) = odd;
        }
    }
}

// PAPER_T decode for g = 4, 8, 16; needs d_in % 8 == 0 and out_pad % 8 == 0.  A group of 8
// consecutive out_features of one in_feature is two codes (g = 4), one code (g = 8) or half a
// code (g = 16): the codebook is read in 8- or 16-byte pieces.
template <int G>
__global__ void __launch_bounds__(256)
decode_transpose_vec_kernel(const uint16_t* __restrict__ C16, const uint16_t* __restrict__ idx, int64_t d_out,
                            int64_t d_in, int64_t out_pad, uint16_t* __restrict__ W_hat) {
    __shared__ unsigned tile[TILE_WORDS];
    const int64_t i0 = (int64_t)blockIdx.x * TD, o0 = (int64_t)blockIdx.y * TD;
    const int c = threadIdx.x & 7, r0 = threadIdx.x >> 3;
#pragma unroll
    for (int p = 0; p < 2; ++p) {               // rows: in_features, vectors along out_features
        const int r = r0 + 32 * p;
        const int64_t i = i0 + r, o = o0 + 8 * c;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (i < d_in && o < out_pad) {
            const int64_t flat = i * out_pad + o;
            const int64_t n = flat / G;
            if constexpr (G == 4) {             // flat is a multiple of 8: n is even, both codes in one word
                const unsigned two = __ldg(reinterpret_cast<const unsigned*>(idx + n));
                const uint2 a = __ldg(reinterpret_cast<const uint2*>(C16 + (int64_t)(two & 0xffffu) * 4));
                const uint2 b = __ldg(reinterpret_cast<const uint2*>(C16 + (int64_t)(two >> 16) * 4));
                v = make_uint4(a.x, a.y, b.x, b.y);
            } else {
                v = __ldg(reinterpret_cast<const uint4*>(C16 + (int64_t)__ldg(idx + n) * G + (flat - n * G)));
            }
        }
        tile_put8(tile, r, c, v);
    }
    __syncthreads();
    {                                           // rows: out_features 2 r0, 2 r0 + 1, vectors along in_features
        uint4 even, odd;
        tile_column8x2(tile, c, r0, even, odd);
        const int64_t o = o0 + 2 * r0, i = i0 + 8 * c;
        if (i < d_in) {
            if (o < d_out) *reinterpret_cast<uint4*>(W_hat + o * d_in + i) = even;
            if (o + 1 < d_out) *reinterpret_cast<uint4*>(W_hat + (o + 1) * d_in + i) = odd;
        }
    }
}

// PAPER_T decode of large matrices for g = 8 and 16: persistent CTAs walk over the tiles with the loads of the
// next tiles already in flight (the codes of tile k+2 and the codebook rows of tile k+1 are
// requested before tile k goes through shared memory), because a tile's chain DRAM (codes) ->
// gather -> transpose -> store is otherwise paid once per tile and four to eight resident CTAs do
// not hide it.  TABLE: the whole FP16 codebook (at most kTableMaxBytes) is staged in shared memory
// once per CTA and the gather is a shared-memory read at the time of use.
constexpr int kTileBytes = (TILE_WORDS * 4 + 15) / 16 * 16;
constexpr int kTableMaxBytes = 46 * 1024;   // four CTAs per SM with their tiles
constexpr int kPipeMaxTableBytes = 128 * 1024;

struct DecodeCodes {
    unsigned code[2];   // element offset of the 8 values in the codebook
    unsigned live;      // bit p: row p of this thread lies inside the matrix
};

struct DecodeTile { int bx, by; };   // tile coordinates along in_features / out_features

// Tile t + gridDim.x from tile t without a division.
__device__ __forceinline__ void decode_next_tile(DecodeTile& p, int step_x, int step_y, int tiles_x) {
    p.bx += step_x;
    p.by += step_y;
    if (p.bx >= tiles_x) { p.bx -= tiles_x; ++p.by; }
}

// opg = out_pad / G: codes per in_feature.  out_pad is a multiple of G and a tile starts at a
// multiple of 64 out_features, so the position inside the sub-vector is (8 c) mod G.
template <int G>
__device__ __forceinline__ void decode_load_codes(const uint16_t* __restrict__ idx, DecodeTile p, int tiles_y, int r0,
                                                  int c, int64_t d_in, int64_t out_pad, int64_t opg, unsigned kmax,
                                                  DecodeCodes& s) {
    s.live = 0u;
    s.code[0] = 0u;
    s.code[1] = 0u;
    if (p.by >= tiles_y) return;
    const int64_t o = (int64_t)p.by * TD + 8 * c;
    if (o >= out_pad) return;
    const int64_t i = (int64_t)p.bx * TD + r0;
    const uint16_t* src = idx + i * opg + (o / G);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        if (i + 32 * q < d_in) {
            s.live |= 1u << q;
            // a code beyond the codebook must not leave it
            s.code[q] = min((unsigned)__ldg(src + 32 * q * opg), kmax) * (unsigned)G + ((8u * c) & (unsigned)(G - 1));
        }
    }
}

template <int G>
__device__ __forceinline__ void decode_gather(const uint16_t* table, const DecodeCodes& s, uint4 (&v)[2]) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        v[q] = make_uint4(0u, 0u, 0u, 0u);
        if (s.live >> q & 1u) {
            v[q] = *reinterpret_cast<const uint4*>(table + s.code[q]);
        }
    }
}

// One tile through shared memory and out to W_hat.
__device__ __forceinline__ void decode_emit(unsigned* tile, DecodeTile p, int r0, int c, const uint4 (&v)[2],
                                            int64_t d_out, int64_t d_in, uint16_t* __restrict__ W_hat) {
    tile_put8(tile, r0, c, v[0]);
    tile_put8(tile, r0 + 32, c, v[1]);
    __syncthreads();
    uint4 even, odd;
    tile_column8x2(tile, c, r0, even, odd);
    const int64_t o = (int64_t)p.by * TD + 2 * r0, i = (int64_t)p.bx * TD + 8 * c;
    if (i < d_in) {
        uint16_t* dst = W_hat + o * d_in + i;
        if (o < d_out) *reinterpret_cast<uint4*>(dst) = even;
        if (o + 1 < d_out) *reinterpret_cast<uint4*>(dst + d_in) = odd;
    }
    __syncthreads();                            // the tile is free for the next round
}

// The loop is unrolled by two so that the two register sets (A, B) keep their roles: a register
// that still waits for a load is never copied.
template <int G, bool TABLE>
__global__ void __launch_bounds__(256, 4)
decode_transpose_pipe_kernel(const uint16_t* __restrict__ C16, const uint16_t* __restrict__ idx, int K, int64_t d_out,
                             int64_t d_in, int64_t out_pad, uint16_t* __restrict__ W_hat, int tiles_x, int tiles_y) {
    extern __shared__ __align__(16) unsigned char decode_smem[];
    unsigned* tile = reinterpret_cast<unsigned*>(decode_smem);
    const uint16_t* table = C16;
    if constexpr (TABLE) {
        uint16_t* staged = reinterpret_cast<uint16_t*>(decode_smem + kTileBytes);
        for (int v = threadIdx.x; v < K * G / 4; v += 256)
            reinterpret_cast<uint2*>(staged)[v] = __ldg(reinterpret_cast<const uint2*>(C16) + v);
        table = staged;
    }
    const int c = threadIdx.x & 7, r0 = threadIdx.x >> 3;
    const unsigned kmax = (unsigned)K - 1u;
    const int64_t opg = out_pad / G;
    const int step_x = (int)(gridDim.x % (unsigned)tiles_x), step_y = (int)(gridDim.x / (unsigned)tiles_x);
    DecodeTile t0 = {(int)(blockIdx.x % (unsigned)tiles_x), (int)(blockIdx.x / (unsigned)tiles_x)};
#define CC_DECODE_CODES(P, S) decode_load_codes<G>(idx, P, tiles_y, r0, c, d_in, out_pad, opg, kmax, S)
    DecodeCodes sA, sB;
    uint4 vA[2], vB[2];
    CC_DECODE_CODES(t0, sA);
    DecodeTile t1 = t0;
    decode_next_tile(t1, step_x, step_y, tiles_x);
    if constexpr (TABLE) {
        __syncthreads();                        // the table is staged
        while (t0.by < tiles_y) {
            CC_DECODE_CODES(t1, sB);
            decode_gather<G>(table, sA, vA);
            decode_emit(tile, t0, r0, c, vA, d_out, d_in, W_hat);
            if (t1.by >= tiles_y) break;
            t0 = t1;
            decode_next_tile(t0, step_x, step_y, tiles_x);
            CC_DECODE_CODES(t0, sA);
            decode_gather<G>(table, sB, vB);
            decode_emit(tile, t1, r0, c, vB, d_out, d_in, W_hat);
            t1 = t0;
            decode_next_tile(t1, step_x, step_y, tiles_x);
        }
    } else {
        CC_DECODE_CODES(t1, sB);
        decode_gather<G>(table, sA, vA);
        while (t0.by < tiles_y) {
            DecodeTile t2 = t1;
            decode_next_tile(t2, step_x, step_y, tiles_x);
            decode_gather<G>(table, sB, vB);    // tile t1 (nothing live past the last tile)
            CC_DECODE_CODES(t2, sA);
            decode_emit(tile, t0, r0, c, vA, d_out, d_in, W_hat);
            if (t1.by >= tiles_y) break;
            t0 = t2;
            decode_next_tile(t0, step_x, step_y, tiles_x);
            decode_gather<G>(table, sA, vA);    // tile t2
            CC_DECODE_CODES(t0, sB);
            decode_emit(tile, t1, r0, c, vB, d_out, d_in, W_hat);
            t1 = t0;
            t0 = t2;
        }
    }
#undef CC_DECODE_CODES
}

template <int G>
cudaError_t launch_decode_pipe(int sm_count, const uint16_t* C16, const uint16_t* idx, int K, int64_t d_out,
                               int64_t d_in, int64_t out_pad, uint16_t* W_hat, int tiles_x, int tiles_y,
                               cudaStream_t st) {
    const int64_t n_tiles = (int64_t)tiles_x * tiles_y;
    const bool staged = K * G * 2 <= kTableMaxBytes;
    const int smem = kTileBytes + (staged ? K * G * 2 : 0);
    int64_t grid = (int64_t)sm_count * 4;
    if (grid > n_tiles) grid = n_tiles;
    if (staged) {
        const cudaError_t e = cudaFuncSetAttribute(decode_transpose_pipe_kernel<G, true>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        decode_transpose_pipe_kernel<G, true><<<(unsigned)grid, 256, smem, st>>>(C16, idx, K, d_out, d_in, out_pad,
                                                                                 W_hat, tiles_x, tiles_y);
    } else {
        decode_transpose_pipe_kernel<G, false><<<(unsigned)grid, 256, smem, st>>>(C16, idx, K, d_out, d_in, out_pad,
                                                                                  W_hat, tiles_x, tiles_y);
    }
    return cudaGetLastError();
}

// ROWS reshape: copy each row, padding it to in_pad elements.
__global__ void __launch_bounds__(256)
reshape_rows_kernel(const uint16_t* __restrict__ W, int64_t d_out, int64_t d_in, int64_t in_pad,
                    uint16_t* __restrict__ X) {
    const int64_t total = d_out * in_pad;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t o = e / in_pad, i = e - o * in_pad;
        X[e] = (i < d_in) ? W[o * d_in + i] : (uint16_t)0;
    }
}

// PAPER_T decode: W_hat[o][i] = C16[idx[(i*out_pad + o) / g]][(i*out_pad + o) % g].  The gather
// runs along o (contiguous in the codes and in each codebook row), the store along i.
__global__ void __launch_bounds__(256)
decode_transpose_kernel(const uint16_t* __restrict__ C16, int g, const uint16_t* __restrict__ idx, int64_t d_out,
                        int64_t d_in, int64_t out_pad, uint16_t* __restrict__ W_hat) {
    __shared__ uint16_t tile[TD][TD + 2];
    const int64_t i0 = (int64_t)blockIdx.x * TD, o0 = (int64_t)blockIdx.y * TD;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    for (int r = ty; r < TD; r += 4) {          // r: in_feature, tx: out_feature
        const int64_t i = i0 + r, o = o0 + tx;
        uint16_t v = 0;
        if (i < d_in && o < d_out) {
            const int64_t flat = i * out_pad + o;
            const int64_t n = flat / g;
            v = __ldg(C16 + (int64_t)__ldg(idx + n) * g + (flat - n * g));
        }
        tile[r][tx] = v;
    }
    __syncthreads();
    for (int r = ty; r < TD; r += 4) {          // r: out_feature, tx: in_feature
        const int64_t o = o0 + r, i = i0 + tx;
        if (o < d_out && i < d_in) W_hat[o * d_in + i] = tile[tx][r];
    }
}

// ROWS decode: W_hat[o][i] = C16[idx[(o*in_pad + i) / g]][(o*in_pad + i) % g].
__global__ void __launch_bounds__(256)
decode_rows_kernel(const uint16_t* __restrict__ C16, int g, const uint16_t* __restrict__ idx, int64_t d_out,
                   int64_t d_in, int64_t in_pad, uint16_t* __restrict__ W_hat) {
    const int64_t total = d_out * d_in;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t o = e / d_in, i = e - o * d_in;
        const int64_t flat = o * in_pad + i;
        const int64_t n = flat / g;
        W_hat[e] = __ldg(C16 + (int64_t)__ldg(idx + n) * g + (flat - n * g));
    }
}

__global__ void gather_init_kernel(const uint16_t* __restrict__ X, int g, int K, const int64_t* __restrict__ pos,
                                   float* __restrict__ C) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= K * g) return;
    const int k = e / g, t = e - k * g;
    C[e] = __half2float(__ushort_as_half(X[pos[k] * g + t]));
}

// C16 = round-to-nearest-even FP16 of C; optionally also the widened value (what the codes of
// the stored codebook are computed against).
__global__ void to_half_kernel(const float* __restrict__ C, int64_t n, uint16_t* __restrict__ C16,
                               float* __restrict__ widened) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    const __half h = __float2half_rn(C[e]);
    C16[e] = __half_as_ushort(h);
    if (widened) widened[e] = __half2float(h);
}

}  // namespace

static inline int64_t pad_to(int64_t len, int g) { return (len + g - 1) / g * g; }

cudaError_t cc_launch_reshape(cc_ctx* ctx, const uint16_t* W, int64_t d_out, int64_t d_in, int g, int layout,
                              uint16_t* X, cudaStream_t st) {
    ProfScope ps(ctx, CC_K_RESHAPE, st);
    if (layout == CC_LAYOUT_PAPER_T) {
        const int64_t out_pad = pad_to(d_out, g);
        dim3 grid((unsigned)((d_in + TD - 1) / TD), (unsigned)((out_pad + TD - 1) / TD));
        if (d_in % 8 == 0 && out_pad % 8 == 0)
            reshape_transpose_vec_kernel<<<grid, 256, 0, st>>>(W, d_out, d_in, out_pad, X);
        else
            reshape_transpose_kernel<<<grid, 256, 0, st>>>(W, d_out, d_in, out_pad, X);
    } else {
        const int64_t in_pad = pad_to(d_in, g);
        int64_t blocks = (d_out * in_pad + 255) / 256;
        if (blocks > (int64_t)ctx->sm_count * 32) blocks = (int64_t)ctx->sm_count * 32;
        reshape_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(W, d_out, d_in, in_pad, X);
    }
    return cudaGetLastError();
}

cudaError_t cc_launch_decode(cc_ctx* ctx, const uint16_t* C16, int K, int g, const uint16_t* idx, int64_t d_out,
                             int64_t d_in, int layout, uint16_t* W_hat, cudaStream_t st) {
    ProfScope ps(ctx, CC_K_DECODE, st);
    if (layout == CC_LAYOUT_PAPER_T) {
        const int64_t out_pad = pad_to(d_out, g);
        dim3 grid((unsigned)((d_in + TD - 1) / TD), (unsigned)((d_out + TD - 1) / TD));
        // the vector kernels read two codes as one 32-bit word
        const bool vec = d_in % 8 == 0 && out_pad % 8 == 0 && (reinterpret_cast<uintptr_t>(idx) & 3u) == 0;
        const int64_t n_tiles = (int64_t)grid.x * grid.y;
        // Enough tiles for persistent CTAs with loads in flight across tiles, and a codebook that
        // stays in L1: there the chain of latencies bounds a tile.  A larger codebook is bound by the
        // L2 sectors its gathers move, and more resident threads (the kernel below) serve it better.
        // With g = 4 (8-byte rows, two gathers per 16 output bytes) the plain kernel measured faster.
        if (vec && (g == 8 || g == 16) && n_tiles >= (int64_t)ctx->sm_count * 8 &&
            (int64_t)K * g * 2 <= kPipeMaxTableBytes) {
            if (g == 8) return launch_decode_pipe<8>(ctx->sm_count, C16, idx, K, d_out, d_in, out_pad, W_hat, (int)grid.x, (int)grid.y, st);
            return launch_decode_pipe<16>(ctx->sm_count, C16, idx, K, d_out, d_in, out_pad, W_hat, (int)grid.x, (int)grid.y, st);
        }
        if (vec && g == 4) decode_transpose_vec_kernel<4><<<grid, 256, 0, st>>>(C16, idx, d_out, d_in, out_pad, W_hat);
        else if (vec && g == 8) decode_transpose_vec_kernel<8><<<grid, 256, 0, st>>>(C16, idx, d_out, d_in, out_pad, W_hat);
        else if (vec && g == 16) decode_transpose_vec_kernel<16><<<grid, 256, 0, st>>>(C16, idx, d_out, d_in, out_pad, W_hat);
        else decode_transpose_kernel<<<grid, 256, 0, st>>>(C16, g, idx, d_out, d_in, out_pad, W_hat);
    } else {
        const int64_t in_pad = pad_to(d_in, g);
        int64_t blocks = (d_out * d_in + 255) / 256;
        if (blocks > (int64_t)ctx->sm_count * 32) blocks = (int64_t)ctx->sm_count * 32;
        decode_rows_kernel<<<(unsigned)blocks, 256, 0, st>>>(C16, g, idx, d_out, d_in, in_pad, W_hat);
    }
    return cudaGetLastError();
}

cudaError_t cc_launch_gather_init(cc_ctx* ctx, const uint16_t* X, int g, int K, const int64_t* pos_dev, float* C,
                                  cudaStream_t st) {
    ProfScope ps(ctx, CC_K_OTHER, st);
    gather_init_kernel<<<(K * g + 255) / 256, 256, 0, st>>>(X, g, K, pos_dev, C);
    return cudaGetLastError();
}

cudaError_t cc_launch_to_half(cc_ctx* ctx, const float* C, int64_t n, uint16_t* C16, float* C_widened,
                              cudaStream_t st) {
    ProfScope ps(ctx, CC_K_OTHER, st);
    to_half_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(C, n, C16, C_widened);
    return cudaGetLastError();
}
