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
    (void)K;
    ProfScope ps(ctx, CC_K_DECODE, st);
    if (layout == CC_LAYOUT_PAPER_T) {
        const int64_t out_pad = pad_to(d_out, g);
        dim3 grid((unsigned)((d_in + TD - 1) / TD), (unsigned)((d_out + TD - 1) / TD));
        decode_transpose_kernel<<<grid, 256, 0, st>>>(C16, g, idx, d_out, d_in, out_pad, W_hat);
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
