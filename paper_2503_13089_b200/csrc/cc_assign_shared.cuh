// Device code shared by the two E-step paths: point loads and the per-point finish (index
// recovery inside the winning chunk, direct-form distance, near-tie flag).
#pragma once

#include "cc_common.cuh"

namespace {

typedef unsigned long long ull;

constexpr float kBig = 3.0e38f;   // score of the padding centroids; above any real score

// Load one point (G halves) as floats; rows beyond N read as zeros.
template <int G>
__device__ __forceinline__ void load_point(const uint16_t* __restrict__ X, int64_t i, int64_t N, float* x,
                                           bool& nonfinite) {
    if (i >= N) {
#pragma unroll
        for (int t = 0; t < G; ++t) x[t] = 0.f;
        return;
    }
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
    } else if constexpr (G % 2 == 0) {
#pragma unroll
        for (int v = 0; v < G / 2; ++v) {
            unsigned u = __ldg(reinterpret_cast<const unsigned*>(row) + v);
            h[v * 2] = u & 0xffffu; h[v * 2 + 1] = u >> 16;
        }
    } else {
#pragma unroll
        for (int t = 0; t < G; ++t) h[t] = __ldg(row + t);
    }
#pragma unroll
    for (int t = 0; t < G; ++t) {
        if ((h[t] & 0x7c00u) == 0x7c00u) nonfinite = true;
        x[t] = __half2float(__ushort_as_half(h[t]));
    }
}

// Finish of one point after the scan.  `chunk` is the CHUNK-centroid chunk holding the smallest
// score, `second_other` the smallest chunk minimum among all other chunks.  The chunk is rescanned
// from the staged codebook (groups of four centroids: G float4 of m = -2c, then the squared norms)
// with the FMA chain s = fma(x_{g-1}, m_{g-1}, ... fma(x_0, m_0, csq)), ascending index, strict
// '<' (lowest index wins).  err_units * 2^-24 * 2 * (5||x||^2 + 4 d^2) is the gap below which the
// two smallest scores may be misordered by rounding; such points go to the exact stage.
template <int G, int CHUNK>
__device__ __forceinline__ void finish_point(const uint16_t* __restrict__ X, int64_t N, const float* __restrict__ C,
                                             int K, const float4* __restrict__ prep, int64_t i, int chunk,
                                             float second_other, double err_units, uint16_t* __restrict__ idx,
                                             float* __restrict__ dist, unsigned* __restrict__ status,
                                             unsigned* __restrict__ flagged) {
    constexpr int ROW4 = G + 1;
    float x[G];
    bool nf = false;
    load_point<G>(X, i, N, x, nf);
    float s1 = INFINITY, s2 = INFINITY;
    int j1 = chunk * CHUNK;
    const float4* cp = prep + (int64_t)chunk * (CHUNK / 4) * ROW4;
#pragma unroll 8
    for (int q = 0; q < CHUNK / 4; ++q) {
        const float4* row = cp + q * ROW4;
        const float4 cs = __ldg(row + G);
        float s[4] = {cs.x, cs.y, cs.z, cs.w};
#pragma unroll
        for (int t = 0; t < G; ++t) {
            const float4 mv = __ldg(row + t);
            s[0] = fmaf(x[t], mv.x, s[0]);
            s[1] = fmaf(x[t], mv.y, s[1]);
            s[2] = fmaf(x[t], mv.z, s[2]);
            s[3] = fmaf(x[t], mv.w, s[3]);
        }
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            if (s[h] < s1) { s2 = s1; s1 = s[h]; j1 = chunk * CHUNK + 4 * q + h; }
            else if (s[h] < s2) s2 = s[h];
        }
    }
    if (j1 >= K) j1 = K - 1;   // only reachable with non-finite input
    s2 = fminf(s2, second_other);
    // squared distance to the winner, direct form in FP64 (no contraction)
    double A = 0.0, D = 0.0;
#pragma unroll
    for (int t = 0; t < G; ++t) {
        const double xdbl = (double)x[t];
        const double df = __dsub_rn(xdbl, (double)__ldg(C + (int64_t)j1 * G + t));
        D = __dadd_rn(D, __dmul_rn(df, df));
        A = __dadd_rn(A, __dmul_rn(xdbl, xdbl));
    }
    idx[i] = (uint16_t)j1;
    dist[i] = (float)D;
    const double gap = (double)s2 - (double)s1;
    if (!(gap > 2.0 * err_units * 5.9604644775390625e-8 * (5.0 * A + 4.0 * D))) {
        const ull slot = atomicAdd(reinterpret_cast<ull*>(status + 2), 1ull);
        flagged[slot] = (unsigned)i;
    }
}

}  // namespace
