/*
 * CPU oracle for the ClusComp clustering path.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, float64 restatement of what the paper's clustering step
 * computes (Section 3.1 "ClusComp-: Clustering"; storage format of Section 3.2;
 * the layer listing in the appendix for the reshape / decode layout).  It exists
 * to check the CUDA library and is never part of the product path: only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may call it.  It
 * shares no source, header, table or helper with the CUDA library.
 *
 * There is no blocking, fusion or reordering here beyond what the definitions
 * state: every distance is the direct sum of squared differences in double,
 * every mean is a sequential double sum divided by an exact integer count.
 * OpenMP only splits the independent points of the E-step across threads.
 *
 * Parity pins (tests, CPU only): exhaustive exact-rational argmin / means on
 * tiny inputs, brute force over all labelings, K=1 closed form, K=N zero error,
 * separated blobs, monotone objective, scipy's vq / kmeans2, numpy's FP16 cast,
 * the values printed in the paper's bits-per-parameter table.  The outputs on
 * the five benchmark workloads themselves are "parity unpinned" by the paper
 * (it prints no clustering output); they rest on the pins above.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC (no fast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define OC_LAYOUT_PAPER_T 0 /* transpose, then group g consecutive out_features   */
#define OC_LAYOUT_ROWS 1    /* group g consecutive in_features of each row of W    */

/* ---- IEEE binary16 <-> wider types, written out bit by bit ------------------- */

static double half_to_double(uint16_t h) {
    int sign = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);                 /* zero / subnormal */
    else if (e == 31) v = m ? (double)NAN : (double)INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);            /* (1+m/1024)*2^(e-15) */
    return sign ? -v : v;
}

/* round-to-nearest-even float -> binary16 (Section 3.2: the codebook is stored FP16) */
static uint16_t float_to_half_rne(float f) {
    uint16_t sign = signbit(f) ? 0x8000u : 0u;
    double a = fabs((double)f);
    if (isnan(f)) return (uint16_t)(sign | 0x7e00u);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);   /* midpoint to 2^16 rounds up */
    if (a < ldexp(1.0, -14)) {                             /* subnormal grid, step 2^-24 */
        double q = nearbyint(ldexp(a, 24));                /* default mode: ties to even */
        return (uint16_t)(sign | (uint16_t)q);             /* q==1024 is the first normal */
    }
    int e;
    double fr = frexp(a, &e);                              /* a = fr*2^e, fr in [0.5,1)  */
    double q = nearbyint(ldexp(fr, 11));                   /* 11-bit significand         */
    if (q == 2048.0) { q = 1024.0; e += 1; }
    return (uint16_t)(sign | ((uint16_t)(e + 14) << 10) | ((uint16_t)q - 1024u));
}

void oc_float_to_half(const float* src, int64_t n, uint16_t* dst) {
    for (int64_t i = 0; i < n; ++i) dst[i] = float_to_half_rne(src[i]);
}
void oc_half_to_double(const uint16_t* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) dst[i] = half_to_double(src[i]);
}

/* ---- Sizes: padded number of codes (appendix listing) and Eq. 1 --------------- */

/* Padded length of the grouped axis: the listing pads out_features up to a
 * multiple of g ("deficiency"); ROWS pads in_features the same way. */
static int64_t padded(int64_t len, int g) { return (len + g - 1) / g * g; }

int64_t oc_num_subvectors(int64_t d_out, int64_t d_in, int g, int layout) {
    if (layout == OC_LAYOUT_PAPER_T) return d_in * (padded(d_out, g) / g);
    return d_out * (padded(d_in, g) / g);
}

/* Eq. 1: (16*k + 16*g*n) / (d_in*d_out), k = number of codes after padding. */
double oc_bits_per_param(int64_t d_out, int64_t d_in, int g, int K) {
    double k = (double)oc_num_subvectors(d_out, d_in, g, OC_LAYOUT_PAPER_T);
    return (16.0 * k + 16.0 * (double)g * (double)K) / ((double)d_in * (double)d_out);
}

/* ---- Reshape W -> W' (Section 3.1 footnote; appendix listing) ----------------- */

/* W is d_out x d_in row-major FP16 bits.  PAPER_T: W' = W^T.view(-1, g) after
 * zero-padding out_features: sub-vector n = i*(out_pad/g) + o/g, element o%g.
 * ROWS: W' = W.view(-1, g) after zero-padding in_features.                      */
void oc_reshape(const uint16_t* W, int64_t d_out, int64_t d_in, int g, int layout, uint16_t* X) {
    if (layout == OC_LAYOUT_PAPER_T) {
        int64_t out_pad = padded(d_out, g);
        for (int64_t i = 0; i < d_in; ++i)
            for (int64_t o = 0; o < out_pad; ++o)
                X[i * out_pad + o] = (o < d_out) ? W[o * d_in + i] : (uint16_t)0;
    } else {
        int64_t in_pad = padded(d_in, g);
        for (int64_t o = 0; o < d_out; ++o)
            for (int64_t i = 0; i < in_pad; ++i)
                X[o * in_pad + i] = (i < d_in) ? W[o * d_in + i] : (uint16_t)0;
    }
}

/* ---- Decode: W_hat = codebook[code] laid back out, pad stripped ---------------- */

void oc_decode(const uint16_t* C16, int K, int g, const int32_t* idx, int64_t d_out, int64_t d_in,
               int layout, uint16_t* W_hat) {
    (void)K;
    if (layout == OC_LAYOUT_PAPER_T) {
        int64_t out_pad = padded(d_out, g);
        for (int64_t i = 0; i < d_in; ++i)
            for (int64_t o = 0; o < d_out; ++o) {
                int64_t flat = i * out_pad + o;            /* position in the (in, out_pad) view */
                W_hat[o * d_in + i] = C16[(int64_t)idx[flat / g] * g + flat % g];
            }
    } else {
        int64_t in_pad = padded(d_in, g);
        for (int64_t o = 0; o < d_out; ++o)
            for (int64_t i = 0; i < d_in; ++i) {
                int64_t flat = o * in_pad + i;
                W_hat[o * d_in + i] = C16[(int64_t)idx[flat / g] * g + flat % g];
            }
    }
}

/* ---- Initialisation: K distinct positions from a seeded partial shuffle -------- */
/* The paper leaves initialisation to its library's defaults; the rule used here:
 * splitmix64 stream; for i < K: j = i + next() mod (N-i); swap a[i], a[j];
 * position i is a[i].  Written with the full array: slow, obvious.             */

static uint64_t splitmix64_next(uint64_t* s) {
    uint64_t z = (*s += 0x9E3779B97F4A7C15ULL);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

int oc_init_positions(int64_t N, int K, uint64_t seed, int64_t* pos) {
    int64_t* a = (int64_t*)malloc(sizeof(int64_t) * (size_t)N);
    if (!a) return 1;
    for (int64_t i = 0; i < N; ++i) a[i] = i;
    uint64_t s = seed;
    for (int64_t i = 0; i < K; ++i) {
        int64_t j = i + (int64_t)(splitmix64_next(&s) % (uint64_t)(N - i));
        int64_t t = a[i]; a[i] = a[j]; a[j] = t;
        pos[i] = a[i];
    }
    free(a);
    return 0;
}

int oc_init_codebook(const uint16_t* X, int64_t N, int g, int K, uint64_t seed, float* C) {
    int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)K);
    if (!pos || oc_init_positions(N, K, seed, pos)) { free(pos); return 1; }
    for (int k = 0; k < K; ++k)
        for (int t = 0; t < g; ++t) C[(int64_t)k * g + t] = (float)half_to_double(X[pos[k] * g + t]);
    free(pos);
    return 0;
}

/* ---- E-step (Section 3.1): nearest centroid by squared Euclidean distance ------ */
/* For the points sel[0..n_sel) (or all N when sel == NULL): d_ij = sum_t
 * (x_it - c_jt)^2 in double; idx = smallest j attaining the minimum; d1 = that
 * minimum, d2 = the second smallest distance (= d1 for an exact tie).          */
void oc_assign(const uint16_t* X, int64_t N, int g, const float* C, int K, const int64_t* sel,
               int64_t n_sel, int32_t* idx, double* d1, double* d2) {
    int64_t n = sel ? n_sel : N;
    double* Cd = (double*)malloc(sizeof(double) * (size_t)K * g);
    for (int64_t e = 0; e < (int64_t)K * g; ++e) Cd[e] = (double)C[e];
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n; ++r) {
        int64_t i = sel ? sel[r] : r;
        double x[64];
        for (int t = 0; t < g; ++t) x[t] = half_to_double(X[i * g + t]);
        double best = INFINITY, second = INFINITY;
        int32_t bj = -1;
        for (int j = 0; j < K; ++j) {
            const double* c = Cd + (int64_t)j * g;
            double d = 0.0;
            for (int t = 0; t < g; ++t) { double df = x[t] - c[t]; d += df * df; }
            if (d < best) { second = best; best = d; bj = j; }
            else if (d < second) second = d;
        }
        idx[r] = bj;
        if (d1) d1[r] = best;
        if (d2) d2[r] = second;
    }
    free(Cd);
}

/* Distance of point i to one given centroid, same arithmetic as above. */
double oc_point_dist(const uint16_t* X, int64_t i, int g, const float* C, int j) {
    double d = 0.0;
    for (int t = 0; t < g; ++t) {
        double df = half_to_double(X[i * g + t]) - (double)C[(int64_t)j * g + t];
        d += df * df;
    }
    return d;
}

/* ---- M-step (Section 3.1): per-cluster mean; empty cluster keeps its centroid -- */
void oc_update(const uint16_t* X, int64_t N, int g, const int32_t* idx, int K, float* C,
               int64_t* counts) {
    double* sum = (double*)calloc((size_t)K * g, sizeof(double));
    memset(counts, 0, sizeof(int64_t) * (size_t)K);
    for (int64_t i = 0; i < N; ++i) {
        int32_t j = idx[i];
        counts[j] += 1;
        for (int t = 0; t < g; ++t) sum[(int64_t)j * g + t] += half_to_double(X[i * g + t]);
    }
    for (int j = 0; j < K; ++j)
        if (counts[j] > 0)
            for (int t = 0; t < g; ++t)
                C[(int64_t)j * g + t] = (float)(sum[(int64_t)j * g + t] / (double)counts[j]);
    free(sum);
}

/* ---- Gradient of the reconstruction with respect to the codebook ----------------
 * The decoded weights are codebook[code] (appendix listing) and the paper trains only the
 * codebook with the codes fixed (Sections 3.2-3.3), so by the chain rule the gradient of any
 * loss with respect to centroid j is the sum of the gradients of the sub-vectors coded j:
 * dC[j][t] = sum_{i : idx[i] = j} dX[i][t].  Double sums, one rounding to float. */
void oc_codebook_grad(const uint16_t* dX, int64_t N, int g, const int32_t* idx, int K, float* dC) {
    double* sum = (double*)calloc((size_t)K * g, sizeof(double));
    for (int64_t i = 0; i < N; ++i) {
        int32_t j = idx[i];
        for (int t = 0; t < g; ++t) sum[(int64_t)j * g + t] += half_to_double(dX[i * g + t]);
    }
    for (int64_t e = 0; e < (int64_t)K * g; ++e) dC[e] = (float)sum[e];
    free(sum);
}

/* ---- Lloyd loop: iters x (E-step, M-step); centroid state held in float -------- */
/* objective[t] = sum_i d1_i at the t-th E-step (a plain sum, as in Section 3.1).  */
void oc_fit(const uint16_t* X, int64_t N, int g, int K, int iters, float* C, int32_t* idx,
            double* d1, int64_t* counts, double* objective) {
    for (int it = 0; it < iters; ++it) {
        oc_assign(X, N, g, C, K, NULL, 0, idx, d1, NULL);
        double J = 0.0;
        for (int64_t i = 0; i < N; ++i) J += d1[i];
        objective[it] = J;
        oc_update(X, N, g, idx, K, C, counts);
    }
}

/* ---- Forward of the compressed linear layer (appendix listing) -------------------
 * weight = codebook[code] viewed as (in_features, out_features + pad) with the padded columns
 * dropped; out = x . weight (+ bias).  x: M x d_in FP16 (row-major), y: M x d_out doubles,
 * y[m][o] = sum_i x[m][i] * weight[i][o] + bias[o], summed over i in increasing order.     */
void oc_linear_forward(const uint16_t* x, int64_t M, const uint16_t* C16, int g, const int32_t* idx,
                       int64_t d_out, int64_t d_in, const float* bias, double* y) {
    int64_t out_pad = padded(d_out, g);
    for (int64_t m = 0; m < M; ++m)
        for (int64_t o = 0; o < d_out; ++o) {
            double s = 0.0;
            for (int64_t i = 0; i < d_in; ++i) {
                int64_t flat = i * out_pad + o;            /* position in the (in, out_pad) view */
                double w = half_to_double(C16[(int64_t)idx[flat / g] * g + flat % g]);
                s += half_to_double(x[m * d_in + i]) * w;
            }
            y[m * d_out + o] = bias ? s + (double)bias[o] : s;
        }
}

/* ---- Uniform quantisation of the codebook (Section 5.3 "Inference latency": the FP16 codebook
 * may be quantised uniformly to 8 or 4 bits; the grid is the symmetric uniform one of the related-
 * work section: q = clamp(round-to-nearest(c / s), -2^(b-1), 2^(b-1) - 1)).  One scale for the whole
 * codebook.  Reading of the scale: s = max|c| / (2^(b-1) - 1), so that the grid spans the values (the
 * printed denominator 2^b - 1 would clip every value above half of the range).  The paper fixes no
 * precision; taken here: s and c / s in float (IEEE single, round-to-nearest), rounding of the
 * quotient to the nearest integer with ties to even.  deq = FP16(q * s) (float product, RNE).    */
void oc_quantize_codebook(const uint16_t* C16, int64_t n, int bits, int8_t* q, float* scale, uint16_t* deq) {
    float maxabs = 0.0f;
    for (int64_t e = 0; e < n; ++e) {
        float a = (float)fabs(half_to_double(C16[e]));
        if (a > maxabs) maxabs = a;
    }
    int L = (1 << (bits - 1)) - 1;
    float s = maxabs > 0.0f ? maxabs / (float)L : 1.0f;
    *scale = s;
    for (int64_t e = 0; e < n; ++e) {
        float c = (float)half_to_double(C16[e]);
        float t = c / s;
        double r = nearbyint((double)t);                   /* default rounding mode: ties to even */
        if (r < -(double)(L + 1)) r = -(double)(L + 1);
        if (r > (double)L) r = (double)L;
        q[e] = (int8_t)r;
        if (deq) deq[e] = float_to_half_rne((float)q[e] * s);
    }
}

/* ---- Second empty-cluster rule: split the most populated cluster ---------------------
 * The paper does not say what happens to a cluster that loses all its points; the default rule of
 * this oracle keeps its centroid.  This optional rule re-seeds it instead, the way k-means
 * libraries commonly do.  After the means: for every empty cluster e in increasing order, the donor
 * d is the cluster with the largest working count (lowest index among equals); if that count is
 * below 2, e keeps its centroid.  Otherwise c_e = c_d, then coordinate t of c_e is multiplied by
 * (1 + eps) and that of c_d by (1 - eps) for even t, the other way round for odd t (eps = 2^-10,
 * float products), and the working counts become n_e = floor(n_d / 2), n_d = n_d - n_e.
 * `counts` (true member counts) is not changed.                                               */
void oc_split_empty(float* C, int K, int g, const int64_t* counts) {
    int64_t* work = (int64_t*)malloc(sizeof(int64_t) * (size_t)K);
    memcpy(work, counts, sizeof(int64_t) * (size_t)K);
    const float up = 1.0f + 0.0009765625f, down = 1.0f - 0.0009765625f;
    for (int e = 0; e < K; ++e) {
        if (counts[e] != 0) continue;
        int d = 0;
        for (int j = 1; j < K; ++j) if (work[j] > work[d]) d = j;
        if (work[d] < 2) continue;
        for (int t = 0; t < g; ++t) {
            float c = C[(int64_t)d * g + t];
            C[(int64_t)e * g + t] = c * ((t & 1) ? down : up);
            C[(int64_t)d * g + t] = c * ((t & 1) ? up : down);
        }
        work[e] = work[d] / 2;
        work[d] -= work[e];
    }
    free(work);
}
