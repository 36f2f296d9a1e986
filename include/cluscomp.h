/*
 * cluscomp.h -- C ABI of the B200 (sm_100a) clustering library.
 *
 * The library computes the clustering step of ClusComp (Section 3.1,
 * "ClusComp-: Clustering"): the sub-vectors of a weight matrix are clustered by
 * Lloyd's k-means into a codebook C (n centroids of dimension g) and codes q
 * (one index per sub-vector); Section 3.2 fixes the storage (FP16 codebook,
 * unsigned 16-bit codes) and the appendix listing fixes the reshape / decode
 * layout.
 *
 * Conventions for every call below
 *  - Pointers are DEVICE pointers owned by the caller unless the name ends in
 *    `_host`.  FP16 data is passed as uint16_t bit patterns (IEEE binary16).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls enqueue work on it and return without waiting; outputs are valid
 *    after the stream has been synchronised.
 *  - Arguments are validated on the host before anything is launched.  A call
 *    that returns a status other than CC_OK has enqueued nothing and its
 *    outputs are undefined.  The library never aborts and its kernels never
 *    trap; problems found on the device (non-finite input) are recorded in a
 *    status word that cc_poll_status() reads back.
 *  - N = number of sub-vectors, g = sub-vector dimension (1..16),
 *    K = number of centroids (1..65536, the paper keeps n <= 2^16 so that a
 *    code fits 16 bits; codes are 0-based).  N < 2^31.
 *  - The same inputs give bit-identical outputs on every call.
 *  - Scratch memory is one caller-owned workspace (cc_workspace_bytes /
 *    cc_set_workspace); the library itself allocates no device memory except
 *    in cc_compress_host (a buffer kept in the context).
 */
#ifndef CLUSCOMP_H_
#define CLUSCOMP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CC_OK = 0,
    CC_ERR_NULL = 1,           /* a required pointer is NULL                              */
    CC_ERR_SHAPE = 2,          /* a size is <= 0 or too large                             */
    CC_ERR_UNSUPPORTED_G = 3,  /* g outside 1..16                                         */
    CC_ERR_K_RANGE = 4,        /* K outside 1..65536                                      */
    CC_ERR_N_LT_K = 5,         /* initialisation needs K distinct sub-vectors             */
    CC_ERR_ALIGN = 6,          /* X / C / W pointers must be 16-byte aligned              */
    CC_ERR_WORKSPACE = 7,      /* no workspace set, or smaller than cc_workspace_bytes    */
    CC_ERR_NONFINITE = 8,      /* Inf / NaN met in the input (reported by cc_poll_status) */
    CC_ERR_DEVICE_TIMEOUT = 9, /* a bounded device-side wait ran out                      */
    CC_ERR_CUDA = 10,          /* a CUDA runtime call failed                              */
    CC_ERR_LAYOUT = 11,        /* unknown layout / path constant                          */
    CC_ERR_STATIC_CAPACITY = 12 /* cc_update_static: K * g above CC_UPDATE_STATIC_MAX_KG  */
} cc_status;

/* How sub-vectors are cut out of W (d_out x d_in, row-major, as a linear layer stores it). */
#define CC_LAYOUT_PAPER_T 0 /* W' = W^T.view(-1, g): g consecutive out_features at a fixed
                               in_feature; out_features zero-padded to a multiple of g
                               (Section 3.1 footnote; "deficiency" in the appendix listing). */
#define CC_LAYOUT_ROWS 1    /* W' = W.view(-1, g): g consecutive in_features of one row;
                               in_features zero-padded to a multiple of g.                   */

/* Which E-step kernel family cc_assign uses. */
#define CC_PATH_AUTO 0   /* the faster path: measured, the tensor-core one for every g */
#define CC_PATH_FFMA 1   /* FP32 FMA pipes, register-tiled                             */
#define CC_PATH_TENSOR 2 /* tcgen05 tensor cores with TMEM accumulators                */

typedef struct cc_ctx cc_ctx; /* opaque; one per device and per concurrent user */

/* Context.  cc_create binds to `device` (cudaSetDevice is called inside every entry point).
 * cc_destroy frees host state and the buffer of cc_compress_host; the workspace stays the caller's. */
cc_status cc_create(cc_ctx** out, int device);
cc_status cc_destroy(cc_ctx* ctx);
const char* cc_status_string(cc_status s);

/* Scratch memory needed by any call on a problem of this size, in bytes (0 on bad arguments).
 * The workspace must stay valid and unshared while calls using it are in flight. */
size_t cc_workspace_bytes(int64_t N, int g, int K);
cc_status cc_set_workspace(cc_ctx* ctx, void* workspace, size_t bytes);

/* CC_PATH_* override for cc_assign / cc_fit / cc_finalize (default CC_PATH_AUTO).
 * Every path returns the same idx and counts. */
cc_status cc_set_path(cc_ctx* ctx, int path);

/* Number of kernels this context has launched so far (host counter). */
int64_t cc_launch_count(const cc_ctx* ctx);

/* Measurement aids (no counterpart in the paper).  With timing enabled every kernel launch is
 * bracketed by a CUDA event pair on its own stream (at most 8192 launches between two reads).
 * cc_profile_read waits for those events, adds up the device time and the number of launches
 * of one kernel class, for all classes at once: total_ms_host / launches_host are host arrays
 * of CC_KERNEL_CLASSES entries (either may be NULL), and the record is cleared. */
#define CC_KERNEL_ASSIGN_MAIN 0   /* the N x K distance scan of the E-step              */
#define CC_KERNEL_ASSIGN_PREP 1   /* staging of the codebook for the scan               */
#define CC_KERNEL_RESOLVE 2       /* exact FP64 stage for near-ties                     */
#define CC_KERNEL_OBJECTIVE 3     /* deterministic sum of the distances                 */
#define CC_KERNEL_UPDATE_ACCUM 4  /* M-step over all points: integer sums and counts    */
#define CC_KERNEL_UPDATE_FINISH 5 /* M-step: division, empty-cluster rule               */
#define CC_KERNEL_RESHAPE 6
#define CC_KERNEL_DECODE 7
#define CC_KERNEL_OTHER 8
#define CC_KERNEL_ASSIGN_FINISH 9 /* tensor path: index, distance, near-tie flag per point */
#define CC_KERNEL_UPDATE_DELTA 10  /* M-step inside cc_fit: only the points whose code changed */
#define CC_KERNEL_LINEAR 11        /* forward of the compressed linear layer: the GEMM with the gathered weight */
#define CC_KERNEL_LINEAR_REDUCE 12 /* ... and the sum of its split-K partial results                          */
#define CC_KERNEL_CLASSES 13
cc_status cc_profile_enable(cc_ctx* ctx, int on);
cc_status cc_profile_read(cc_ctx* ctx, double* total_ms_host, int64_t* launches_host);

/* Runs a register-only FP32 FMA loop on every SM (the ceiling the FP32 E-step is measured
 * against) and returns the achieved TFLOP/s (2 flops per FMA) for the scalar and the packed
 * two-wide instruction form.  Synchronises `stream`.  Outputs are host doubles. */
cc_status cc_measure_fp32_peak(cc_ctx* ctx, double* tflops_scalar_host, double* tflops_packed_host,
                               void* stream);

/* Runs register-only loops of the FP32 minimum (the instruction that bounds the tensor-core E-step:
 * every score is compared once) with one 512-thread block per SM and writes to the HOST array
 * lane_instr_per_clk_per_sm[3] the measured lane-instructions per SM clock per SM for
 *   [0] two-input min.f32, [1] three-input min.f32 (two new values each), [2] both alternating
 * (median over the blocks of block lane-instructions / the block's own clock64 cycle count).
 * sm_mhz (host, may be NULL): SM clock during the loops = cycles of the longest block / CUDA-event
 * time of its launch.  distinct_sms (host, may be NULL): on how many different SMs the blocks ran
 * (equal to the SM count when every block had an SM to itself).  Synchronises `stream`; allocates
 * and frees a few KB of device memory. */
cc_status cc_measure_min_rate(cc_ctx* ctx, double* lane_instr_per_clk_per_sm_host, double* sm_mhz_host,
                              int32_t* distinct_sms_host, void* stream);

/* Host helpers.  Number of sub-vectors after padding: the appendix listing's
 * num_codes = in_features * (out_features + deficiency) / g (PAPER_T), or the same rule along
 * in_features (ROWS); -1 on bad arguments.  Average bits per parameter, Eq. 1 of Section 3.2:
 * (16 * codes + 16 * g * K) / (d_in * d_out), codes counted after padding. */
int64_t cc_num_subvectors(int64_t d_out, int64_t d_in, int g, int layout);
double cc_bits_per_param(int64_t d_out, int64_t d_in, int g, int K);

/* Section 3.1 (footnote) / appendix listing: cut W into sub-vectors.
 * W: d_out x d_in FP16 row-major.  X (out): N x g FP16 row-major, N = cc_num_subvectors(...);
 * padded elements are +0.  W and X must not overlap. */
cc_status cc_reshape_subvectors(cc_ctx* ctx, const uint16_t* W, int64_t d_out, int64_t d_in, int g,
                                int layout, uint16_t* X, void* stream);

/* Initial codebook.  The paper leaves this to its library's defaults; the rule here: K distinct
 * positions from a partial Fisher-Yates shuffle of 0..N-1 driven by splitmix64(seed)
 * (for i < K: j = i + next() mod (N - i); swap a[i], a[j]; position i is a[i]);
 * C[k] = X[position k] widened to FP32.  cc_init_positions writes the K positions to host memory
 * (no device work).  C (out): K x g FP32.  Needs 1 <= K <= N. */
cc_status cc_init_positions(int64_t N, int K, uint64_t seed, int64_t* positions_host);
cc_status cc_init_codebook(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, uint64_t seed,
                           float* C, void* stream);

/* Caller-chosen initial codebook (for reproducing a run or starting from another method's centroids;
 * the paper only uses its library's default start): copies K x g FP32 values from C0, which may be
 * a host or a device pointer, to the device array C on `stream`.  A pageable host source is staged
 * before the call returns; a pinned one must stay valid until the stream has passed the copy. */
cc_status cc_set_codebook(cc_ctx* ctx, const float* C0_host_or_device, int K, int g, float* C, void* stream);

/* E-step of Section 3.1: idx[i] = the centroid minimising ||x_i - c_j||^2 (lowest j on exact
 * ties), dist[i] = that squared distance (FP32), *objective = sum_i dist[i] (the Section 3.1
 * objective for this assignment, a plain sum).  X: N x g FP16; C: K x g FP32.
 * idx (out): N x uint16.  dist (out, may be NULL): N x FP32.  objective (out, device, may be
 * NULL): one double.  n_resolved (out, device, may be NULL): one int64 = how many points had
 * their two best FP32 scores closer than the rounding bound and were decided in FP64.
 * N = 0 is allowed (objective 0). */
cc_status cc_assign(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K,
                    uint16_t* idx, float* dist, double* objective, int64_t* n_resolved, void* stream);

/* Verification aid (no counterpart in the paper): which points the last cc_assign on this
 * context, with the same (N, g, K), sent to the exact FP64 stage.  Copies the first `count`
 * entries of that list (point numbers, in no particular order; count <= the n_resolved the call
 * reported) to `points`, a device or host array of uint32.  Valid until the next E-step. */
cc_status cc_last_flagged(cc_ctx* ctx, int64_t N, int g, int K, uint32_t* points, int64_t count, void* stream);

/* Verification aid for the tensor-core E-step (no counterpart in the paper): writes the raw
 * comparison scores s_ij = ||c_j||^2 - 2 x_i.c_j exactly as that path computes them (FP16 operand
 * pieces, FP32 accumulation in tensor memory), so that a test can check the rounding bound the
 * near-tie flag relies on.  scores (out): N rows of cc_tensor_scores_ld(K) floats (K rounded up
 * to the centroid tile; columns >= K hold the padding score).  1 <= N <= 65536. */
int64_t cc_tensor_scores_ld(int K);
cc_status cc_tensor_scores(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K,
                           float* scores, void* stream);

/* Verification aid for the tensor-core E-step (no counterpart in the paper): runs its second
 * kernel alone on scan results supplied by the caller.  scan: N records of 8 bytes,
 * {float: smallest score among the centroids outside the winning chunk, +inf if unknown;
 *  int32: id of the 64-centroid chunk that holds the winner}.  For every point the chunk is
 * searched in FP32, idx / dist (out, both required) get the chunk's best centroid and its FP64
 * squared distance; the exact stage for near-ties is NOT run.  A chunk id outside
 * 0 .. ceil(K / 64) - 1 (what a scan that gave up on a bounded wait may leave behind) is moved to
 * the nearest valid chunk, so no such record can make the kernel read out of bounds.  N >= 1. */
cc_status cc_tensor_finish_only(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K,
                                const void* scan, uint16_t* idx, float* dist, void* stream);

/* Self-test of the bounded waits of the tensor-core E-step (no counterpart in the paper).  Every
 * wait of those kernels on a shared-memory barrier gives up after a clock limit, raises a flag that
 * makes the CTA's other waits return, and the kernel then reports CC_ERR_DEVICE_TIMEOUT through
 * cc_poll_status instead of hanging.  This call runs one warp through that wait code with the
 * given limit (1e3 .. 4e9 clock cycles) and copies to the HOST arrays:
 *   results[0] = 1: a wait on a barrier whose phase completes succeeds;
 *   results[1] = 0: a wait on a barrier nobody arrives on gives up;
 *   results[2] = 1: the abort flag is up afterwards;
 *   results[3] = 0: a further wait returns unsuccessfully;
 *   cycles[0], cycles[1]: how long the second and third wait took (the second a little more than
 *   the limit, the third far less).
 * Synchronous; allocates and frees 64 bytes of device memory. */
cc_status cc_selftest_bounded_wait(cc_ctx* ctx, int64_t limit_cycles, int32_t* results, int64_t* cycles);

/* M-step of Section 3.1: counts[j] = |{i : idx[i] = j}| (exact), C[j] = mean of those x_i
 * (exact, order-independent integer sum; converted to double, divided by the count in double and
 * rounded to FP32, as a sequential float64 sum would be); a cluster with no member keeps its centroid
 * bit for bit (the paper does not say; this library's rule).  C: in = previous, out = new.
 * counts (out): K x int32.  idx values must be < K. */
cc_status cc_update(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const uint16_t* idx, int K,
                    float* C, int32_t* counts, void* stream);

/* M-step without any device allocation (the paper has no counterpart: this is a deployment
 * variant of cc_update, not a step of the method).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a process
 * whose device memory is owned by a framework's pool and may not be grown behind its back, a
 * serving container whose device memory is fully committed at start-up so that a later
 * allocation would simply fail, or a latency-critical loop that must never reach the allocator
 * because cudaMalloc and cudaFree may wait for the whole device.  Such callers have no spare
 * buffer to hand over as a workspace either, so cc_update (which needs one) is closed to them.
 *
 * What it does: exactly what cc_update does, with the same results bit for bit, but the integer
 * sum accumulators live in a fixed array inside the library image (2 * CC_UPDATE_STATIC_MAX_KG
 * 64-bit words = 4 MiB).  Every GPU on which the library's device code is loaded holds that array
 * until the process exits.  The function takes no context and calls no cudaMalloc / cudaFree nor
 * any other allocating routine; the caller still provides
 * X, idx, C and counts exactly as for cc_update, plus the device ordinal (< 64) that owns them.
 *
 * Limits and rules
 *  - K * g must not exceed CC_UPDATE_STATIC_MAX_KG (262144: K = 65536 at g = 4, K = 16384 at
 *    g = 16); larger problems return CC_ERR_STATIC_CAPACITY and enqueue nothing.
 *  - The first call on a device looks up the array's device address (once per device, with
 *    that device made current).  Where the CUDA runtime loads device code lazily, that look-up is
 *    also what loads this library's module and reserves the array on the device, so the memory is
 *    taken at that moment rather than when the library is loaded: make the first call at start-up,
 *    before any stream capture begins and before device memory becomes scarce.  The cached address
 *    does not survive cudaDeviceReset; do not call the function again in a process that reset the
 *    device.
 *  - All calls on one device share the one array, and it keeps the previous call's contents:
 *    each call clears the part it uses on `stream` before accumulating.  Two calls whose work
 *    overlaps on the GPU (different streams, no dependency) race on it and give wrong sums;
 *    order them on one stream or with events.  The function is not thread-safe for first calls
 *    issued concurrently from several host threads on the same device. */
#define CC_UPDATE_STATIC_MAX_KG 262144
cc_status cc_update_static(int device, const uint16_t* X, int64_t N, int g, const uint16_t* idx, int K,
                           float* C, int32_t* counts, void* stream);

/* Gradient with respect to the codebook (Sections 3.2-3.3: block-wise error minimisation, recovery
 * training and finetuning all train the codebook with the codes kept fixed; the layer's weight is
 * codebook[code], appendix listing).  By the chain rule dC[j] = sum over the sub-vectors coded j of
 * dX[i], where dX is the gradient with respect to the decoded weight cut into sub-vectors exactly
 * as cc_reshape_subvectors cuts W (padded coordinates are zero there and contribute nothing).
 * dX: N x g FP16.  dC (out): K x g FP32, the exact integer sum rounded once; clusters without a
 * member get 0.  Deterministic: the result does not depend on the order of the points. */
cc_status cc_codebook_grad(cc_ctx* ctx, const uint16_t* dX, int64_t N, int g, const uint16_t* idx, int K,
                           float* dC, void* stream);

/* Lloyd loop of Section 3.1: iters x (E-step, M-step), no early stop (the paper runs a fixed
 * 20).  C: in = initial, out = after the last M-step.  idx / dist / counts (out): those of the
 * last iteration.  objective_trace (out, device, may be NULL): iters doubles, entry t = the
 * objective at the t-th E-step.  N >= 1, iters >= 0. */
cc_status cc_fit(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, int iters, float* C,
                 uint16_t* idx, float* dist, int32_t* counts, double* objective_trace, void* stream);

/* What the M-step does with a cluster that has no member (the paper does not say; it runs its
 * k-means library with default settings).  CC_EMPTY_KEEP (default): the centroid is kept bit for bit.
 * CC_EMPTY_SPLIT_LARGEST: after the means, every empty cluster e, in increasing order, is re-seeded from
 * the most populated cluster d (largest working count, lowest index among equals; nothing happens once
 * that count is below 2): c_e = c_d, then coordinate t of c_e is multiplied by 1 + 2^-10 and that of c_d
 * by 1 - 2^-10 for even t and the other way round for odd t (FP32 products), and the working counts become
 * n_e = floor(n_d / 2), n_d = n_d - n_e.  `counts` always reports the true member counts.  Applies to
 * cc_update, cc_fit, cc_fit_sampled and cc_compress_host on this context (not to cc_update_static). */
#define CC_EMPTY_KEEP 0
#define CC_EMPTY_SPLIT_LARGEST 1
cc_status cc_set_empty_rule(cc_ctx* ctx, int rule);

/* Lloyd loop on a subsample of the points, then one E-step over all of them (k-means libraries, the
 * paper's included, by default train on at most a fixed number of points per centroid; the paper
 * states no such number, so it is an argument here).  n = cc_train_points(N, K, max_points_per_centroid)
 * = min(N, max_points_per_centroid * K) distinct positions are drawn by the seeded partial shuffle of
 * cc_init_positions (the first n entries for `seed`), those rows are copied in that order to X_train
 * (device scratch of n x g FP16, 16-byte aligned; may be NULL when n == N), cc_fit runs on them, and a
 * final cc_assign over all N points against the fitted codebook fills idx / dist (N entries each; dist
 * may be NULL).  counts and objective_trace are those of the training set.  C: in = initial codebook. */
int64_t cc_train_points(int64_t N, int K, int max_points_per_centroid);
/* Host only: the first n entries of that seeded shuffle of 0..N-1 (0 <= n <= N < 2^31) as 32-bit
 * positions -- the rows cc_fit_sampled trains on; for n <= 65536 the same positions as
 * cc_init_positions. */
cc_status cc_sample_positions(int64_t N, int64_t n, uint64_t seed, uint32_t* positions_host);
cc_status cc_fit_sampled(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, int iters, int max_points_per_centroid,
                         uint64_t seed, uint16_t* X_train, float* C, uint16_t* idx, float* dist, int32_t* counts,
                         double* objective_trace, void* stream);

/* Uniform quantisation of the stored codebook (Section 5.3 "Inference latency": for inference the FP16
 * codebook may be quantised uniformly to 8 or 4 bits) on the symmetric uniform grid of the related-work
 * section: q = clamp(round-to-nearest(c / s), -2^(b-1), 2^(b-1) - 1), one scale s for the whole codebook.
 * Reading of the scale: s = max|c| / (2^(b-1) - 1), so that the grid spans the values (the printed
 * denominator 2^b - 1 would clip everything above half of the range); s = 1 for an all-zero codebook.
 * s and c / s are IEEE single precision, the quotient is rounded to the nearest integer, ties to even.
 * bits: 8 or 4.  q (out): K * g signed bytes (8 bits), or ceil(K * g / 2) bytes holding element 2k in
 * the low and element 2k + 1 in the high nibble, two's complement (4 bits).  scale (out, device): one
 * float.  C16_dequantized (out, may be NULL): K x g FP16 = round-to-nearest-even of q * s, usable with
 * cc_decode and cc_linear_forward.  Needs a workspace (any size cc_set_workspace accepts). */
cc_status cc_quantize_codebook(cc_ctx* ctx, const uint16_t* C16, int K, int g, int bits, uint8_t* q, float* scale,
                               uint16_t* C16_dequantized, void* stream);

/* The clustering of different weight matrices is independent (remark at the end of Section 3.1), so a
 * model is spread over GPUs matrix by matrix with nothing exchanged.  cc_schedule_matrices (host only):
 * longest-processing-time-first split of n matrices with costs sizes_host[i] (e.g. their numbers of
 * sub-vectors) over `world` ranks -- matrices by decreasing cost, lower index first among equals, each to
 * the rank with the smallest load so far, lowest rank among equals; writes the indices that fall to
 * `rank`, in increasing order, to mine_host (room for n) and their number to *n_mine_host.
 * cc_compress_many runs cc_compress_host on each of n matrices in turn (arrays of n host pointers and
 * sizes; objective_trace_hosts and W_hat_hosts, or single entries of them, may be NULL) and stops at
 * the first status other than CC_OK. */
cc_status cc_schedule_matrices(int n, const int64_t* sizes_host, int world, int rank, int32_t* mine_host,
                               int32_t* n_mine_host);
cc_status cc_compress_many(cc_ctx* ctx, int n, const uint16_t* const* W_hosts, const int64_t* d_outs, const int64_t* d_ins,
                           int g, int K, int iters, const uint64_t* seeds, int layout, uint16_t* const* C16_hosts,
                           uint16_t* const* idx_hosts, double* const* objective_trace_hosts, uint16_t* const* W_hat_hosts,
                           void* stream);

/* Section 3.1 (codes = nearest centroid of the final codebook) and Section 3.2 (FP16 storage):
 * C16 = round-to-nearest-even FP16 of C; idx / dist / objective = E-step against C16, so the
 * stored pair (C16, idx) is consistent and ||W - decode||^2 equals *objective (no padding). */
cc_status cc_finalize(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K,
                      uint16_t* C16, uint16_t* idx, float* dist, double* objective, void* stream);

/* Reconstruction, Section 3.1 / appendix listing (codebook[code].view(in_features, -1) with
 * the padded columns dropped): W_hat (out): d_out x d_in FP16 row-major, the layout of W.
 * idx: cc_num_subvectors(...) codes, each < K. */
cc_status cc_decode(cc_ctx* ctx, const uint16_t* C16, int K, int g, const uint16_t* idx,
                    int64_t d_out, int64_t d_in, int layout, uint16_t* W_hat, void* stream);

/* Forward of the compressed linear layer, appendix listing (ClusCompLinear.forward):
 *   weight = codebook[code].view(in_features, -1) with the padded columns dropped;  y = x . weight (+ bias).
 * The decoded weight is never written to memory: codebook rows are gathered straight into the
 * shared-memory operand of a tensor-core GEMM (FP16 inputs, FP32 accumulation).
 * x: M x d_in FP16 row-major (M tokens).  C16: K x g FP16.  idx: cc_num_subvectors(d_out, d_in, g,
 * CC_LAYOUT_PAPER_T) codes, each < K.  bias (may be NULL): d_out FP32.  y (out): M x d_out FP32
 * row-major.  The listing keeps every tensor in a 16-bit type; here the accumulator is handed out
 * unrounded.  Scratch: cc_linear_workspace_bytes(M, d_out, d_in) bytes of the context's workspace
 * (cc_set_workspace; used when the in_features are split across thread blocks, which happens for
 * small M; the partial sums are added in a fixed order, so the result is the same on every call).
 * 1 <= M < 2^31 / d_out; x, C16, y 16-byte aligned. */
size_t cc_linear_workspace_bytes(cc_ctx* ctx, int64_t M, int64_t d_out, int64_t d_in);
cc_status cc_linear_forward(cc_ctx* ctx, const uint16_t* x, int64_t M, const uint16_t* C16, int K, int g,
                            const uint16_t* idx, int64_t d_out, int64_t d_in, const float* bias, float* y,
                            void* stream);

/* The same forward with the codebook quantised to 4 bits (Section 5.3, "Inference latency": for
 * inference the codebook may be quantised uniformly, and it is the 4-bit codebook that speeds the layer
 * up).  q and scale are what cc_quantize_codebook(bits = 4) wrote: ceil(K * g / 2) bytes, element 2k in
 * the low nibble, and one device float.  The weight is the dequantised codebook, value = round-to-nearest-
 * even FP16 of nibble * scale -- exactly the C16_dequantized of cc_quantize_codebook, so the result is
 * that of cc_linear_forward on that codebook (bit for bit for 5 <= M <= 64, where both take the same
 * tensor-core route; otherwise up to the order of the FP32 additions).  The packed codebook (at most
 * 128 KB: K * g <= 262144) is held in every thread block's shared memory, which turns the gathers from
 * requests to L2 into shared-memory reads.  For a handful of tokens (M <= 4; M <= 2 when g > 8) a
 * kernel without the tensor core runs: table look-ups and FP32 multiply-adds, partial sums added in a
 * fixed order (the same bits on every call).  g even (2..16; other g: CC_ERR_UNSUPPORTED_G); a larger
 * codebook: CC_ERR_SHAPE; q 16-byte aligned; workspace as for cc_linear_forward.  Calls on one context
 * must not overlap on the device (they share the workspace and its counters). */
cc_status cc_linear_forward_q4(cc_ctx* ctx, const uint16_t* x, int64_t M, const uint8_t* q, const float* scale, int K,
                               int g, const uint16_t* idx, int64_t d_out, int64_t d_in, const float* bias, float* y,
                               void* stream);

/* Waits for `stream`, reads the device status word and clears it.  Returns CC_OK,
 * CC_ERR_NONFINITE, CC_ERR_DEVICE_TIMEOUT or CC_ERR_CUDA. */
cc_status cc_poll_status(cc_ctx* ctx, void* stream);

/* Whole path on HOST buffers (Sections 3.1-3.2 end to end): copies W to the device, reshapes,
 * initialises, runs `iters` Lloyd iterations, finalises, and copies the FP16 codebook, the
 * codes and the final objective back; optionally also decodes into W_hat_host (may be NULL).
 * Uses a device buffer of its own that the context keeps and grows on demand (the first call of a
 * size allocates, later calls do not; cc_destroy frees it) and synchronises before returning.
 * All pointers are host pointers (pinned memory makes the copies asynchronous).
 * objective_trace_host (may be NULL): iters + 1 doubles, the last being the final objective. */
cc_status cc_compress_host(cc_ctx* ctx, const uint16_t* W_host, int64_t d_out, int64_t d_in, int g,
                           int K, int iters, uint64_t seed, int layout, uint16_t* C16_host,
                           uint16_t* idx_host, double* objective_trace_host, uint16_t* W_hat_host,
                           void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CLUSCOMP_H_ */
