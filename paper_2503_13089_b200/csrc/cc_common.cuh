// Shared host-side declarations of the library's translation units.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cluscomp.h"

// Bits of the device status word (workspace, word 0).
#define CC_DEV_NONFINITE 1u
#define CC_DEV_TIMEOUT 2u

// Kernel classes for the optional per-kernel event timing (cc_profile_*).
enum { CC_K_ASSIGN_MAIN = 0, CC_K_ASSIGN_PREP = 1, CC_K_RESOLVE = 2, CC_K_OBJECTIVE = 3, CC_K_UPDATE_ACCUM = 4,
       CC_K_UPDATE_FINISH = 5, CC_K_RESHAPE = 6, CC_K_DECODE = 7, CC_K_OTHER = 8, CC_K_ASSIGN_FINISH = 9, CC_K_UPDATE_DELTA = 10,
       CC_K_LINEAR = 11, CC_K_LINEAR_REDUCE = 12, CC_K_COUNT = 13 };
constexpr int CC_PROF_CAP = 8192;

struct cc_prof_slot { cudaEvent_t a, b; int kind; };

struct cc_ctx {
    int device;
    int sm_count;
    int path;             // CC_PATH_*
    void* ws;             // caller-owned workspace
    size_t ws_bytes;
    int64_t launches;     // kernels launched so far
    int64_t* pos_host;    // staging for cc_init_codebook (K positions)
    int pos_cap;
    int prof_on;          // record an event pair around every kernel launch
    int prof_used, prof_made;
    cc_prof_slot* prof;   // CC_PROF_CAP slots, events created on first use
    void* e2e_buf;        // device memory of cc_compress_host, grown on demand, freed by cc_destroy
    size_t e2e_bytes;
    int empty_rule;       // CC_EMPTY_*
};

// Brackets one kernel launch with events on its stream when timing is enabled, and counts it.
struct ProfScope {
    cc_ctx* c; cudaStream_t st; cc_prof_slot* slot;
    ProfScope(cc_ctx* ctx, int kind, cudaStream_t s) : c(ctx), st(s), slot(nullptr) {
        c->launches++;
        if (!c->prof_on || !c->prof || c->prof_used >= CC_PROF_CAP) return;
        cc_prof_slot* sl = c->prof + c->prof_used;
        if (c->prof_used >= c->prof_made) {
            if (cudaEventCreate(&sl->a) != cudaSuccess || cudaEventCreate(&sl->b) != cudaSuccess) return;
            c->prof_made = c->prof_used + 1;
        }
        sl->kind = kind;
        cudaEventRecord(sl->a, st);
        slot = sl;
        c->prof_used++;
    }
    ~ProfScope() { if (slot) cudaEventRecord(slot->b, st); }
};

// Status block at the start of every workspace: cleared by cc_set_workspace.
constexpr size_t CC_STATUS_BYTES = 4096;
constexpr int CC_ARRIVAL_WORD = 64, CC_ARRIVAL_COUNTERS = 960;

// Carving of the workspace for a problem (N, g, K).  All offsets 256-byte aligned.
struct WsLayout {
    size_t status;     // CC_STATUS_BYTES: 1024 x u32: [0] status bits, [2..3] flagged counter (u64), [8] last-block counter of the objective
                       // sum, [32..35] tensor-path parameters, [36] codebook quantiser's maximum, [64..1023] arrival
                       // counters of the layer forward's split reduction (zero between calls)
    size_t cprep;      // staged codebook for the FFMA E-step
    size_t flagged;    // u32 list of points sent to the exact stage
    size_t partials;   // doubles: per-block objective partial sums
    size_t sum_lo;     // int64 R x K x g: sums of |x| < 8 in units of 2^-24 (R = cc_sum_copies)
    size_t sum_hi;     // int64 R x K x g: sums of |x| >= 8 in units of 2^-7
    size_t count_copies;  // int32 R x K: per-copy member counts of the M-step (R > 1)
    size_t tmp_c;      // float K x g: widened FP16 codebook (finalize)
    size_t positions;  // int64 K: initial positions
    size_t dist_tmp;   // float N: distances when the caller passes dist == NULL
    size_t tensor;     // staging of the tensor-core E-step (split codebook operand)
    size_t tstate;     // float2 N: (second-best chunk minimum, best chunk id) from the tensor-core scan
    size_t idx_prev;   // u16 N: codes of the previous M-step inside cc_fit
    size_t total;
};

constexpr int CC_KPAD = 1024;          // staged codebook is padded to a multiple of this
constexpr int CC_OBJ_BLOCKS = 1024;    // partial sums of the objective reduction

WsLayout cc_ws_layout(int64_t N, int g, int K);

// Copies of the M-step's sums (small codebooks only: at most CC_SUM_COPY_ELEMS words per array).
#ifndef CC_SUM_COPIES_MAX
#define CC_SUM_COPIES_MAX 16
#endif
constexpr int CC_SUM_COPY_ELEMS = 262144;
static inline int cc_sum_copies(int K, int g) {
    const int r = CC_SUM_COPY_ELEMS / (K * g);
    return r < 1 ? 1 : (r > CC_SUM_COPIES_MAX ? CC_SUM_COPIES_MAX : r);
}

static inline size_t cc_align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Launchers (each returns cudaGetLastError() of its launches and bumps ctx->launches).
cudaError_t cc_launch_reshape(cc_ctx*, const uint16_t* W, int64_t d_out, int64_t d_in, int g, int layout,
                              uint16_t* X, cudaStream_t);
cudaError_t cc_launch_decode(cc_ctx*, const uint16_t* C16, int K, int g, const uint16_t* idx, int64_t d_out,
                             int64_t d_in, int layout, uint16_t* W_hat, cudaStream_t);
cudaError_t cc_launch_gather_init(cc_ctx*, const uint16_t* X, int g, int K, const int64_t* pos_dev, float* C,
                                  cudaStream_t);
cudaError_t cc_launch_to_half(cc_ctx*, const float* C, int64_t n, uint16_t* C16, float* C_widened, cudaStream_t);

cudaError_t cc_launch_assign_ffma(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const float* C,
                                  int K, uint16_t* idx, float* dist, double* objective, int64_t* n_resolved,
                                  cudaStream_t);
cudaError_t cc_launch_prep_ffma(cc_ctx*, const WsLayout&, int g, const float* C, int K, cudaStream_t);
bool cc_tensor_path_supported(int g, int K);
cudaError_t cc_launch_assign_tensor(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const float* C,
                                    int K, uint16_t* idx, float* dist, double* objective, int64_t* n_resolved,
                                    cudaStream_t);
// Verification aid: every comparison score of the tensor-core scan, N x cc_tensor_score_ld(K) floats.
int cc_tensor_score_ld(int K);
cudaError_t cc_launch_wait_selftest(long long limit_cycles, int* out_dev, long long* cycles_dev, cudaStream_t);
cudaError_t cc_launch_tensor_scores(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const float* C,
                                    int K, float* scores, cudaStream_t);
cudaError_t cc_launch_tensor_finish_only(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const float* C,
                                         int K, const void* scan, uint16_t* idx, float* dist, cudaStream_t);
// Second stage shared by both E-step paths: exact FP64 decision for the flagged points, then
// the deterministic objective sum.
cudaError_t cc_launch_assign_tail(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const float* C,
                                  int K, uint16_t* idx, float* dist, double* objective, int64_t* n_resolved,
                                  cudaStream_t);

// Compressed linear layer: y = x . decode(C16, idx)^T (+ bias), the decoded weight never stored.
size_t cc_linear_scratch_bytes(int64_t M, int64_t d_out, int64_t d_in, int sm_count);
int cc_linear_q_table_max(void);
cudaError_t cc_launch_linear_forward(cc_ctx*, const uint16_t* x, int64_t M, const uint16_t* C16, const unsigned char* qtab,
                                     const float* qscale, int K, int g, const uint16_t* idx, int64_t d_out, int64_t d_in,
                                     const float* bias, float* y, cudaStream_t);

cudaError_t cc_launch_quantize_codebook(cc_ctx*, const uint16_t* C16, int64_t n, int bits, uint8_t* q, float* scale,
                                        uint16_t* deq, cudaStream_t);
cudaError_t cc_launch_gather_rows(cc_ctx*, const uint16_t* X, int g, const unsigned* pos_dev, int64_t n, uint16_t* out,
                                  cudaStream_t);
cudaError_t cc_launch_split_empty(cc_ctx*, const WsLayout&, float* C, int K, int g, const int32_t* counts, cudaStream_t);

cudaError_t cc_launch_update(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const uint16_t* idx,
                             int K, float* C, int32_t* counts, cudaStream_t);
cudaError_t cc_launch_codebook_grad(cc_ctx*, const WsLayout&, const uint16_t* dX, int64_t N, int g, const uint16_t* idx,
                                    int K, float* dC, cudaStream_t);
cudaError_t cc_launch_update_delta(cc_ctx*, const WsLayout&, const uint16_t* X, int64_t N, int g, const uint16_t* idx,
                                   uint16_t* idx_prev, int K, float* C, int32_t* counts, cudaStream_t);
