// C ABI of the library: host-side validation, workspace carving, the Lloyd loop.
// Every step of the path runs in the kernels of the other translation units; nothing here
// computes on the host except the seeded choice of the K initial positions.
#include <new>
#include <unordered_map>
#include <vector>

#include "cc_common.cuh"

WsLayout cc_ws_layout(int64_t N, int g, int K) {
    WsLayout L;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += cc_align_up(bytes ? bytes : 1, 256); return o; };
    const size_t Kpad = cc_align_up((size_t)K, CC_KPAD);
    L.status = take(CC_STATUS_BYTES);
    L.cprep = take(Kpad / 2 * (size_t)(g + 1) * 16);
    L.flagged = take((size_t)N * 4);
    L.partials = take((size_t)CC_OBJ_BLOCKS * 8);
    const size_t R = (size_t)cc_sum_copies(K, g);
    L.sum_lo = take(R * K * g * 8);
    L.sum_hi = take(R * K * g * 8);
    L.count_copies = take(R * K * 4);
    L.tmp_c = take((size_t)K * g * 4);
    L.positions = take((size_t)K * 8);
    L.dist_tmp = take((size_t)N * 4);
    // tensor-core staging: FP16 operand image (at most 96 bytes per centroid) followed by the FP32
    // rows of the finish kernel (at most 68 bytes per centroid)
    L.tensor = take(Kpad * (size_t)(64 + 1) * 4);
    L.tstate = take((size_t)N * 8);
    L.idx_prev = take((size_t)N * 2);
    L.total = off;
    return L;
}

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

cc_status check_common(const cc_ctx* ctx, int64_t N, int g, int K, bool need_ws) {
    if (!ctx) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (N < 0 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (need_ws) {
        if (!ctx->ws) return CC_ERR_WORKSPACE;
        if (ctx->ws_bytes < cc_ws_layout(N, g, K).total) return CC_ERR_WORKSPACE;
    }
    return CC_OK;
}

inline cc_status from_cuda(cudaError_t e) { return e == cudaSuccess ? CC_OK : CC_ERR_CUDA; }

inline uint64_t splitmix64(uint64_t& s) {
    uint64_t z = (s += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// The same shuffle for any number n <= N of positions, written to 32-bit words: with many positions
// the whole array is kept, with few only the touched entries.
bool partial_shuffle_u32(int64_t N, int64_t n, uint64_t seed, uint32_t* pos) {
    uint64_t s = seed;
    if (n * 8 >= N) {
        std::vector<uint32_t> a;
        try { a.resize((size_t)N); } catch (...) { return false; }
        for (int64_t i = 0; i < N; ++i) a[(size_t)i] = (uint32_t)i;
        for (int64_t i = 0; i < n; ++i) {
            const int64_t j = i + (int64_t)(splitmix64(s) % (uint64_t)(N - i));
            const uint32_t t = a[(size_t)i];
            a[(size_t)i] = a[(size_t)j];
            a[(size_t)j] = t;
            pos[i] = a[(size_t)i];
        }
        return true;
    }
    std::unordered_map<int64_t, int64_t> moved;
    moved.reserve((size_t)n * 2);
    for (int64_t i = 0; i < n; ++i) {
        const int64_t j = i + (int64_t)(splitmix64(s) % (uint64_t)(N - i));
        auto itj = moved.find(j);
        const int64_t vj = (itj == moved.end()) ? j : itj->second;
        auto iti = moved.find(i);
        const int64_t vi = (iti == moved.end()) ? i : iti->second;
        moved[j] = vi;
        moved[i] = vj;
        pos[i] = (uint32_t)vj;
    }
    return true;
}

// Only the K touched entries of the shuffled array are kept (a map from position to content).
void partial_shuffle(int64_t N, int K, uint64_t seed, int64_t* pos) {
    std::unordered_map<int64_t, int64_t> moved;
    moved.reserve((size_t)K * 2);
    uint64_t s = seed;
    for (int64_t i = 0; i < K; ++i) {
        const int64_t j = i + (int64_t)(splitmix64(s) % (uint64_t)(N - i));
        auto itj = moved.find(j);
        const int64_t vj = (itj == moved.end()) ? j : itj->second;
        auto iti = moved.find(i);
        const int64_t vi = (iti == moved.end()) ? i : iti->second;
        moved[j] = vi;
        moved[i] = vj;
        pos[i] = vj;
    }
}

bool use_tensor_path(const cc_ctx* ctx, int g, int K) {
    if (ctx->path == CC_PATH_FFMA) return false;
    if (!cc_tensor_path_supported(g, K)) return false;
    return true;   // AUTO and TENSOR: the tensor-core kernels win wherever they apply
}

cudaError_t assign_any(cc_ctx* ctx, const WsLayout& L, const uint16_t* X, int64_t N, int g, const float* C, int K,
                       uint16_t* idx, float* dist, double* objective, int64_t* n_resolved, cudaStream_t st) {
    if (!dist) dist = reinterpret_cast<float*>(static_cast<char*>(ctx->ws) + L.dist_tmp);
    if (use_tensor_path(ctx, g, K))
        return cc_launch_assign_tensor(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, st);
    return cc_launch_assign_ffma(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, st);
}

}  // namespace

extern "C" {

const char* cc_status_string(cc_status s) {
    switch (s) {
        case CC_OK: return "ok";
        case CC_ERR_NULL: return "null pointer";
        case CC_ERR_SHAPE: return "bad size";
        case CC_ERR_UNSUPPORTED_G: return "g outside 1..16";
        case CC_ERR_K_RANGE: return "K outside 1..65536";
        case CC_ERR_N_LT_K: return "fewer sub-vectors than centroids";
        case CC_ERR_ALIGN: return "pointer not 16-byte aligned";
        case CC_ERR_WORKSPACE: return "workspace missing or too small";
        case CC_ERR_NONFINITE: return "non-finite input";
        case CC_ERR_DEVICE_TIMEOUT: return "device-side wait ran out";
        case CC_ERR_CUDA: return "CUDA runtime error";
        case CC_ERR_LAYOUT: return "unknown layout or path";
        case CC_ERR_STATIC_CAPACITY: return "K * g above the fixed capacity of cc_update_static";
    }
    return "unknown status";
}

cc_status cc_create(cc_ctx** out, int device) {
    if (!out) return CC_ERR_NULL;
    *out = nullptr;
    int n = 0;
    if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return CC_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return CC_ERR_CUDA;
    cc_ctx* c = new (std::nothrow) cc_ctx();
    if (!c) return CC_ERR_CUDA;
    c->device = device;
    c->sm_count = prop.multiProcessorCount;
    c->path = CC_PATH_AUTO;
    c->ws = nullptr;
    c->ws_bytes = 0;
    c->launches = 0;
    c->pos_host = nullptr;
    c->pos_cap = 0;
    c->prof_on = 0;
    c->prof_used = c->prof_made = 0;
    c->prof = nullptr;
    c->e2e_buf = nullptr;
    c->e2e_bytes = 0;
    c->empty_rule = CC_EMPTY_KEEP;
    *out = c;
    return CC_OK;
}

cc_status cc_destroy(cc_ctx* ctx) {
    if (!ctx) return CC_ERR_NULL;
    delete[] ctx->pos_host;
    if (ctx->e2e_buf) {
        cudaSetDevice(ctx->device);
        cudaFree(ctx->e2e_buf);
    }
    if (ctx->prof) {
        cudaSetDevice(ctx->device);
        for (int i = 0; i < ctx->prof_made; ++i) { cudaEventDestroy(ctx->prof[i].a); cudaEventDestroy(ctx->prof[i].b); }
        delete[] ctx->prof;
    }
    delete ctx;
    return CC_OK;
}

size_t cc_workspace_bytes(int64_t N, int g, int K) {
    if (g < 1 || g > 16 || K < 1 || K > 65536 || N < 0 || N >= (int64_t)1 << 31) return 0;
    return cc_ws_layout(N, g, K).total;
}

cc_status cc_set_workspace(cc_ctx* ctx, void* workspace, size_t bytes) {
    if (!ctx) return CC_ERR_NULL;
    if (workspace && (!aligned16(workspace) || bytes < CC_STATUS_BYTES)) return CC_ERR_ALIGN;
    ctx->ws = workspace;
    ctx->ws_bytes = workspace ? bytes : 0;
    if (workspace) {
        if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
        if (cudaMemset(workspace, 0, CC_STATUS_BYTES) != cudaSuccess) return CC_ERR_CUDA;   // status block
    }
    return CC_OK;
}

cc_status cc_set_path(cc_ctx* ctx, int path) {
    if (!ctx) return CC_ERR_NULL;
    if (path != CC_PATH_AUTO && path != CC_PATH_FFMA && path != CC_PATH_TENSOR) return CC_ERR_LAYOUT;
    ctx->path = path;
    return CC_OK;
}

int64_t cc_launch_count(const cc_ctx* ctx) { return ctx ? ctx->launches : -1; }

int64_t cc_num_subvectors(int64_t d_out, int64_t d_in, int g, int layout) {
    if (d_out < 1 || d_in < 1 || g < 1) return -1;
    if (layout == CC_LAYOUT_PAPER_T) return d_in * ((d_out + g - 1) / g);
    if (layout == CC_LAYOUT_ROWS) return d_out * ((d_in + g - 1) / g);
    return -1;
}

double cc_bits_per_param(int64_t d_out, int64_t d_in, int g, int K) {
    const int64_t codes = cc_num_subvectors(d_out, d_in, g, CC_LAYOUT_PAPER_T);
    if (codes < 0 || K < 1) return -1.0;
    return (16.0 * (double)codes + 16.0 * (double)g * (double)K) / ((double)d_in * (double)d_out);
}

cc_status cc_reshape_subvectors(cc_ctx* ctx, const uint16_t* W, int64_t d_out, int64_t d_in, int g, int layout,
                                uint16_t* X, void* stream) {
    if (!ctx || !W || !X) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (layout != CC_LAYOUT_PAPER_T && layout != CC_LAYOUT_ROWS) return CC_ERR_LAYOUT;
    const int64_t N = cc_num_subvectors(d_out, d_in, g, layout);
    if (N < 1 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (!aligned16(W) || !aligned16(X)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cc_launch_reshape(ctx, W, d_out, d_in, g, layout, X, (cudaStream_t)stream));
}

cc_status cc_init_positions(int64_t N, int K, uint64_t seed, int64_t* positions_host) {
    if (!positions_host) return CC_ERR_NULL;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (N < 1 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (N < K) return CC_ERR_N_LT_K;
    partial_shuffle(N, K, seed, positions_host);
    return CC_OK;
}

cc_status cc_init_codebook(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, uint64_t seed, float* C,
                           void* stream) {
    if (!ctx || !X || !C) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1) return CC_ERR_SHAPE;
    if (N < K) return CC_ERR_N_LT_K;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    if (ctx->pos_cap < K) {
        delete[] ctx->pos_host;
        ctx->pos_host = new (std::nothrow) int64_t[K];
        ctx->pos_cap = ctx->pos_host ? K : 0;
        if (!ctx->pos_host) return CC_ERR_CUDA;
    }
    partial_shuffle(N, K, seed, ctx->pos_host);
    const WsLayout L = cc_ws_layout(N, g, K);
    int64_t* pos_dev = reinterpret_cast<int64_t*>(static_cast<char*>(ctx->ws) + L.positions);
    cudaStream_t st = (cudaStream_t)stream;
    // pageable source: the copy is staged before the call returns, so pos_host may be reused
    if (cudaMemcpyAsync(pos_dev, ctx->pos_host, sizeof(int64_t) * (size_t)K, cudaMemcpyHostToDevice, st) !=
        cudaSuccess)
        return CC_ERR_CUDA;
    return from_cuda(cc_launch_gather_init(ctx, X, g, K, pos_dev, C, st));
}

cc_status cc_set_codebook(cc_ctx* ctx, const float* C0, int K, int g, float* C, void* stream) {
    if (!ctx || !C0 || !C) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (!aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cudaMemcpyAsync(C, C0, sizeof(float) * (size_t)K * g, cudaMemcpyDefault, (cudaStream_t)stream));
}

cc_status cc_assign(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K, uint16_t* idx,
                    float* dist, double* objective, int64_t* n_resolved, void* stream) {
    if (!ctx || !C || (N > 0 && (!X || !idx))) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(assign_any(ctx, L, X, N, g, C, K, idx, dist, objective, n_resolved, (cudaStream_t)stream));
}

cc_status cc_last_flagged(cc_ctx* ctx, int64_t N, int g, int K, uint32_t* points, int64_t count, void* stream) {
    if (!ctx || (count > 0 && !points)) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (count < 0 || count > N) return CC_ERR_SHAPE;
    if (count == 0) return CC_OK;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(cudaMemcpyAsync(points, static_cast<char*>(ctx->ws) + L.flagged, sizeof(uint32_t) * (size_t)count,
                                     cudaMemcpyDefault, (cudaStream_t)stream));
}

int64_t cc_tensor_scores_ld(int K) { return (K < 1 || K > 65536) ? -1 : cc_tensor_score_ld(K); }

cc_status cc_tensor_scores(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K, float* scores,
                           void* stream) {
    if (!ctx || !C || !X || !scores) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1 || N > 65536) return CC_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(cc_launch_tensor_scores(ctx, L, X, N, g, C, K, scores, (cudaStream_t)stream));
}

cc_status cc_tensor_finish_only(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K,
                                const void* scan, uint16_t* idx, float* dist, void* stream) {
    if (!ctx || !C || !X || !scan || !idx || !dist) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1) return CC_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(C) || (reinterpret_cast<uintptr_t>(scan) & 7u)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(cc_launch_tensor_finish_only(ctx, L, X, N, g, C, K, scan, idx, dist, (cudaStream_t)stream));
}

cc_status cc_selftest_bounded_wait(cc_ctx* ctx, int64_t limit_cycles, int32_t* results, int64_t* cycles) {
    if (!ctx || !results || !cycles) return CC_ERR_NULL;
    if (limit_cycles < 1000 || limit_cycles > 4000000000LL) return CC_ERR_SHAPE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    void* dev = nullptr;
    if (cudaMalloc(&dev, 64) != cudaSuccess) return CC_ERR_CUDA;
    int* out_dev = static_cast<int*>(dev);
    long long* cyc_dev = reinterpret_cast<long long*>(static_cast<char*>(dev) + 16);
    cc_status st = CC_OK;
    long long cyc[2] = {0, 0};
    if (cudaMemset(dev, 0, 64) != cudaSuccess || cc_launch_wait_selftest(limit_cycles, out_dev, cyc_dev, 0) != cudaSuccess ||
        cudaMemcpy(results, out_dev, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(cyc, cyc_dev, sizeof(cyc), cudaMemcpyDeviceToHost) != cudaSuccess)
        st = CC_ERR_CUDA;
    cycles[0] = cyc[0];
    cycles[1] = cyc[1];
    cudaFree(dev);
    return st;
}

cc_status cc_update(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const uint16_t* idx, int K, float* C,
                    int32_t* counts, void* stream) {
    if (!ctx || !C || !counts || (N > 0 && (!X || !idx))) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(cc_launch_update(ctx, L, X, N, g, idx, K, C, counts, (cudaStream_t)stream));
}

cc_status cc_codebook_grad(cc_ctx* ctx, const uint16_t* dX, int64_t N, int g, const uint16_t* idx, int K, float* dC,
                           void* stream) {
    if (!ctx || !dC || (N > 0 && (!dX || !idx))) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (!aligned16(dX) || !aligned16(dC)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    return from_cuda(cc_launch_codebook_grad(ctx, L, dX, N, g, idx, K, dC, (cudaStream_t)stream));
}

cc_status cc_fit(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, int iters, float* C, uint16_t* idx,
                 float* dist, int32_t* counts, double* objective_trace, void* stream) {
    if (!ctx || !X || !C || !idx || !counts) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1 || iters < 0) return CC_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    cudaStream_t st = (cudaStream_t)stream;
    for (int it = 0; it < iters; ++it) {
        cudaError_t e = assign_any(ctx, L, X, N, g, C, K, idx, dist, objective_trace ? objective_trace + it : nullptr,
                                   nullptr, st);
        if (e != cudaSuccess) return CC_ERR_CUDA;
        // first M-step: all points; later ones: only the points whose code changed
        uint16_t* idx_prev = reinterpret_cast<uint16_t*>(static_cast<char*>(ctx->ws) + L.idx_prev);
        if (it == 0) {
            e = cc_launch_update(ctx, L, X, N, g, idx, K, C, counts, st);
            if (e == cudaSuccess && iters > 1)
                e = cudaMemcpyAsync(idx_prev, idx, sizeof(uint16_t) * (size_t)N, cudaMemcpyDeviceToDevice, st);
        } else {
            e = cc_launch_update_delta(ctx, L, X, N, g, idx, idx_prev, K, C, counts, st);
        }
        if (e != cudaSuccess) return CC_ERR_CUDA;
    }
    return CC_OK;
}

cc_status cc_set_empty_rule(cc_ctx* ctx, int rule) {
    if (!ctx) return CC_ERR_NULL;
    if (rule != CC_EMPTY_KEEP && rule != CC_EMPTY_SPLIT_LARGEST) return CC_ERR_LAYOUT;
    ctx->empty_rule = rule;
    return CC_OK;
}

int64_t cc_train_points(int64_t N, int K, int max_points_per_centroid) {
    if (N < 1 || K < 1 || K > 65536 || max_points_per_centroid < 1) return -1;
    const int64_t n = (int64_t)max_points_per_centroid * K;
    return n < N ? n : N;
}

cc_status cc_sample_positions(int64_t N, int64_t n, uint64_t seed, uint32_t* positions_host) {
    if (!positions_host) return CC_ERR_NULL;
    if (N < 1 || N >= (int64_t)1 << 31 || n < 0 || n > N) return CC_ERR_SHAPE;
    return partial_shuffle_u32(N, n, seed, positions_host) ? CC_OK : CC_ERR_CUDA;
}

cc_status cc_fit_sampled(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, int K, int iters, int max_points_per_centroid,
                         uint64_t seed, uint16_t* X_train, float* C, uint16_t* idx, float* dist, int32_t* counts,
                         double* objective_trace, void* stream) {
    if (!ctx || !X || !C || !idx || !counts) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1 || iters < 0 || max_points_per_centroid < 1) return CC_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(C)) return CC_ERR_ALIGN;
    const int64_t n = cc_train_points(N, K, max_points_per_centroid);
    if (n < N && !X_train) return CC_ERR_NULL;
    if (n < N && !aligned16(X_train)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    if (n < N) {
        std::vector<uint32_t> pos;
        try { pos.resize((size_t)n); } catch (...) { return CC_ERR_CUDA; }
        if (!partial_shuffle_u32(N, n, seed, pos.data())) return CC_ERR_CUDA;
        const WsLayout L = cc_ws_layout(N, g, K);
        unsigned* pos_dev = reinterpret_cast<unsigned*>(static_cast<char*>(ctx->ws) + L.flagged);   // free until the first E-step
        // pageable source: the copy is staged before the call returns, so `pos` may go out of scope
        if (cudaMemcpyAsync(pos_dev, pos.data(), sizeof(uint32_t) * (size_t)n, cudaMemcpyHostToDevice, st) != cudaSuccess)
            return CC_ERR_CUDA;
        if (cc_launch_gather_rows(ctx, X, g, pos_dev, n, X_train, st) != cudaSuccess) return CC_ERR_CUDA;
        s = cc_fit(ctx, X_train, n, g, K, iters, C, idx, dist, counts, objective_trace, stream);
    } else {
        s = cc_fit(ctx, X, N, g, K, iters, C, idx, dist, counts, objective_trace, stream);
    }
    if (s != CC_OK) return s;
    return cc_assign(ctx, X, N, g, C, K, idx, dist, nullptr, nullptr, stream);
}

cc_status cc_quantize_codebook(cc_ctx* ctx, const uint16_t* C16, int K, int g, int bits, uint8_t* q, float* scale,
                               uint16_t* C16_dequantized, void* stream) {
    if (!ctx || !C16 || !q || !scale) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (bits != 8 && bits != 4) return CC_ERR_SHAPE;
    if (!ctx->ws || ctx->ws_bytes < 256) return CC_ERR_WORKSPACE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cc_launch_quantize_codebook(ctx, C16, (int64_t)K * g, bits, q, scale, C16_dequantized,
                                                 (cudaStream_t)stream));
}

cc_status cc_schedule_matrices(int n, const int64_t* sizes_host, int world, int rank, int32_t* mine_host, int32_t* n_mine_host) {
    if (!sizes_host || !mine_host || !n_mine_host) return CC_ERR_NULL;
    if (n < 0 || world < 1 || rank < 0 || rank >= world) return CC_ERR_SHAPE;
    // longest-processing-time first: matrices by decreasing size (lower index first among equals), each to
    // the rank with the smallest load so far (lowest rank among equals)
    std::vector<int> order((size_t)n);
    for (int i = 0; i < n; ++i) order[(size_t)i] = i;
    for (int i = 1; i < n; ++i) {                 // insertion sort: stable, n is a few hundred at most
        const int v = order[(size_t)i];
        int j = i - 1;
        while (j >= 0 && sizes_host[order[(size_t)j]] < sizes_host[v]) { order[(size_t)j + 1] = order[(size_t)j]; --j; }
        order[(size_t)j + 1] = v;
    }
    std::vector<int64_t> load((size_t)world, 0);
    std::vector<char> is_mine((size_t)n, 0);
    for (int k = 0; k < n; ++k) {
        const int i = order[(size_t)k];
        int r = 0;
        for (int q = 1; q < world; ++q) if (load[(size_t)q] < load[(size_t)r]) r = q;
        load[(size_t)r] += sizes_host[i];
        if (r == rank) is_mine[(size_t)i] = 1;
    }
    int m = 0;
    for (int i = 0; i < n; ++i) if (is_mine[(size_t)i]) mine_host[m++] = i;
    *n_mine_host = m;
    return CC_OK;
}

cc_status cc_compress_many(cc_ctx* ctx, int n, const uint16_t* const* W_hosts, const int64_t* d_outs, const int64_t* d_ins,
                           int g, int K, int iters, const uint64_t* seeds, int layout, uint16_t* const* C16_hosts,
                           uint16_t* const* idx_hosts, double* const* objective_trace_hosts, uint16_t* const* W_hat_hosts,
                           void* stream) {
    if (!ctx || !W_hosts || !d_outs || !d_ins || !seeds || !C16_hosts || !idx_hosts) return CC_ERR_NULL;
    if (n < 0) return CC_ERR_SHAPE;
    for (int i = 0; i < n; ++i) {
        const cc_status s = cc_compress_host(ctx, W_hosts[i], d_outs[i], d_ins[i], g, K, iters, seeds[i], layout, C16_hosts[i],
                                             idx_hosts[i], objective_trace_hosts ? objective_trace_hosts[i] : nullptr,
                                             W_hat_hosts ? W_hat_hosts[i] : nullptr, stream);
        if (s != CC_OK) return s;
    }
    return CC_OK;
}

cc_status cc_finalize(cc_ctx* ctx, const uint16_t* X, int64_t N, int g, const float* C, int K, uint16_t* C16,
                      uint16_t* idx, float* dist, double* objective, void* stream) {
    if (!ctx || !X || !C || !C16 || !idx) return CC_ERR_NULL;
    cc_status s = check_common(ctx, N, g, K, true);
    if (s != CC_OK) return s;
    if (N < 1) return CC_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(C) || !aligned16(C16)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    const WsLayout L = cc_ws_layout(N, g, K);
    cudaStream_t st = (cudaStream_t)stream;
    float* widened = reinterpret_cast<float*>(static_cast<char*>(ctx->ws) + L.tmp_c);
    cudaError_t e = cc_launch_to_half(ctx, C, (int64_t)K * g, C16, widened, st);
    if (e != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(assign_any(ctx, L, X, N, g, widened, K, idx, dist, objective, nullptr, st));
}

cc_status cc_decode(cc_ctx* ctx, const uint16_t* C16, int K, int g, const uint16_t* idx, int64_t d_out,
                    int64_t d_in, int layout, uint16_t* W_hat, void* stream) {
    if (!ctx || !C16 || !idx || !W_hat) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (layout != CC_LAYOUT_PAPER_T && layout != CC_LAYOUT_ROWS) return CC_ERR_LAYOUT;
    const int64_t N = cc_num_subvectors(d_out, d_in, g, layout);
    if (N < 1 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (!aligned16(C16) || !aligned16(W_hat)) return CC_ERR_ALIGN;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cc_launch_decode(ctx, C16, K, g, idx, d_out, d_in, layout, W_hat, (cudaStream_t)stream));
}

size_t cc_linear_workspace_bytes(cc_ctx* ctx, int64_t M, int64_t d_out, int64_t d_in) {
    if (!ctx || M < 1 || d_out < 1 || d_in < 1 || M * d_out >= (int64_t)1 << 31 || d_in >= (int64_t)1 << 31) return 0;
    return cc_linear_scratch_bytes(M, d_out, d_in, ctx->sm_count);
}

cc_status cc_linear_forward(cc_ctx* ctx, const uint16_t* x, int64_t M, const uint16_t* C16, int K, int g,
                            const uint16_t* idx, int64_t d_out, int64_t d_in, const float* bias, float* y,
                            void* stream) {
    if (!ctx || !x || !C16 || !idx || !y) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    const int64_t N = cc_num_subvectors(d_out, d_in, g, CC_LAYOUT_PAPER_T);
    if (N < 1 || N >= (int64_t)1 << 31 || M < 1 || M * d_out >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(C16) || !aligned16(y)) return CC_ERR_ALIGN;
    if (!ctx->ws || ctx->ws_bytes < cc_linear_scratch_bytes(M, d_out, d_in, ctx->sm_count)) return CC_ERR_WORKSPACE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cc_launch_linear_forward(ctx, x, M, C16, nullptr, nullptr, K, g, idx, d_out, d_in, bias, y,
                                              (cudaStream_t)stream));
}

cc_status cc_linear_forward_q4(cc_ctx* ctx, const uint16_t* x, int64_t M, const uint8_t* q, const float* scale, int K, int g,
                               const uint16_t* idx, int64_t d_out, int64_t d_in, const float* bias, float* y, void* stream) {
    if (!ctx || !x || !q || !scale || !idx || !y) return CC_ERR_NULL;
    if (g < 2 || g > 16 || (g & 1)) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    const int64_t N = cc_num_subvectors(d_out, d_in, g, CC_LAYOUT_PAPER_T);
    if (N < 1 || N >= (int64_t)1 << 31 || M < 1 || M * d_out >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if ((int64_t)K * (g / 2) > cc_linear_q_table_max()) return CC_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(q) || !aligned16(y)) return CC_ERR_ALIGN;
    if (!ctx->ws || ctx->ws_bytes < cc_linear_scratch_bytes(M, d_out, d_in, ctx->sm_count)) return CC_ERR_WORKSPACE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    return from_cuda(cc_launch_linear_forward(ctx, x, M, nullptr, q, scale, K, g, idx, d_out, d_in, bias, y,
                                              (cudaStream_t)stream));
}

cc_status cc_poll_status(cc_ctx* ctx, void* stream) {
    if (!ctx) return CC_ERR_NULL;
    if (!ctx->ws) return CC_ERR_WORKSPACE;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    unsigned word = 0;
    if (cudaMemcpyAsync(&word, ctx->ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return CC_ERR_CUDA;
    if (cudaMemsetAsync(ctx->ws, 0, sizeof(word), st) != cudaSuccess) return CC_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return CC_ERR_CUDA;
    if (word & CC_DEV_TIMEOUT) return CC_ERR_DEVICE_TIMEOUT;
    if (word & CC_DEV_NONFINITE) return CC_ERR_NONFINITE;
    return CC_OK;
}

cc_status cc_compress_host(cc_ctx* ctx, const uint16_t* W_host, int64_t d_out, int64_t d_in, int g, int K, int iters,
                           uint64_t seed, int layout, uint16_t* C16_host, uint16_t* idx_host,
                           double* objective_trace_host, uint16_t* W_hat_host, void* stream) {
    if (!ctx || !W_host || !C16_host || !idx_host) return CC_ERR_NULL;
    if (g < 1 || g > 16) return CC_ERR_UNSUPPORTED_G;
    if (K < 1 || K > 65536) return CC_ERR_K_RANGE;
    if (layout != CC_LAYOUT_PAPER_T && layout != CC_LAYOUT_ROWS) return CC_ERR_LAYOUT;
    if (iters < 0) return CC_ERR_SHAPE;
    const int64_t N = cc_num_subvectors(d_out, d_in, g, layout);
    if (N < 1 || N >= (int64_t)1 << 31) return CC_ERR_SHAPE;
    if (N < K) return CC_ERR_N_LT_K;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return CC_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;

    const size_t w_bytes = (size_t)d_out * d_in * 2, x_bytes = (size_t)N * g * 2;
    const size_t ws_bytes = cc_ws_layout(N, g, K).total;
    // one allocation, carved: W | X | C | C16 | idx | dist | counts | trace | workspace
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off += cc_align_up(b, 256); return o; };
    const size_t oW = take(w_bytes), oX = take(x_bytes), oC = take((size_t)K * g * 4), oC16 = take((size_t)K * g * 2),
                 oIdx = take((size_t)N * 2), oDist = take((size_t)N * 4), oCnt = take((size_t)K * 4),
                 oTr = take((size_t)(iters + 1) * 8), oWs = take(ws_bytes);
    if (ctx->e2e_bytes < off) {          // grown on demand and kept: repeated calls allocate nothing
        if (ctx->e2e_buf) cudaFree(ctx->e2e_buf);
        ctx->e2e_buf = nullptr;
        ctx->e2e_bytes = 0;
        if (cudaMalloc(&ctx->e2e_buf, off) != cudaSuccess) return CC_ERR_CUDA;
        ctx->e2e_bytes = off;
    }
    char* base = static_cast<char*>(ctx->e2e_buf);
    void* saved_ws = ctx->ws;
    const size_t saved_bytes = ctx->ws_bytes;
    cc_status s = cc_set_workspace(ctx, base + oWs, ws_bytes);
    uint16_t* W = (uint16_t*)(base + oW);
    uint16_t* X = (uint16_t*)(base + oX);
    float* C = (float*)(base + oC);
    uint16_t* C16 = (uint16_t*)(base + oC16);
    uint16_t* idx = (uint16_t*)(base + oIdx);
    float* dist = (float*)(base + oDist);
    int32_t* counts = (int32_t*)(base + oCnt);
    double* trace = (double*)(base + oTr);
    if (s == CC_OK && cudaMemcpyAsync(W, W_host, w_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) s = CC_ERR_CUDA;
    if (s == CC_OK) s = cc_reshape_subvectors(ctx, W, d_out, d_in, g, layout, X, st);
    if (s == CC_OK) s = cc_init_codebook(ctx, X, N, g, K, seed, C, st);
    if (s == CC_OK) s = cc_fit(ctx, X, N, g, K, iters, C, idx, dist, counts, trace, st);
    if (s == CC_OK) s = cc_finalize(ctx, X, N, g, C, K, C16, idx, dist, trace + iters, st);
    if (s == CC_OK && W_hat_host) {
        s = cc_decode(ctx, C16, K, g, idx, d_out, d_in, layout, W, st);   // W is no longer needed
        if (s == CC_OK && cudaMemcpyAsync(W_hat_host, W, w_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
            s = CC_ERR_CUDA;
    }
    if (s == CC_OK && cudaMemcpyAsync(C16_host, C16, (size_t)K * g * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        s = CC_ERR_CUDA;
    if (s == CC_OK && cudaMemcpyAsync(idx_host, idx, (size_t)N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        s = CC_ERR_CUDA;
    if (s == CC_OK && objective_trace_host &&
        cudaMemcpyAsync(objective_trace_host, trace, (size_t)(iters + 1) * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        s = CC_ERR_CUDA;
    if (s == CC_OK) s = cc_poll_status(ctx, st);
    else cudaStreamSynchronize(st);
    ctx->ws = saved_ws;
    ctx->ws_bytes = saved_bytes;
    return s;
}

}  // extern "C"
