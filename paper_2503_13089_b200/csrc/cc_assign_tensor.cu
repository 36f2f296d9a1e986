// E-step on the tcgen05 tensor cores (placeholder until the kernels land: reports "unsupported",
// so every call takes the FP32 FMA path).
#include "cc_common.cuh"

bool cc_tensor_path_supported(int, int) { return false; }

cudaError_t cc_launch_assign_tensor(cc_ctx*, const WsLayout&, const uint16_t*, int64_t, int, const float*, int,
                                    uint16_t*, float*, double*, int64_t*, cudaStream_t) {
    return cudaErrorNotSupported;
}
