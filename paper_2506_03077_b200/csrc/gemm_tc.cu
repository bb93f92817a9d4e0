// tcgen05 tensor-core GEMM (placeholder until the kernel lands): reports every shape as unsupported.
#include "common.cuh"

namespace sbp {
bool gemm_tc_supported(GemmOp, int64_t, int64_t, int64_t, int64_t, int64_t, int64_t, const void *, const void *,
                       const void *, bool) {
    return false;
}
int gemm_tc(GemmOp, int64_t, int64_t, int64_t, const bf16 *, int64_t, const bf16 *, int64_t, void *, int64_t, bool,
            const bf16 *, bool, cudaStream_t) {
    return STREAMBP_E_SHAPE;
}
}  // namespace sbp
