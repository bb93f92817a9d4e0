// Attention backward for callers that cannot provide (or allocate) the row-sum scratch.
//
// streambp_attention_backward needs a scratch array delta[n_q_heads, n] = rowsum(dO * O) in device
// memory, normally handed in by the caller.  Some callers have no way to get such a buffer at the
// point of the call: a host thread inside a latency-critical loop where cudaMalloc / cudaFree would
// synchronise the whole device, a plug-in running under a framework that has already reserved all
// device memory for its own pool, or code that runs after the process's memory budget was frozen.
// For them this file keeps the scratch in a fixed array that is part of the library image: every GPU
// that loads the library holds STREAMBP_STATIC_DELTA_MAX_FLOATS * 4 bytes (4 MiB) from load to exit.
//
// The array's name is only a host-side handle; kernels need its device address, which is looked up
// once per device with cudaGetSymbolAddress (with that device current) on the first call made on
// that device.  Nothing here calls cudaMalloc, cudaFree or any allocating library routine.
#include "common.cuh"

namespace sbp {
namespace {

constexpr int64_t kMaxDeltaFloats = STREAMBP_STATIC_DELTA_MAX_FLOATS;

static __device__ __align__(256) float g_static_delta[kMaxDeltaFloats];

std::mutex g_setup_mutex;
float *g_delta_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch on the current device (looked up on first use).
int static_delta(float **out) {
    int dev = -1;
    if (!cuda_ok(cudaGetDevice(&dev))) return STREAMBP_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return STREAMBP_E_SHAPE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_delta_ptr[dev] == nullptr) {
        void *p = nullptr;
        if (!cuda_ok(cudaGetSymbolAddress(&p, g_static_delta)) || p == nullptr) return STREAMBP_E_CUDA;
        g_delta_ptr[dev] = static_cast<float *>(p);
    }
    *out = g_delta_ptr[dev];
    return STREAMBP_OK;
}

}  // namespace
}  // namespace sbp

using namespace sbp;

extern "C" int streambp_attention_backward_static(const void *q, const void *k, const void *v, const void *o,
                                                  const void *d_o, const float *lse, int64_t n, int64_t q0,
                                                  int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                                  int32_t dtype, float *dq, float *dk, float *dv, int engine,
                                                  void *cuda_stream) {
    if (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv) return STREAMBP_E_NULL;
    if (n < 1 || q0 < 0 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
        (head_dim != 64 && head_dim != 128))
        return STREAMBP_E_SHAPE;
    // the fixed scratch holds n_q_heads * n row sums: larger problems are refused, never truncated
    if (n > kMaxDeltaFloats / n_q_heads) return STREAMBP_E_WORKSPACE;
    if (dtype != STREAMBP_F32 && dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (engine < 0 || engine > 2) return STREAMBP_E_SHAPE;      // 0 automatic, 1 CUDA cores, 2 tensor cores (two-role kernel)
    if (dtype == STREAMBP_F32 && engine == 2) return STREAMBP_E_DTYPE;
    // misaligned tensors are refused on the host: on the device they would fault and poison the context
    if (!attention_bwd_aligned(q, k, v, o, d_o, lse, nullptr, dq, dk, dv)) return STREAMBP_E_ALIGN;
    float *delta = nullptr;
    SBP_TRY(static_delta(&delta));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    call_state().cuda_error = 0;
    call_state().launches = 0;
    // delta is fully rewritten for rows [0, n) of every head before it is read: nothing to clear.
    if (dtype == STREAMBP_F32)
        return attention_bwd<float>((const float *)q, (const float *)k, (const float *)v, (const float *)o,
                                    (const float *)d_o, lse, n, q0, n_q_heads, n_kv_heads, head_dim, delta, dq, dk, dv,
                                    st);
    const bf16 *qb = (const bf16 *)q, *kb = (const bf16 *)k, *vb = (const bf16 *)v, *ob = (const bf16 *)o,
               *dob = (const bf16 *)d_o;
    const bool tc_ok = attention_tc_supported(n, q0, n_q_heads, n_kv_heads, head_dim, q, k, v);
    if (engine == 2 && !tc_ok) return STREAMBP_E_SHAPE;
    if (engine != 1 && tc_ok) {
        SBP_TRY(attention_delta<bf16>(ob, dob, n, n_q_heads, head_dim, delta, st));
        return attention_bwd_tc(qb, kb, vb, dob, lse, delta, n, q0, n_q_heads, n_kv_heads, dq, dk, dv, st);
    }
    return attention_bwd<bf16>(qb, kb, vb, ob, dob, lse, n, q0, n_q_heads, n_kv_heads, head_dim, delta, dq, dk, dv, st);
}
