// Shared declarations of the streamed-backward CUDA library (internal).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>
#include <vector>

#include "../../include/streambp.h"

namespace sbp {

typedef __nv_bfloat16 bf16;

// ---- per-thread call context -------------------------------------------------
struct CallState {
    int cuda_error = 0;
    int64_t launches = 0;
    // Optional device-side gate for the launches that follow: kernels that honour it return at once
    // (or write exact zeros, where an output must still be defined) when *gate == 0.  Used by the LM
    // head to skip chunks whose labels are all ignored without a host round trip.
    const int *gate = nullptr;
    // Device memory for the dynamic tile schedule of grouped products: kSchedSlots pairs of ints inside the
    // current call's workspace header (zero between launches), used in rotation; nullptr = static schedule.
    int *sched = nullptr;
    int sched_slot = 0;
};
CallState &call_state();

inline bool cuda_ok(cudaError_t e) {
    if (e != cudaSuccess) {
        call_state().cuda_error = (int)e;
        return false;
    }
    return true;
}

// ---- per-device one-time state ------------------------------------------------------
// The SM count, the opt-in to large dynamic shared memory (cudaFuncSetAttribute) and the choice of product kernel
// are properties of a DEVICE, and one process may drive several: each is computed once per device ordinal (the
// device current at the call), under a mutex, so host threads and devices never see each other's answer.
constexpr int kMaxDevices = 64;
int current_device_ordinal();             // cudaGetDevice, or the ordinal a test has put in its place; -1 on error
class PerDevice {
    std::mutex m_;
    int value_[kMaxDevices];
    bool have_[kMaxDevices] = {};
public:
    // the value for the current device; `init` runs once per device (again on every call where the ordinal
    // cannot be read or is out of range: nothing is cached then)
    template <typename F> int get(F init) {
        const int dev = current_device_ordinal();
        if (dev < 0 || dev >= kMaxDevices) return init();
        std::lock_guard<std::mutex> lock(m_);
        if (!have_[dev]) {
            value_[dev] = init();
            have_[dev] = true;
        }
        return value_[dev];
    }
};

// Every kernel launch goes through this so launches are counted and launch errors
// are caught without synchronising.
// Every kernel of the library starts with pdl_enter(): it waits until the grids before it in the stream have
// completed and their writes are visible, then lets the grid after it be scheduled early (programmatic dependent
// launch: that grid's blocks become resident as this grid's blocks retire and sit in their own pdl_enter() until this
// grid is done).  At most one grid is launched ahead, and no kernel touches memory before the wait.
__device__ __forceinline__ void pdl_enter() {
#ifdef __CUDA_ARCH__
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#endif
}
bool pdl_enabled();   // STREAMBP_PDL (read once per process)

#define SBP_LAUNCH(kernel, grid_, block_, smem_, stream_, ...)                     \
    do {                                                                           \
        cudaLaunchConfig_t _cfg;                                                   \
        memset(&_cfg, 0, sizeof(_cfg));                                            \
        _cfg.gridDim = dim3(grid_);                                                \
        _cfg.blockDim = dim3(block_);                                              \
        _cfg.dynamicSmemBytes = (smem_);                                           \
        _cfg.stream = (stream_);                                                   \
        cudaLaunchAttribute _attr[1];                                              \
        _attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;          \
        _attr[0].val.programmaticStreamSerializationAllowed = 1;                   \
        _cfg.attrs = _attr;                                                        \
        _cfg.numAttrs = ::sbp::pdl_enabled() ? 1 : 0;                              \
        cudaError_t _le = cudaLaunchKernelEx(&_cfg, kernel, __VA_ARGS__);          \
        ::sbp::call_state().launches++;                                            \
        if (!::sbp::cuda_ok(_le) || !::sbp::cuda_ok(cudaGetLastError())) return STREAMBP_E_CUDA; \
    } while (0)

#define SBP_TRY(expr)                         \
    do {                                      \
        int _st = (expr);                     \
        if (_st != STREAMBP_OK) return _st;   \
    } while (0)

// ---- NVTX ranges -----------------------------------------------------------------------
// Host-side ranges around every call, chunk and phase of the schedulers, visible in a timeline profiler
// (header-only NVTX: without a profiler attached a range costs a null-pointer check).
struct NvtxRange {
    explicit NvtxRange(const char *name);
    NvtxRange(const char *name, long long index);     // "name index"
    ~NvtxRange();
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};

// ---- optional per-class device timing (off by default) -----------------------------
// When enabled through streambp_profile_enable(), every product and attention launch is bracketed
// by CUDA events on the caller's stream; the algorithmic FLOPs of the bracketed work are summed.
enum KernelClass { KC_GEMM = 0, KC_ATTN_FWD = 1, KC_ATTN_BWD = 2, KC_CLASSES = 3 };
struct ProfScope {
    int idx;
    cudaStream_t st;
    ProfScope(int cls, double flops, cudaStream_t stream);
    ~ProfScope();
};

__device__ __forceinline__ bool gated_off(const int *gate) { return gate != nullptr && *gate == 0; }

// ---- scalar conversion -------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// ---- 16-byte vector access -----------------------------------------------------
// Vec<T>::N elements of T in one 16-byte load/store.
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    float v[4];
    __device__ __forceinline__ void load(const float *p) {
        float4 t = *reinterpret_cast<const float4 *>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    __device__ __forceinline__ void store(float *p) const {
        *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Vec<bf16> {
    static constexpr int N = 8;
    float v[8];
    __device__ __forceinline__ void load(const bf16 *p) {
        uint4 t = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ __forceinline__ void store(bf16 *p) const {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Block-wide sum for blocks of up to 1024 threads; `red` holds 33 floats of shared memory.
__device__ __forceinline__ float block_sum(float v, float *red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    if (w == 0) {
        float t = lane < nw ? red[lane] : 0.f;
        t = warp_sum(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}
__device__ __forceinline__ float block_max(float v, float *red) {
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) red[w] = v;
    __syncthreads();
    if (w == 0) {
        float t = lane < nw ? red[lane] : -INFINITY;
        t = warp_max(t);
        if (lane == 0) red[32] = t;
    }
    __syncthreads();
    return red[32];
}

// ---- workspace header ----------------------------------------------------------
// First 256 bytes of every workspace. `status` is the first non-OK device status.
struct WsHeader {
    int32_t status;
    int32_t detail;
    unsigned long long n_valid;
    double loss_sum;
    float factor;       // DPO: sigmoid(beta * ell) - 1, the in-place correction applied after the chunk loop
    int32_t pad_[9];
    int32_t sched[16];  // tile counters of grouped products (see CallState::sched), at byte 64
};
static constexpr size_t kHeaderBytes = 256;
static constexpr int kSchedSlots = 8;
static_assert(sizeof(WsHeader) <= kHeaderBytes, "workspace header too large");

// Points the grouped products of the enclosed launches at the counters of this workspace header.
struct SchedScope {
    int *saved;
    explicit SchedScope(WsHeader *hdr) : saved(call_state().sched) {
        call_state().sched = reinterpret_cast<int *>(reinterpret_cast<char *>(hdr) + 64);
    }
    ~SchedScope() { call_state().sched = saved; }
};

__device__ __forceinline__ void set_status(WsHeader *h, int st, int detail) {
    if (atomicCAS(&h->status, 0, st) == 0) h->detail = detail;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Bump allocator over the caller's workspace; also used (with base == nullptr) to plan sizes.
// Debug mode (environment STREAMBP_WS_GUARD set, read once per process): every sub-buffer is followed by a
// 256-byte guard that the schedulers fill with a pattern before the first launch of a call and check after the
// last one; a kernel that wrote past the end of its sub-buffer shows up as STREAMBP_E_WORKSPACE_GUARD in
// streambp_last_device_status (detail = index of the sub-buffer).  The stand-in for a memory checker on a pool
// where none can be run.  Workspace sizes grow accordingly, consistently in the size queries and in the calls.
bool ws_guard_enabled();
constexpr size_t kGuardBytes = 256;
struct Arena {
    char *base;
    size_t off;
    std::vector<size_t> guards;     // byte offsets of the guards (debug mode only)
    bool guarded;
    explicit Arena(void *b) : base(static_cast<char *>(b)), off(0), guarded(ws_guard_enabled()) {}
    template <typename T> T *take(size_t count) {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += count * sizeof(T);
        if (guarded) {      // the guard starts right behind the last element (rounded up to a word), not at the next boundary
            off = align_up(off, 4);
            guards.push_back(off);
            off += kGuardBytes;
        }
        return p;
    }
    void *take_bytes(size_t bytes) { return take<char>(bytes); }
    size_t size() const { return align_up(off, 256); }
};
// Fill / check the guards of a planned workspace (no-ops when the list is empty).
int ws_guards_arm(void *base, const std::vector<size_t> &guards, cudaStream_t st);
int ws_guards_check(void *base, const std::vector<size_t> &guards, WsHeader *hdr, cudaStream_t st);

// ---- internal kernels (host launchers); T = storage dtype -----------------------
enum GemmOp { OP_NT = 0, OP_NN = 1, OP_TN = 2 };

// CUDA-core GEMM: C[M,N] (+)= op(A,B) (+ bias[N]); TC is the type of C. Returns a streambp_status.
template <typename TI, typename TC>
int gemm(GemmOp op, int64_t M, int64_t N, int64_t K, const TI *A, int64_t lda, const TI *B, int64_t ldb,
         TC *C, int64_t ldc, const TI *bias, bool accumulate, cudaStream_t st);

// tcgen05 GEMM (bf16 operands, fp32 accumulation in tensor memory).
bool gemm_tc_supported(GemmOp op, int64_t M, int64_t N, int64_t K, int64_t lda, int64_t ldb, int64_t ldc,
                       const void *A, const void *B, const void *C, bool c_is_f32);
int gemm_tc(GemmOp op, int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *B, int64_t ldb,
            void *C, int64_t ldc, bool c_is_f32, const bf16 *bias, bool accumulate, cudaStream_t st);

// Several independent products in one launch.  A problem is C (+)= sum_s op(A_s, B_s) (+ bias) over
// up to three K segments that share M, N, the operand layout and C.
struct GemmSeg {
    const bf16 *A;
    int64_t lda;
    const bf16 *B;
    int64_t ldb;
    int64_t K;
};
struct GemmProb {
    GemmOp op;
    int64_t M, N;
    int nseg;
    GemmSeg seg[3];
    void *C;
    int64_t ldc;
    bool c_is_f32;
    const bf16 *bias;
    bool accumulate;
    // SwiGLU pair (CTA-pair kernel only): op NT, seg[0].B = W_gate, seg[1].B = W_up (same A, K); the three bf16
    // outputs C = g = A W_gate^T, C_up = u = A W_up^T and C_act = silu(g) * u share ldc.  N counts the columns of each.
    bool swiglu = false;
    void *C_up = nullptr, *C_act = nullptr;
    // Rotary embedding in the epilogue (bf16 output, heads of 128 columns, N a multiple of 128): row r of `rope` holds
    // (cos, sin) of the 64 frequencies at the position of row r of C; C = rotate(A B^T + bias), rounded once.
    const float *rope = nullptr;
};
bool gemm_tc_group_supported(const GemmProb *probs, int n);
// sched: two ints of device memory that are zero when the launch starts (the kernel leaves them zero),
// enabling the dynamic tile schedule; nullptr selects the static one.
int gemm_tc_group(const GemmProb *probs, int n, int *sched, cudaStream_t st);

// Reads and clears the flag a tensor-core kernel raises when one of its bounded waits expires.
int gemm_tc_take_fault();
int gemm_tc_variant();   // 2: CTA-pair kernel, 1: single-CTA kernel, 0: tensor maps unavailable

// Engine choice for the dispatching product below: 0 automatic, 1 CUDA cores only, 2 tensor cores required
// (STREAMBP_GEMM_ENGINE, read once per process).
int gemm_engine();

// Dispatching product used by the schedulers.
template <typename TI, typename TC>
int mm(GemmOp op, int64_t M, int64_t N, int64_t K, const TI *A, int64_t lda, const TI *B, int64_t ldb, TC *C,
       int64_t ldc, const TI *bias, bool accumulate, cudaStream_t st);

// h = x * rstd * gain ; rstd[t] saved. If res != nullptr: r = x + res is formed first, written to
// r_out (fp32) and normalised instead of x.
template <typename T>
int rmsnorm_fwd(const T *x, const float *res, const T *gain, float eps, int64_t rows, int d, T *h, float *rstd,
                float *r_out, cudaStream_t st);
// out = add + ((dh*gain) - xhat*mean((dh*gain)*xhat)) * rstd ; x is given as xT (storage) or xF (fp32).
// add: optional addT and/or addF. Outputs: optional outF (fp32) and outT (storage).
// dgain += sum_t dh*xhat, reduced through partials[rmsnorm_bwd_partials_rows(rows), d].
template <typename T>
int rmsnorm_bwd(const float *dh, const T *xT, const float *xF, const float *rstd, const T *gain, const T *addT,
                const float *addF, int64_t rows, int d, float *outF, T *outT, float *dgain, float *partials,
                cudaStream_t st);
int rmsnorm_bwd_partials_rows(int64_t rows);

// cs[t, j] = (cos, sin)((pos0 + t) * theta^(-2j/dh)), j < dh/2
int rope_table(float *cs, int64_t pos0, int64_t rows, int dh, float theta, cudaStream_t st);
// out[t,h,:] = R(t) in[t,h,:] (transpose = false) or R(t)^T in[t,h,:]; cs row 0 belongs to in row 0.
template <typename TO>
int rope_apply(const float *in, const float *cs, int64_t rows, int heads, int dh, bool transpose, TO *out,
               cudaStream_t st);
template <typename T>
int swiglu_fwd(const T *g, const T *u, int64_t n, T *m, cudaStream_t st);
// in place: g := dg = dm*u*silu'(g), u := du = dm*silu(g)
template <typename T>
int swiglu_bwd(const T *dm, T *g, T *u, int64_t n, cudaStream_t st);
// out (+)= column sums of a [rows, cols]; partials: [colsum_partial_rows(rows), cols]
template <typename T>
int colsum(const T *a, int64_t rows, int cols, float *out, bool accumulate, float *partials, cudaStream_t st);
int colsum_partial_rows(int64_t rows);
// o_i += column sums of a_i [rows, c_i], i = 0..2, in one pair of launches; partials: [colsum_partial_rows(rows), c0+c1+c2]
template <typename T>
int colsum3_add(const T *a0, int c0, float *o0, const T *a1, int c1, float *o1, const T *a2, int c2, float *o2,
                int64_t rows, float *partials, cudaStream_t st);
template <typename T>
int cast_from_f32(const float *in, int64_t n, T *out, cudaStream_t st);
// out = a + b (fp32 inputs)
template <typename T>
int add_cast(const float *a, const float *b, int64_t n, T *out, cudaStream_t st);
int fill_zero(void *p, size_t bytes, cudaStream_t st);
int ws_guard_selftest(void *ws, size_t bytes, int overrun, cudaStream_t st);

// Attention of one chunk of queries against the key/value prefix [0, q0 + n).
// q,o,do: [n, Hq, dh]; k,v: [q0+n, Hkv, dh]; query row i sits at absolute row q0 + i and sees keys <= q0 + i.
// lse: [Hq, n] (natural log, scores scaled by 1/sqrt(dh)).
template <typename T>
int attention_fwd(const T *q, const T *k, const T *v, int64_t n, int64_t q0, int Hq, int Hkv, int dh, T *o,
                  float *lse, cudaStream_t st);
// delta[h, i] = sum_j do*o (scratch [Hq, n]); dq fp32 [n,Hq,dh] overwritten; dk, dv fp32 [q0+n,Hkv,dh] accumulated.
template <typename T>
int attention_bwd(const T *q, const T *k, const T *v, const T *o, const T *dout, const float *lse, int64_t n,
                  int64_t q0, int Hq, int Hkv, int dh, float *delta, float *dq, float *dk, float *dv,
                  cudaStream_t st);

// tcgen05 attention (bf16, head_dim 128)
bool attention_tc_supported(int64_t n, int64_t q0, int Hq, int Hkv, int dh, const void *q, const void *k,
                            const void *v);
// tiles_per_cta: 0 = chosen from the grid size, 1 / 2 = one / two 128-query tiles per CTA (tests, profiling)
int attention_fwd_tc(const bf16 *q, const bf16 *k, const bf16 *v, int64_t n, int64_t q0, int Hq, int Hkv, bf16 *o,
                     float *lse, cudaStream_t st, int tiles_per_cta = 0);
// delta [Hq, n] must already hold rowsum(dO * O) (attention_delta below).  five_products: the single-role kernel
// whose key-tile owners also form dQ and add it into global memory (dq is cleared first; not bit-reproducible).
int attention_bwd_tc(const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *dout, const float *lse,
                     const float *delta, int64_t n, int64_t q0, int Hq, int Hkv, float *dq, float *dk, float *dv,
                     cudaStream_t st, bool five_products = false);
template <typename T>
int attention_delta(const T *o, const T *dout, int64_t n, int Hq, int dh, float *delta, cudaStream_t st);
int attention_tc_take_fault();
// Test kernel whose bounded wait is made to run out (wait_probe.cu).
int wait_probe_launch(unsigned long long limit_ns, cudaStream_t st);
int wait_probe_take_fault();
// Pointer alignment the attention backward entry points require (delta may be nullptr: not checked then).
bool attention_bwd_aligned(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                           const void *lse, const void *delta, const void *dq, const void *dk, const void *dv);
// Dispatching attention used by the schedulers (tensor cores when supported, else CUDA cores).
template <typename T>
int attn_fwd(const T *q, const T *k, const T *v, int64_t n, int64_t q0, int Hq, int Hkv, int dh, T *o, float *lse,
             cudaStream_t st);
// engine: -1 = the process-wide choice (gemm_engine()), else 0 / 1 / 2 as above for this call only; 5 = tensor cores,
// five-product kernel (the process-wide default of that choice: STREAMBP_ATTN_BWD=five).
template <typename T>
int attn_bwd(const T *q, const T *k, const T *v, const T *o, const T *dout, const float *lse, int64_t n, int64_t q0,
             int Hq, int Hkv, int dh, float *delta, float *dq, float *dk, float *dv, cudaStream_t st, int engine = -1);

// LM head pieces
int count_valid_labels(const int64_t *labels, int64_t T, int64_t vocab, int64_t ignore, WsHeader *hdr,
                       cudaStream_t st);
// counts[i] = number of labels != ignore in rows [i*chunk, min(T, (i+1)*chunk))
int count_valid_per_chunk(const int64_t *labels, int64_t T, int64_t chunk, int64_t ignore, int *counts,
                          cudaStream_t st);
// z: [rows, V] fp32 logits -> dz (storage dtype; may alias z when T == float); row_loss[rows] fp32.
template <typename T>
int ce_rows(const float *z, const int64_t *labels, int64_t rows, int64_t V, int64_t ignore, const WsHeader *hdr,
            T *dz, float *row_loss, cudaStream_t st);
int loss_accumulate(const float *row_loss, int64_t rows, WsHeader *hdr, cudaStream_t st);
// RL objectives of the LM head: per row, log pi(token) from the logits, then dz = c * (onehot - softmax) with the
// objective's coefficient c.  row_val: the row's contribution to the loss (GRPO) or to ell (DPO).
struct RlRows {
    int objective;            // STREAMBP_OBJ_GRPO / STREAMBP_OBJ_DPO
    float beta, clip_eps;
    const float *logp_old;    // GRPO
    const float *logp_ref;
    const float *advantage;   // GRPO
    const float *weight;      // GRPO: per-token weight; DPO: +1 chosen / -1 rejected
    float *logp_out;          // optional
};
template <typename T>
int rl_rows(const float *z, const int64_t *tokens, int64_t rows, int64_t V, int64_t ignore, const RlRows &rl,
            int64_t row0, T *dz, float *row_val, cudaStream_t st);
int rl_finalize(WsHeader *hdr, int objective, float beta, float *loss, float *ell, cudaStream_t st);
// p[i] *= hdr->factor
template <typename T>
int scale_by_factor(T *p, int64_t n, const WsHeader *hdr, cudaStream_t st);
int loss_finalize(WsHeader *hdr, float *loss, int64_t *n_valid, cudaStream_t st);

template <typename T>
int embedding_gather(const T *embed, const int64_t *ids, int64_t rows, int d, int64_t vocab, T *out, WsHeader *hdr,
                     cudaStream_t st);
template <typename T>
int embedding_scatter_add(const T *dx, const int64_t *ids, int64_t rows, int d, int64_t vocab, float *d_embed,
                          cudaStream_t st);

// Grouped products used by the schedulers: independent problems that become ready together go out as one
// launch (tensor cores) or one after the other (CUDA cores); a problem may sum several K segments.
template <typename T>
struct MmSeg {
    const T *A;
    int64_t lda;
    const T *B;
    int64_t ldb;
    int64_t K;
};
template <typename T>
struct MmProb {
    GemmOp op;
    int64_t M, N;
    int nseg;
    MmSeg<T> seg[3];
    void *C;            // fp32 if c_is_f32, else T
    int64_t ldc;
    bool c_is_f32;
    const T *bias;
    bool accumulate;
    // optional rotary embedding of the output (set by mm_set_rope): C (type T) = rotate(A B^T + bias)
    const float *rope = nullptr;
    float *rope_tmp = nullptr;
    int rope_heads = 0, rope_dh = 0;
};
template <typename T>
MmProb<T> mm_prob(GemmOp op, int64_t M, int64_t N, int64_t K, const T *A, int64_t lda, const T *B, int64_t ldb, void *C,
                  int64_t ldc, bool c_is_f32, const T *bias, bool accumulate) {
    MmProb<T> g{};
    g.op = op; g.M = M; g.N = N; g.nseg = 1;
    g.seg[0] = MmSeg<T>{A, lda, B, ldb, K};
    g.C = C; g.ldc = ldc; g.c_is_f32 = c_is_f32; g.bias = bias; g.accumulate = accumulate;
    return g;
}
// The output of g (type T, c_is_f32 must be false unless T is float) becomes the rotary embedding of the product:
// `cs` holds, per row of C, (cos, sin) of dh / 2 frequencies (rope_table's layout).  The tensor-core kernel rotates
// in its epilogue when dh = 128; otherwise the product goes to `tmp` (fp32 [M, N], dense) and a row kernel rotates.
template <typename T>
void mm_set_rope(MmProb<T> &g, const float *cs, int heads, int dh, float *tmp) {
    g.rope = cs; g.rope_heads = heads; g.rope_dh = dh; g.rope_tmp = tmp;
}
template <typename T>
void mm_add_seg(MmProb<T> &g, int64_t K, const T *A, int64_t lda, const T *B, int64_t ldb) {
    g.seg[g.nseg++] = MmSeg<T>{A, lda, B, ldb, K};
}
template <typename T>
int mm_group(const MmProb<T> *probs, int n, cudaStream_t st);
// g = A Wg^T, u = A Wu^T, m = silu(g) * u  (A [M, K], Wg / Wu [N, K], outputs [M, N], all row-major of type T).
// bf16 on the CTA-pair product kernel: ONE launch -- the even CTA of a pair fetches Wg rows, the odd one Wu rows, so
// g and u of the same output columns land in one accumulator row and the epilogue writes all three.  Otherwise two
// products and the element-wise kernel.
template <typename T>
int mm_swiglu(int64_t M, int64_t N, int64_t K, const T *A, int64_t lda, const T *Wg, const T *Wu, int64_t ldb, T *g, T *u,
              T *m, int64_t ldc, cudaStream_t st);

// ---- schedulers (T = storage dtype) --------------------------------------------------
// wgrad_group: consecutive chunks whose weight-gradient products are summed in one pass (1 = every chunk)
template <typename T>
size_t layer_workspace(const streambp_layer_cfg &c, int64_t T_, int64_t chunk, int wgrad_group = 1);
template <typename T>
int layer_backward(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, const T *dY, int64_t T_,
                   int64_t chunk, int64_t pos0, bool accumulate, const streambp_layer_grads &g, T *dX, void *ws,
                   cudaStream_t st, const int64_t *cu_seqlens = nullptr, int n_seqs = 0, int wgrad_group = 1);
// Y = layer(X), chunked; uses the same workspace plan as layer_backward.
template <typename T>
// cu_seqlens (host, n_seqs + 1 entries, 0 ... T): sequence boundaries of a packed batch, or nullptr.
int layer_forward(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, int64_t T_, int64_t chunk,
                  int64_t pos0, T *Y, void *ws, cudaStream_t st, const int64_t *cu_seqlens = nullptr, int n_seqs = 0);

template <typename T>
size_t lmhead_workspace(const streambp_head_cfg &c, int64_t T_, int64_t chunk, int wgrad_group = 1);
// rl == nullptr: SFT cross-entropy (labels = targets); else the RL objective described by *rl (labels = the
// sampled tokens, rl->logp_* etc. indexed by absolute row), `ell` optional (DPO).  wgrad_group >= 1: the vocabulary
// weight gradient is formed once per group of that many chunks.
template <typename T>
int lmhead_backward(const streambp_head_cfg &c, const T *g_final, const T *w_vocab, const T *H, const int64_t *labels,
                    int64_t T_, int64_t chunk, bool accumulate, float *loss, int64_t *n_valid, T *dH, float *d_w_vocab,
                    float *d_g_final, void *ws, cudaStream_t st, const RlRows *rl = nullptr, float *ell = nullptr,
                    int wgrad_group = 1);

template <typename T>
size_t model_workspace(const streambp_model_cfg &c, int64_t T_, int64_t chunk_layer, int64_t chunk_head);
template <typename T>
int model_backward(const streambp_model_cfg &c, const T *embed, const streambp_layer_weights *layers, const T *g_final,
                   const T *w_vocab, const int64_t *ids, const T *X0, const int64_t *labels, int64_t T_,
                   int64_t chunk_layer, int64_t chunk_head, bool accumulate, float *loss, float *d_embed,
                   const streambp_layer_grads *layer_grads, float *d_g_final, float *d_w_vocab, T *dX0, void *ws,
                   cudaStream_t st);

}  // namespace sbp
