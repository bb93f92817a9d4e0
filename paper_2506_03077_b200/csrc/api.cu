// extern "C" boundary: argument validation, dtype dispatch, status handling.
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <vector>

#include <cstdio>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace sbp {

NvtxRange::NvtxRange(const char *name) { nvtxRangePushA(name); }
NvtxRange::NvtxRange(const char *name, long long index) {
    char buf[64];
    std::snprintf(buf, sizeof(buf), "%s %lld", name, index);
    nvtxRangePushA(buf);
}
NvtxRange::~NvtxRange() { nvtxRangePop(); }

CallState &call_state() {
    static thread_local CallState s;
    return s;
}

namespace {
std::atomic<int> g_device_override{-1};

struct ProfRec {
    cudaEvent_t a, b;
    int cls;
    double flops;
};
bool g_prof_on = false;
std::vector<ProfRec> g_prof;      // event pairs, reused across resets
size_t g_prof_used = 0;
}  // namespace

ProfScope::ProfScope(int cls, double flops, cudaStream_t stream) : idx(-1), st(stream) {
    if (!g_prof_on) return;
    if (g_prof_used == g_prof.size()) {
        ProfRec r;
        if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
        g_prof.push_back(r);
    }
    idx = (int)g_prof_used++;
    g_prof[idx].cls = cls;
    g_prof[idx].flops = flops;
    cudaEventRecord(g_prof[idx].a, st);
}
ProfScope::~ProfScope() {
    if (idx >= 0) cudaEventRecord(g_prof[idx].b, st);
}

bool pdl_enabled() {
    static const bool on = [] {
        const char *e = getenv("STREAMBP_PDL");      // on unless set to 0
        return !e || atoi(e) != 0;
    }();
    return on;
}

int gemm_engine() {
    static const int engine = [] {
        const char *e = std::getenv("STREAMBP_GEMM_ENGINE");
        if (e && !std::strcmp(e, "simt")) return 1;
        if (e && !std::strcmp(e, "tc")) return 2;
        return 0;
    }();
    return engine;
}

bool ws_guard_enabled() {
    static const bool on = std::getenv("STREAMBP_WS_GUARD") != nullptr;
    return on;
}

int current_device_ordinal() {
    const int fake = g_device_override.load();
    if (fake >= 0) return fake;
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess ? dev : -1;
}

template <typename TI, typename TC>
int mm(GemmOp op, int64_t M, int64_t N, int64_t K, const TI *A, int64_t lda, const TI *B, int64_t ldb, TC *C,
       int64_t ldc, const TI *bias, bool accumulate, cudaStream_t st) {
    ProfScope prof(KC_GEMM, 2.0 * (double)M * (double)N * (double)K, st);
    return gemm<TI, TC>(op, M, N, K, A, lda, B, ldb, C, ldc, bias, accumulate, st);
}
template <>
int mm<bf16, float>(GemmOp op, int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *B, int64_t ldb,
                    float *C, int64_t ldc, const bf16 *bias, bool accumulate, cudaStream_t st) {
    ProfScope prof(KC_GEMM, 2.0 * (double)M * (double)N * (double)K, st);
    const int e = gemm_engine();
    if (e != 1 && gemm_tc_supported(op, M, N, K, lda, ldb, ldc, A, B, C, true))
        return gemm_tc(op, M, N, K, A, lda, B, ldb, C, ldc, true, bias, accumulate, st);
    if (e == 2) return STREAMBP_E_SHAPE;
    return gemm<bf16, float>(op, M, N, K, A, lda, B, ldb, C, ldc, bias, accumulate, st);
}
template <>
int mm<bf16, bf16>(GemmOp op, int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *B, int64_t ldb,
                   bf16 *C, int64_t ldc, const bf16 *bias, bool accumulate, cudaStream_t st) {
    ProfScope prof(KC_GEMM, 2.0 * (double)M * (double)N * (double)K, st);
    const int e = gemm_engine();
    if (e != 1 && !accumulate && gemm_tc_supported(op, M, N, K, lda, ldb, ldc, A, B, C, false))
        return gemm_tc(op, M, N, K, A, lda, B, ldb, C, ldc, false, bias, false, st);
    if (e == 2) return STREAMBP_E_SHAPE;
    return gemm<bf16, bf16>(op, M, N, K, A, lda, B, ldb, C, ldc, bias, accumulate, st);
}
template <>
int mm_group<float>(const MmProb<float> *probs, int n, cudaStream_t st);
template <>
int mm_group<bf16>(const MmProb<bf16> *probs, int n, cudaStream_t st);
// Products whose output is to be rotated, without the fused epilogue: the product goes to the fp32 scratch the
// caller named, a row kernel rotates it into C.
template <typename T>
static int mm_group_rope_unfused(const MmProb<T> *probs, int n, cudaStream_t st) {
    if (n > 4) return STREAMBP_E_SHAPE;
    MmProb<T> plain[4];
    for (int i = 0; i < n; i++) {
        plain[i] = probs[i];
        if (!probs[i].rope) continue;
        if (!probs[i].rope_tmp || probs[i].ldc != probs[i].N || probs[i].accumulate ||
            probs[i].N != (int64_t)probs[i].rope_heads * probs[i].rope_dh)
            return STREAMBP_E_SHAPE;
        plain[i].rope = nullptr;
        plain[i].C = probs[i].rope_tmp;
        plain[i].c_is_f32 = true;
    }
    SBP_TRY(mm_group<T>(plain, n, st));
    for (int i = 0; i < n; i++)
        if (probs[i].rope)
            SBP_TRY(rope_apply<T>(probs[i].rope_tmp, probs[i].rope, probs[i].M, probs[i].rope_heads, probs[i].rope_dh,
                                  false, (T *)probs[i].C, st));
    return STREAMBP_OK;
}
template <>
int mm_group<float>(const MmProb<float> *probs, int n, cudaStream_t st) {
    for (int i = 0; i < n; i++)
        if (probs[i].rope) return mm_group_rope_unfused<float>(probs, n, st);
    for (int i = 0; i < n; i++) {
        const MmProb<float> &g = probs[i];
        for (int s = 0; s < g.nseg; s++)
            SBP_TRY((mm<float, float>(g.op, g.M, g.N, g.seg[s].K, g.seg[s].A, g.seg[s].lda, g.seg[s].B, g.seg[s].ldb,
                                      (float *)g.C, g.ldc, s == 0 ? g.bias : nullptr, g.accumulate || s > 0, st)));
    }
    return STREAMBP_OK;
}
template <>
int mm_group<bf16>(const MmProb<bf16> *probs, int n, cudaStream_t st) {
    GemmProb gp[4];
    bool grouped = gemm_engine() != 1 && n <= 4;
    bool any_rope = false;
    for (int i = 0; i < n; i++) {
        any_rope = any_rope || probs[i].rope != nullptr;
        // the fused rotation handles heads of 128 columns written as bf16
        if (probs[i].rope && (probs[i].rope_dh != 128 || probs[i].c_is_f32 ||
                              probs[i].N != (int64_t)probs[i].rope_heads * probs[i].rope_dh))
            grouped = false;
    }
    if (grouped) {
        for (int i = 0; i < n; i++) {
            const MmProb<bf16> &g = probs[i];
            gp[i].rope = g.rope;
            gp[i].op = g.op; gp[i].M = g.M; gp[i].N = g.N; gp[i].nseg = g.nseg;
            for (int s = 0; s < g.nseg; s++) gp[i].seg[s] = GemmSeg{g.seg[s].A, g.seg[s].lda, g.seg[s].B, g.seg[s].ldb, g.seg[s].K};
            gp[i].C = g.C; gp[i].ldc = g.ldc; gp[i].c_is_f32 = g.c_is_f32; gp[i].bias = g.bias; gp[i].accumulate = g.accumulate;
        }
        grouped = gemm_tc_group_supported(gp, n);
    }
    if (grouped) {
        double flops = 0.0;
        for (int i = 0; i < n; i++)
            for (int s = 0; s < probs[i].nseg; s++) flops += 2.0 * (double)probs[i].M * (double)probs[i].N * (double)probs[i].seg[s].K;
        ProfScope prof(KC_GEMM, flops, st);
        CallState &cs = call_state();
        int *sched = cs.sched ? cs.sched + 2 * (cs.sched_slot++ % kSchedSlots) : nullptr;
        return gemm_tc_group(gp, n, sched, st);
    }
    if (any_rope) return mm_group_rope_unfused<bf16>(probs, n, st);
    for (int i = 0; i < n; i++) {
        const MmProb<bf16> &g = probs[i];
        // a bf16 output cannot be accumulated into: several segments need an fp32 C
        if (!g.c_is_f32 && g.nseg > 1) return STREAMBP_E_SHAPE;
        for (int s = 0; s < g.nseg; s++) {
            const bf16 *b = s == 0 ? g.bias : nullptr;
            const bool acc = g.accumulate || s > 0;
            if (g.c_is_f32)
                SBP_TRY((mm<bf16, float>(g.op, g.M, g.N, g.seg[s].K, g.seg[s].A, g.seg[s].lda, g.seg[s].B, g.seg[s].ldb,
                                         (float *)g.C, g.ldc, b, acc, st)));
            else
                SBP_TRY((mm<bf16, bf16>(g.op, g.M, g.N, g.seg[s].K, g.seg[s].A, g.seg[s].lda, g.seg[s].B, g.seg[s].ldb,
                                        (bf16 *)g.C, g.ldc, b, acc, st)));
        }
    }
    return STREAMBP_OK;
}

template <typename T>
static int mm_swiglu_unfused(int64_t M, int64_t N, int64_t K, const T *A, int64_t lda, const T *Wg, const T *Wu, int64_t ldb,
                             T *g, T *u, T *m, int64_t ldc, cudaStream_t st) {
    if (ldc != N) return STREAMBP_E_SHAPE;      // the element-wise kernel walks dense [M, N] buffers
    const MmProb<T> gu[2] = {mm_prob<T>(OP_NT, M, N, K, A, lda, Wg, ldb, g, ldc, sizeof(T) == 4, nullptr, false),
                             mm_prob<T>(OP_NT, M, N, K, A, lda, Wu, ldb, u, ldc, sizeof(T) == 4, nullptr, false)};
    SBP_TRY(mm_group<T>(gu, 2, st));
    return swiglu_fwd<T>(g, u, M * N, m, st);
}
template <>
int mm_swiglu<float>(int64_t M, int64_t N, int64_t K, const float *A, int64_t lda, const float *Wg, const float *Wu,
                     int64_t ldb, float *g, float *u, float *m, int64_t ldc, cudaStream_t st) {
    return mm_swiglu_unfused<float>(M, N, K, A, lda, Wg, Wu, ldb, g, u, m, ldc, st);
}
template <>
int mm_swiglu<bf16>(int64_t M, int64_t N, int64_t K, const bf16 *A, int64_t lda, const bf16 *Wg, const bf16 *Wu,
                    int64_t ldb, bf16 *g, bf16 *u, bf16 *m, int64_t ldc, cudaStream_t st) {
    GemmProb gp;
    gp.op = OP_NT; gp.M = M; gp.N = N; gp.nseg = 2;
    gp.seg[0] = GemmSeg{A, lda, Wg, ldb, K};
    gp.seg[1] = GemmSeg{A, lda, Wu, ldb, K};
    gp.C = g; gp.ldc = ldc; gp.c_is_f32 = false; gp.bias = nullptr; gp.accumulate = false;
    gp.swiglu = true; gp.C_up = u; gp.C_act = m;
    if (gemm_engine() != 1 && gemm_tc_group_supported(&gp, 1)) {
        ProfScope prof(KC_GEMM, 2.0 * 2.0 * (double)M * (double)N * (double)K, st);
        CallState &cs = call_state();
        int *sched = cs.sched ? cs.sched + 2 * (cs.sched_slot++ % kSchedSlots) : nullptr;
        return gemm_tc_group(&gp, 1, sched, st);
    }
    return mm_swiglu_unfused<bf16>(M, N, K, A, lda, Wg, Wu, ldb, g, u, m, ldc, st);
}

template <>
int attn_fwd<float>(const float *q, const float *k, const float *v, int64_t n, int64_t q0, int Hq, int Hkv, int dh,
                    float *o, float *lse, cudaStream_t st) {
    return attention_fwd<float>(q, k, v, n, q0, Hq, Hkv, dh, o, lse, st);
}
template <>
int attn_fwd<bf16>(const bf16 *q, const bf16 *k, const bf16 *v, int64_t n, int64_t q0, int Hq, int Hkv, int dh,
                   bf16 *o, float *lse, cudaStream_t st) {
    const int e = gemm_engine();
    if (e != 1 && attention_tc_supported(n, q0, Hq, Hkv, dh, q, k, v))
        return attention_fwd_tc(q, k, v, n, q0, Hq, Hkv, o, lse, st);
    if (e == 2) return STREAMBP_E_SHAPE;
    return attention_fwd<bf16>(q, k, v, n, q0, Hq, Hkv, dh, o, lse, st);
}
template <>
int attn_bwd<float>(const float *q, const float *k, const float *v, const float *o, const float *dout,
                    const float *lse, int64_t n, int64_t q0, int Hq, int Hkv, int dh, float *delta, float *dq,
                    float *dk, float *dv, cudaStream_t st, int) {
    return attention_bwd<float>(q, k, v, o, dout, lse, n, q0, Hq, Hkv, dh, delta, dq, dk, dv, st);
}
template <>
int attn_bwd<bf16>(const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *o, const bf16 *dout, const float *lse,
                   int64_t n, int64_t q0, int Hq, int Hkv, int dh, float *delta, float *dq, float *dk, float *dv,
                   cudaStream_t st, int engine) {
    static const bool five_default = [] {
        const char *v = std::getenv("STREAMBP_ATTN_BWD");
        return v && !std::strcmp(v, "five");
    }();
    const int e = engine < 0 ? gemm_engine() : engine;
    if (e != 1 && attention_tc_supported(n, q0, Hq, Hkv, dh, q, k, v)) {
        SBP_TRY(attention_delta<bf16>(o, dout, n, Hq, dh, delta, st));
        return attention_bwd_tc(q, k, v, dout, lse, delta, n, q0, Hq, Hkv, dq, dk, dv, st,
                                e == 5 || (engine < 0 && five_default));
    }
    if (e == 2 || e == 5) return STREAMBP_E_SHAPE;
    return attention_bwd<bf16>(q, k, v, o, dout, lse, n, q0, Hq, Hkv, dh, delta, dq, dk, dv, st);
}

template int mm<float, float>(GemmOp, int64_t, int64_t, int64_t, const float *, int64_t, const float *, int64_t,
                              float *, int64_t, const float *, bool, cudaStream_t);

namespace {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_layer_cfg(const streambp_layer_cfg *c) {
    if (!c) return STREAMBP_E_NULL;
    if (c->dtype != STREAMBP_F32 && c->dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (c->d_model < 8 || c->d_model % 8) return STREAMBP_E_SHAPE;
    if (c->head_dim != 64 && c->head_dim != 128) return STREAMBP_E_SHAPE;
    if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return STREAMBP_E_SHAPE;
    if (c->d_ff < 8 || c->d_ff % 8) return STREAMBP_E_SHAPE;
    if (!(c->rope_theta > 0.f) || !(c->rms_eps >= 0.f)) return STREAMBP_E_SHAPE;
    return STREAMBP_OK;
}
int check_head_cfg(const streambp_head_cfg *c) {
    if (!c) return STREAMBP_E_NULL;
    if (c->dtype != STREAMBP_F32 && c->dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (c->d_model < 8 || c->d_model % 8) return STREAMBP_E_SHAPE;
    if (c->vocab < 1) return STREAMBP_E_SHAPE;
    if (!(c->rms_eps >= 0.f)) return STREAMBP_E_SHAPE;
    return STREAMBP_OK;
}
int check_layer_weights(const streambp_layer_cfg *c, const streambp_layer_weights *w) {
    if (!w) return STREAMBP_E_NULL;
    const void *req[] = {w->g1, w->wq, w->wk, w->wv, w->wo, w->g2, w->w_gate, w->w_up, w->w_down};
    for (const void *p : req) {
        if (!p) return STREAMBP_E_NULL;
        if (!aligned(p, 16)) return STREAMBP_E_ALIGN;
    }
    if (c->qkv_bias) {
        const void *b[] = {w->bq, w->bk, w->bv};
        for (const void *p : b) {
            if (!p) return STREAMBP_E_NULL;
            if (!aligned(p, 16)) return STREAMBP_E_ALIGN;
        }
    }
    return STREAMBP_OK;
}
int check_layer_grads(const streambp_layer_cfg *c, const streambp_layer_grads *g) {
    if (!g) return STREAMBP_E_NULL;
    float *req[] = {g->g1, g->wq, g->wk, g->wv, g->wo, g->g2, g->w_gate, g->w_up, g->w_down};
    for (float *p : req) {
        if (!p) return STREAMBP_E_NULL;
        if (!aligned(p, 16)) return STREAMBP_E_ALIGN;
    }
    if (c->qkv_bias) {
        float *b[] = {g->bq, g->bk, g->bv};
        for (float *p : b) {
            if (!p) return STREAMBP_E_NULL;
            if (!aligned(p, 16)) return STREAMBP_E_ALIGN;
        }
    }
    return STREAMBP_OK;
}
// weights with the bias pointers dropped when the configuration has no bias
streambp_layer_weights effective(const streambp_layer_cfg *c, const streambp_layer_weights *w) {
    streambp_layer_weights e = *w;
    if (!c->qkv_bias) e.bq = e.bk = e.bv = nullptr;
    return e;
}
}  // namespace

// Alignment the attention backward needs of its arguments (16-byte vector accesses and TMA tiles on the tensors,
// 4 bytes on the per-row vectors); `delta` may be nullptr where the caller does not pass one.
bool attention_bwd_aligned(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                           const void *lse, const void *delta, const void *dq, const void *dk, const void *dv) {
    const void *t16[] = {q, k, v, o, d_o, dq, dk, dv};
    for (const void *p : t16)
        if (!aligned(p, 16)) return false;
    return aligned(lse, 4) && (delta == nullptr || aligned(delta, 4));
}

namespace {
int begin_call(void *ws, cudaStream_t st) {
    call_state().cuda_error = 0;
    call_state().launches = 0;
    call_state().sched = nullptr;
    call_state().sched_slot = 0;
    return fill_zero(ws, kHeaderBytes, st);
}

}  // namespace
}  // namespace sbp

using namespace sbp;

namespace {
// largest chunk in {128, 256, ..., } U {T} with bytes(chunk) <= budget; bytes() is non-decreasing in chunk
template <typename F>
int64_t suggest_chunk(int64_t T, size_t budget, F bytes) {
    if (T < 1) return 0;
    const size_t full = bytes(T);
    if (full == 0) return 0;
    if (full <= budget) return T;
    int64_t lo = 0, hi = (T - 1) / 128;          // chunk = 128 * k for k in [1, hi] is < T
    while (lo < hi) {
        const int64_t mid = (lo + hi + 1) / 2;
        if (bytes(128 * mid) <= budget) lo = mid;
        else hi = mid - 1;
    }
    return 128 * lo;
}
}  // namespace

extern "C" {

size_t streambp_layer_workspace_bytes_grouped(const streambp_layer_cfg *cfg, int64_t T, int64_t chunk,
                                              int32_t wgrad_group) {
    if (check_layer_cfg(cfg) != STREAMBP_OK || T < 1 || chunk < 1 || wgrad_group < 1) return 0;
    return cfg->dtype == STREAMBP_F32 ? layer_workspace<float>(*cfg, T, chunk, wgrad_group)
                                      : layer_workspace<bf16>(*cfg, T, chunk, wgrad_group);
}

size_t streambp_layer_workspace_bytes(const streambp_layer_cfg *cfg, int64_t T, int64_t chunk) {
    return streambp_layer_workspace_bytes_grouped(cfg, T, chunk, 1);
}

static int layer_backward_checked(const streambp_layer_cfg *cfg, const streambp_layer_weights *w, const void *X,
                                  const void *dY, int64_t T, int64_t chunk, const int64_t *cu_seqlens, int n_seqs,
                                  int64_t pos0, int accumulate, const streambp_layer_grads *grads, void *dX,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream, int wgrad_group = 1) {
    SBP_TRY(check_layer_cfg(cfg));
    if (T < 1 || chunk < 1 || pos0 < 0 || wgrad_group < 1) return STREAMBP_E_SHAPE;
    SBP_TRY(check_layer_weights(cfg, w));
    SBP_TRY(check_layer_grads(cfg, grads));
    if (!X || !dY || !dX || !workspace) return STREAMBP_E_NULL;
    if (!aligned(X, 16) || !aligned(dY, 16) || !aligned(dX, 16) || !aligned(workspace, 256)) return STREAMBP_E_ALIGN;
    if (dX == X || dX == dY) return STREAMBP_E_SHAPE;
    if (cu_seqlens) {
        if (n_seqs < 1 || cu_seqlens[0] != 0 || cu_seqlens[n_seqs] != T) return STREAMBP_E_SHAPE;
        for (int i = 0; i < n_seqs; i++)
            if (cu_seqlens[i + 1] <= cu_seqlens[i]) return STREAMBP_E_SHAPE;
    }
    if (workspace_bytes < streambp_layer_workspace_bytes_grouped(cfg, T, chunk, wgrad_group)) return STREAMBP_E_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SBP_TRY(begin_call(workspace, st));
    const streambp_layer_weights we = effective(cfg, w);
    if (cfg->dtype == STREAMBP_F32)
        return layer_backward<float>(*cfg, we, (const float *)X, (const float *)dY, T, chunk, pos0, accumulate != 0,
                                     *grads, (float *)dX, workspace, st, cu_seqlens, n_seqs, wgrad_group);
    return layer_backward<bf16>(*cfg, we, (const bf16 *)X, (const bf16 *)dY, T, chunk, pos0, accumulate != 0, *grads,
                                (bf16 *)dX, workspace, st, cu_seqlens, n_seqs, wgrad_group);
}

int streambp_layer_backward_grouped(const streambp_layer_cfg *cfg, const streambp_layer_weights *w, const void *X,
                                    const void *dY, int64_t T, int64_t chunk, int32_t wgrad_group,
                                    const int64_t *cu_seqlens, int32_t n_seqs, int64_t pos0, int accumulate,
                                    const streambp_layer_grads *grads, void *dX, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream) {
    return layer_backward_checked(cfg, w, X, dY, T, chunk, cu_seqlens, cu_seqlens ? n_seqs : 0, pos0, accumulate, grads,
                                  dX, workspace, workspace_bytes, cuda_stream, wgrad_group);
}

int streambp_layer_backward(const streambp_layer_cfg *cfg, const streambp_layer_weights *w, const void *X,
                            const void *dY, int64_t T, int64_t chunk, int64_t pos0, int accumulate,
                            const streambp_layer_grads *grads, void *dX, void *workspace, size_t workspace_bytes,
                            void *cuda_stream) {
    return layer_backward_checked(cfg, w, X, dY, T, chunk, nullptr, 0, pos0, accumulate, grads, dX, workspace,
                                  workspace_bytes, cuda_stream);
}

int streambp_layer_backward_packed(const streambp_layer_cfg *cfg, const streambp_layer_weights *w, const void *X,
                                   const void *dY, int64_t T, int64_t chunk, const int64_t *cu_seqlens, int32_t n_seqs,
                                   int64_t pos0, int accumulate, const streambp_layer_grads *grads, void *dX,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!cu_seqlens) return STREAMBP_E_NULL;
    return layer_backward_checked(cfg, w, X, dY, T, chunk, cu_seqlens, n_seqs, pos0, accumulate, grads, dX, workspace,
                                  workspace_bytes, cuda_stream);
}

size_t streambp_lmhead_workspace_bytes_grouped(const streambp_head_cfg *cfg, int64_t T, int64_t chunk,
                                               int32_t wgrad_group) {
    if (check_head_cfg(cfg) != STREAMBP_OK || T < 1 || chunk < 1 || wgrad_group < 1) return 0;
    return cfg->dtype == STREAMBP_F32 ? lmhead_workspace<float>(*cfg, T, chunk, wgrad_group)
                                      : lmhead_workspace<bf16>(*cfg, T, chunk, wgrad_group);
}

size_t streambp_lmhead_workspace_bytes(const streambp_head_cfg *cfg, int64_t T, int64_t chunk) {
    return streambp_lmhead_workspace_bytes_grouped(cfg, T, chunk, 1);
}

int streambp_lmhead_ce_backward_grouped(const streambp_head_cfg *cfg, const void *g_final, const void *w_vocab,
                                        const void *H, const int64_t *labels, int64_t T, int64_t chunk,
                                        int32_t wgrad_group, int accumulate, float *loss, int64_t *n_valid, void *dH,
                                        float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream) {
    SBP_TRY(check_head_cfg(cfg));
    if (T < 1 || chunk < 1 || wgrad_group < 1) return STREAMBP_E_SHAPE;
    if (!g_final || !w_vocab || !H || !labels || !loss || !dH || !d_w_vocab || !d_g_final || !workspace)
        return STREAMBP_E_NULL;
    if (!aligned(g_final, 16) || !aligned(w_vocab, 16) || !aligned(H, 16) || !aligned(dH, 16) ||
        !aligned(d_w_vocab, 16) || !aligned(d_g_final, 16) || !aligned(labels, 8) || !aligned(workspace, 256))
        return STREAMBP_E_ALIGN;
    if (workspace_bytes < streambp_lmhead_workspace_bytes_grouped(cfg, T, chunk, wgrad_group))
        return STREAMBP_E_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SBP_TRY(begin_call(workspace, st));
    if (cfg->dtype == STREAMBP_F32)
        return lmhead_backward<float>(*cfg, (const float *)g_final, (const float *)w_vocab, (const float *)H, labels, T,
                                      chunk, accumulate != 0, loss, n_valid, (float *)dH, d_w_vocab, d_g_final,
                                      workspace, st, nullptr, nullptr, wgrad_group);
    return lmhead_backward<bf16>(*cfg, (const bf16 *)g_final, (const bf16 *)w_vocab, (const bf16 *)H, labels, T, chunk,
                                 accumulate != 0, loss, n_valid, (bf16 *)dH, d_w_vocab, d_g_final, workspace, st,
                                 nullptr, nullptr, wgrad_group);
}

int streambp_lmhead_ce_backward(const streambp_head_cfg *cfg, const void *g_final, const void *w_vocab, const void *H,
                                const int64_t *labels, int64_t T, int64_t chunk, int accumulate, float *loss,
                                int64_t *n_valid, void *dH, float *d_w_vocab, float *d_g_final, void *workspace,
                                size_t workspace_bytes, void *cuda_stream) {
    return streambp_lmhead_ce_backward_grouped(cfg, g_final, w_vocab, H, labels, T, chunk, 1, accumulate, loss, n_valid,
                                               dH, d_w_vocab, d_g_final, workspace, workspace_bytes, cuda_stream);
}

int streambp_lmhead_rl_backward_grouped(const streambp_head_cfg *cfg, const streambp_rl_cfg *rl, const void *g_final,
                                        const void *w_vocab, const void *H, const int64_t *tokens,
                                        const float *logp_old, const float *logp_ref, const float *advantage,
                                        const float *weight, int64_t T, int64_t chunk, int32_t wgrad_group,
                                        int accumulate, float *loss, float *logp, float *ell, void *dH,
                                        float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream) {
    SBP_TRY(check_head_cfg(cfg));
    if (!rl) return STREAMBP_E_NULL;
    if (rl->objective != STREAMBP_OBJ_GRPO && rl->objective != STREAMBP_OBJ_DPO) return STREAMBP_E_SHAPE;
    if (T < 1 || chunk < 1 || wgrad_group < 1 || !(rl->beta >= 0.f)) return STREAMBP_E_SHAPE;
    if (rl->objective == STREAMBP_OBJ_GRPO && !(rl->clip_eps >= 0.f && rl->clip_eps < 1.f)) return STREAMBP_E_SHAPE;
    if (rl->objective == STREAMBP_OBJ_DPO && accumulate) return STREAMBP_E_SHAPE;   // in-place correction at the end
    if (!g_final || !w_vocab || !H || !tokens || !logp_ref || !weight || !loss || !dH || !d_w_vocab || !d_g_final ||
        !workspace)
        return STREAMBP_E_NULL;
    if (rl->objective == STREAMBP_OBJ_GRPO && (!logp_old || !advantage)) return STREAMBP_E_NULL;
    if (!aligned(g_final, 16) || !aligned(w_vocab, 16) || !aligned(H, 16) || !aligned(dH, 16) ||
        !aligned(d_w_vocab, 16) || !aligned(d_g_final, 16) || !aligned(tokens, 8) || !aligned(workspace, 256))
        return STREAMBP_E_ALIGN;
    if (workspace_bytes < streambp_lmhead_workspace_bytes_grouped(cfg, T, chunk, wgrad_group))
        return STREAMBP_E_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SBP_TRY(begin_call(workspace, st));
    const RlRows rows{rl->objective, rl->beta, rl->clip_eps, logp_old, logp_ref, advantage, weight, logp};
    if (cfg->dtype == STREAMBP_F32)
        return lmhead_backward<float>(*cfg, (const float *)g_final, (const float *)w_vocab, (const float *)H, tokens, T,
                                      chunk, accumulate != 0, loss, nullptr, (float *)dH, d_w_vocab, d_g_final,
                                      workspace, st, &rows, ell, wgrad_group);
    return lmhead_backward<bf16>(*cfg, (const bf16 *)g_final, (const bf16 *)w_vocab, (const bf16 *)H, tokens, T, chunk,
                                 accumulate != 0, loss, nullptr, (bf16 *)dH, d_w_vocab, d_g_final, workspace, st, &rows,
                                 ell, wgrad_group);
}

int streambp_lmhead_rl_backward(const streambp_head_cfg *cfg, const streambp_rl_cfg *rl, const void *g_final,
                                const void *w_vocab, const void *H, const int64_t *tokens, const float *logp_old,
                                const float *logp_ref, const float *advantage, const float *weight, int64_t T,
                                int64_t chunk, int accumulate, float *loss, float *logp, float *ell, void *dH,
                                float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                void *cuda_stream) {
    return streambp_lmhead_rl_backward_grouped(cfg, rl, g_final, w_vocab, H, tokens, logp_old, logp_ref, advantage,
                                               weight, T, chunk, 1, accumulate, loss, logp, ell, dH, d_w_vocab,
                                               d_g_final, workspace, workspace_bytes, cuda_stream);
}

static int check_model_cfg(const streambp_model_cfg *cfg) {
    if (!cfg) return STREAMBP_E_NULL;
    SBP_TRY(check_layer_cfg(&cfg->layer));
    SBP_TRY(check_head_cfg(&cfg->head));
    if (cfg->n_layers < 1) return STREAMBP_E_SHAPE;
    if (cfg->layer.dtype != cfg->head.dtype) return STREAMBP_E_DTYPE;
    if (cfg->layer.d_model != cfg->head.d_model) return STREAMBP_E_SHAPE;
    return STREAMBP_OK;
}

size_t streambp_model_workspace_bytes(const streambp_model_cfg *cfg, int64_t T, int64_t chunk_layer,
                                      int64_t chunk_head) {
    if (check_model_cfg(cfg) != STREAMBP_OK || T < 1 || chunk_layer < 1 || chunk_head < 1) return 0;
    return cfg->layer.dtype == STREAMBP_F32 ? model_workspace<float>(*cfg, T, chunk_layer, chunk_head)
                                            : model_workspace<bf16>(*cfg, T, chunk_layer, chunk_head);
}

int streambp_model_backward(const streambp_model_cfg *cfg, const void *embed, const streambp_layer_weights *layers,
                            const void *g_final, const void *w_vocab, const int64_t *ids, const void *X0,
                            const int64_t *labels, int64_t T, int64_t chunk_layer, int64_t chunk_head, int accumulate,
                            float *loss, float *d_embed, const streambp_layer_grads *layer_grads, float *d_g_final,
                            float *d_w_vocab, void *dX0, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    SBP_TRY(check_model_cfg(cfg));
    if (T < 1 || chunk_layer < 1 || chunk_head < 1) return STREAMBP_E_SHAPE;
    if (!layers || !layer_grads || !g_final || !w_vocab || !labels || !loss || !d_g_final || !d_w_vocab || !workspace)
        return STREAMBP_E_NULL;
    if (ids ? !embed : !X0) return STREAMBP_E_NULL;
    if (!aligned(g_final, 16) || !aligned(w_vocab, 16) || !aligned(d_g_final, 16) || !aligned(d_w_vocab, 16) ||
        !aligned(workspace, 256) || (embed && !aligned(embed, 16)) || (X0 && !aligned(X0, 16)) ||
        (dX0 && !aligned(dX0, 16)) || (d_embed && !aligned(d_embed, 16)))
        return STREAMBP_E_ALIGN;
    std::vector<streambp_layer_weights> eff(cfg->n_layers);
    for (int l = 0; l < cfg->n_layers; l++) {
        SBP_TRY(check_layer_weights(&cfg->layer, &layers[l]));
        SBP_TRY(check_layer_grads(&cfg->layer, &layer_grads[l]));
        eff[l] = effective(&cfg->layer, &layers[l]);
    }
    if (workspace_bytes < streambp_model_workspace_bytes(cfg, T, chunk_layer, chunk_head)) return STREAMBP_E_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    SBP_TRY(begin_call(workspace, st));
    if (cfg->layer.dtype == STREAMBP_F32)
        return model_backward<float>(*cfg, (const float *)embed, eff.data(), (const float *)g_final,
                                     (const float *)w_vocab, ids, (const float *)X0, labels, T, chunk_layer, chunk_head,
                                     accumulate != 0, loss, d_embed, layer_grads, d_g_final, d_w_vocab, (float *)dX0,
                                     workspace, st);
    return model_backward<bf16>(*cfg, (const bf16 *)embed, eff.data(), (const bf16 *)g_final, (const bf16 *)w_vocab,
                                ids, (const bf16 *)X0, labels, T, chunk_layer, chunk_head, accumulate != 0, loss,
                                d_embed, layer_grads, d_g_final, d_w_vocab, (bf16 *)dX0, workspace, st);
}

int64_t streambp_layer_suggest_chunk(const streambp_layer_cfg *cfg, int64_t T, size_t budget_bytes) {
    if (check_layer_cfg(cfg) != STREAMBP_OK) return 0;
    return suggest_chunk(T, budget_bytes, [&](int64_t c) { return streambp_layer_workspace_bytes(cfg, T, c); });
}

int64_t streambp_lmhead_suggest_chunk(const streambp_head_cfg *cfg, int64_t T, size_t budget_bytes) {
    if (check_head_cfg(cfg) != STREAMBP_OK) return 0;
    return suggest_chunk(T, budget_bytes, [&](int64_t c) { return streambp_lmhead_workspace_bytes(cfg, T, c); });
}

int streambp_last_device_status(void *workspace, void *cuda_stream) {
    if (!workspace) return STREAMBP_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    WsHeader h;
    if (!cuda_ok(cudaMemcpyAsync(&h, workspace, sizeof(h), cudaMemcpyDeviceToHost, st))) return STREAMBP_E_CUDA;
    if (!cuda_ok(cudaStreamSynchronize(st))) return STREAMBP_E_CUDA;
    const int f1 = gemm_tc_take_fault(), f2 = attention_tc_take_fault(), f3 = wait_probe_take_fault();
    if (f1 < 0 || f2 < 0 || f3 < 0) return STREAMBP_E_CUDA;
    if (f1 > 0 || f2 > 0 || f3 > 0) return STREAMBP_E_DEVICE_TIMEOUT;
    return h.status;
}

const char *streambp_status_string(int s) {
    switch (s) {
        case STREAMBP_OK: return "ok";
        case STREAMBP_E_NULL: return "a required pointer is NULL";
        case STREAMBP_E_SHAPE: return "unsupported or inconsistent sizes";
        case STREAMBP_E_ALIGN: return "pointer not sufficiently aligned";
        case STREAMBP_E_WORKSPACE: return "workspace too small";
        case STREAMBP_E_DTYPE: return "unknown dtype";
        case STREAMBP_E_CUDA: return "CUDA call failed";
        case STREAMBP_E_BAD_LABEL: return "label or token id out of range";
        case STREAMBP_E_NO_VALID_LABELS: return "no unmasked label";
        case STREAMBP_E_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case STREAMBP_E_WORKSPACE_GUARD: return "a kernel wrote past a workspace sub-buffer (guard overwritten)";
        default: return "unknown status";
    }
}

int streambp_last_cuda_error(void) { return call_state().cuda_error; }
int64_t streambp_last_launch_count(void) { return call_state().launches; }

int streambp_attention_forward(const void *q, const void *k, const void *v, int64_t n, int64_t q0, int32_t n_q_heads,
                               int32_t n_kv_heads, int32_t head_dim, int32_t dtype, void *o, float *lse, int engine,
                               void *cuda_stream) {
    if (!q || !k || !v || !o || !lse) return STREAMBP_E_NULL;
    if (n < 1 || q0 < 0 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
        (head_dim != 64 && head_dim != 128))
        return STREAMBP_E_SHAPE;
    // the kernels use 16-byte vector accesses and TMA tiles on every tensor: refused here, never faulted on the device
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(o, 16) || !aligned(lse, 4))
        return STREAMBP_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    call_state().cuda_error = 0;
    call_state().launches = 0;
    if (dtype == STREAMBP_F32) {
        if (engine >= 2) return STREAMBP_E_DTYPE;
        return attention_fwd<float>((const float *)q, (const float *)k, (const float *)v, n, q0, n_q_heads, n_kv_heads,
                                    head_dim, (float *)o, lse, st);
    }
    if (dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    const bool tc_ok = attention_tc_supported(n, q0, n_q_heads, n_kv_heads, head_dim, q, k, v);
    if (engine >= 2 && !tc_ok) return STREAMBP_E_SHAPE;
    if (engine != 1 && tc_ok)
        return attention_fwd_tc((const bf16 *)q, (const bf16 *)k, (const bf16 *)v, n, q0, n_q_heads, n_kv_heads,
                                (bf16 *)o, lse, st, engine == 3 ? 1 : (engine == 4 ? 2 : 0));
    return attention_fwd<bf16>((const bf16 *)q, (const bf16 *)k, (const bf16 *)v, n, q0, n_q_heads, n_kv_heads,
                               head_dim, (bf16 *)o, lse, st);
}

int streambp_attention_backward(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                const float *lse, int64_t n, int64_t q0, int32_t n_q_heads, int32_t n_kv_heads,
                                int32_t head_dim, int32_t dtype, float *delta, float *dq, float *dk, float *dv,
                                int engine, void *cuda_stream) {
    if (!q || !k || !v || !o || !d_o || !lse || !delta || !dq || !dk || !dv) return STREAMBP_E_NULL;
    if (n < 1 || q0 < 0 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads ||
        (head_dim != 64 && head_dim != 128))
        return STREAMBP_E_SHAPE;
    if (!attention_bwd_aligned(q, k, v, o, d_o, lse, delta, dq, dk, dv)) return STREAMBP_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    call_state().cuda_error = 0;
    call_state().launches = 0;
    if (dtype == STREAMBP_F32) {
        if (engine == 2 || engine == 5) return STREAMBP_E_DTYPE;
        return attention_bwd<float>((const float *)q, (const float *)k, (const float *)v, (const float *)o,
                                    (const float *)d_o, lse, n, q0, n_q_heads, n_kv_heads, head_dim, delta, dq, dk, dv,
                                    st);
    }
    if (dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (engine < 0 || (engine > 2 && engine != 5)) return STREAMBP_E_SHAPE;
    return attn_bwd<bf16>((const bf16 *)q, (const bf16 *)k, (const bf16 *)v, (const bf16 *)o, (const bf16 *)d_o, lse, n,
                          q0, n_q_heads, n_kv_heads, head_dim, delta, dq, dk, dv, st, engine);
}

int streambp_product_kernel(void) { return gemm_tc_variant(); }

int streambp_test_expire_wait(uint64_t limit_ns, void *cuda_stream) {
    if (limit_ns < 1000 || limit_ns > 100000000ull) return STREAMBP_E_SHAPE;     // 1 us .. 100 ms
    call_state().cuda_error = 0;
    call_state().launches = 0;
    return wait_probe_launch(limit_ns, static_cast<cudaStream_t>(cuda_stream));
}

int streambp_test_workspace_guard(void *workspace, size_t workspace_bytes, int32_t overrun, void *cuda_stream) {
    if (!workspace) return STREAMBP_E_NULL;
    if (!aligned(workspace, 256)) return STREAMBP_E_ALIGN;
    if (overrun < 0 || overrun > 64) return STREAMBP_E_SHAPE;
    call_state().cuda_error = 0;
    call_state().launches = 0;
    return ws_guard_selftest(workspace, workspace_bytes, overrun, static_cast<cudaStream_t>(cuda_stream));
}

int streambp_test_per_device_value(int ordinal, int value) {
    static PerDevice cache;
    if (ordinal < 0) return STREAMBP_E_SHAPE;
    g_device_override.store(ordinal);
    const int got = cache.get([&] { return value; });
    g_device_override.store(-1);
    return got;
}

void streambp_profile_enable(int on) {
    g_prof_on = on != 0;
    g_prof_used = 0;
}

int streambp_profile_read(int kernel_class, double *milliseconds, int64_t *calls, double *flops) {
    if (kernel_class < 0 || kernel_class >= KC_CLASSES) return STREAMBP_E_SHAPE;
    double ms = 0.0, fl = 0.0;
    int64_t n = 0;
    for (size_t i = 0; i < g_prof_used; i++) {
        if (g_prof[i].cls != kernel_class) continue;
        if (!cuda_ok(cudaEventSynchronize(g_prof[i].b))) return STREAMBP_E_CUDA;
        float t = 0.f;
        if (!cuda_ok(cudaEventElapsedTime(&t, g_prof[i].a, g_prof[i].b))) return STREAMBP_E_CUDA;
        ms += t;
        fl += g_prof[i].flops;
        n++;
    }
    if (milliseconds) *milliseconds = ms;
    if (calls) *calls = n;
    if (flops) *flops = fl;
    return STREAMBP_OK;
}

int streambp_gemm(int op, int64_t M, int64_t N, int64_t K, const void *A, int64_t lda, const void *B, int64_t ldb,
                  void *C, int64_t ldc, int32_t in_dtype, int32_t out_dtype, int accumulate, int engine,
                  void *cuda_stream) {
    if (op < 0 || op > 2 || M < 1 || N < 1 || K < 1) return STREAMBP_E_SHAPE;
    if (!A || !B || !C) return STREAMBP_E_NULL;
    if (!aligned(A, 16) || !aligned(B, 16) || !aligned(C, 16)) return STREAMBP_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    call_state().cuda_error = 0;
    call_state().launches = 0;
    const GemmOp g = static_cast<GemmOp>(op);
    const bool acc = accumulate != 0;
    if (in_dtype == STREAMBP_F32) {
        if (out_dtype != STREAMBP_F32 || engine == 2) return STREAMBP_E_DTYPE;
        return gemm<float, float>(g, M, N, K, (const float *)A, lda, (const float *)B, ldb, (float *)C, ldc, nullptr,
                                  acc, st);
    }
    if (in_dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    const bool c32 = out_dtype == STREAMBP_F32;
    if (!c32 && out_dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (!c32 && acc) return STREAMBP_E_DTYPE;
    const bool tc_ok = gemm_tc_supported(g, M, N, K, lda, ldb, ldc, A, B, C, c32);
    if (engine == 2 && !tc_ok) return STREAMBP_E_SHAPE;
    if (engine != 1 && tc_ok)
        return gemm_tc(g, M, N, K, (const bf16 *)A, lda, (const bf16 *)B, ldb, C, ldc, c32, nullptr, acc, st);
    if (c32)
        return gemm<bf16, float>(g, M, N, K, (const bf16 *)A, lda, (const bf16 *)B, ldb, (float *)C, ldc, nullptr, acc,
                                 st);
    return gemm<bf16, bf16>(g, M, N, K, (const bf16 *)A, lda, (const bf16 *)B, ldb, (bf16 *)C, ldc, nullptr, false, st);
}

int streambp_gemm_grouped(const streambp_gemm_problem *problems, int32_t n, int32_t *sched, void *cuda_stream) {
    if (!problems) return STREAMBP_E_NULL;
    if (n < 1 || n > 4) return STREAMBP_E_SHAPE;
    if (sched && !aligned(sched, 8)) return STREAMBP_E_ALIGN;
    GemmProb gp[4];
    for (int i = 0; i < n; i++) {
        const streambp_gemm_problem &q = problems[i];
        if (q.op < 0 || q.op > 2 || q.n_segments < 1 || q.n_segments > 3 || q.M < 1 || q.N < 1) return STREAMBP_E_SHAPE;
        if (q.out_dtype != STREAMBP_F32 && q.out_dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
        if (q.out_dtype == STREAMBP_BF16 && q.accumulate) return STREAMBP_E_DTYPE;
        if (!q.C) return STREAMBP_E_NULL;
        gp[i].op = static_cast<GemmOp>(q.op);
        gp[i].M = q.M;
        gp[i].N = q.N;
        gp[i].nseg = q.n_segments;
        for (int s = 0; s < q.n_segments; s++) {
            if (!q.A[s] || !q.B[s]) return STREAMBP_E_NULL;
            if (q.K[s] < 1) return STREAMBP_E_SHAPE;
            gp[i].seg[s] = GemmSeg{(const bf16 *)q.A[s], q.lda[s], (const bf16 *)q.B[s], q.ldb[s], q.K[s]};
        }
        gp[i].C = q.C;
        gp[i].ldc = q.ldc;
        gp[i].c_is_f32 = q.out_dtype == STREAMBP_F32;
        gp[i].bias = nullptr;
        gp[i].accumulate = q.accumulate != 0;
    }
    call_state().cuda_error = 0;
    call_state().launches = 0;
    if (!gemm_tc_group_supported(gp, n)) return STREAMBP_E_SHAPE;
    return gemm_tc_group(gp, n, sched, static_cast<cudaStream_t>(cuda_stream));
}

int streambp_gemm_swiglu(const void *A, int64_t lda, const void *w_gate, const void *w_up, int64_t ldb, int64_t M,
                         int64_t N, int64_t K, void *g, void *u, void *m, int32_t dtype, void *cuda_stream) {
    if (!A || !w_gate || !w_up || !g || !u || !m) return STREAMBP_E_NULL;
    if (M < 1 || N < 1 || K < 1 || lda < K || ldb < K) return STREAMBP_E_SHAPE;
    if (dtype != STREAMBP_F32 && dtype != STREAMBP_BF16) return STREAMBP_E_DTYPE;
    if (!aligned(A, 16) || !aligned(w_gate, 16) || !aligned(w_up, 16) || !aligned(g, 16) || !aligned(u, 16) || !aligned(m, 16))
        return STREAMBP_E_ALIGN;
    call_state().cuda_error = 0;
    call_state().launches = 0;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (dtype == STREAMBP_F32)
        return mm_swiglu<float>(M, N, K, (const float *)A, lda, (const float *)w_gate, (const float *)w_up, ldb, (float *)g,
                                (float *)u, (float *)m, N, st);
    return mm_swiglu<bf16>(M, N, K, (const bf16 *)A, lda, (const bf16 *)w_gate, (const bf16 *)w_up, ldb, (bf16 *)g, (bf16 *)u,
                           (bf16 *)m, N, st);
}

}  // extern "C"
