// Host-side chunk scheduler of one decoder layer: the partitioned re-forward and the accumulation
// of the paper's Sec. 3.2.2, as a fixed sequence of kernel launches on the caller's stream.
//
// K and V (rotated) are produced once for all T rows and cached; chunks are then processed from
// the LAST to the first.  The order does not change the sum (any order of the terms of Eq. (1) is
// exact); running backwards makes the fp32 dK/dV rows of chunk i final as soon as chunk i itself
// has been processed (only chunks >= i attend to them), so the K/V-projection backward of chunk i
// runs inside the same iteration, on the h1 rows that are already resident.
#include <vector>

#include "common.cuh"

namespace sbp {

namespace {

// Sequence boundaries of a packed batch: rows [b[i], b[i+1]) form sequence i.  A single sequence [0, T)
// when the caller passes none.  Only the attention and the rotary positions see the boundaries: every
// other step of the layer is row-wise.
struct Segments {
    std::vector<int64_t> b;
    Segments(const int64_t *cu, int n, int64_t T_) {
        if (cu && n > 0) b.assign(cu, cu + n + 1);
        else b = {0, T_};
    }
    // calls f(a, e, s) for every maximal run of rows [a, e) inside [r0, r1) that lies in one sequence (start s)
    template <typename F> int for_each(int64_t r0, int64_t r1, F f) const {
        for (size_t i = 0; i + 1 < b.size(); i++) {
            const int64_t a = b[i] > r0 ? b[i] : r0, e = b[i + 1] < r1 ? b[i + 1] : r1;
            if (a < e) SBP_TRY(f(a, e, b[i]));
        }
        return STREAMBP_OK;
    }
};

template <typename T>
struct LayerWs {
    WsHeader *hdr;
    float *cs;            // [T, dh/2] (cos, sin)
    T *K, *V;             // [T, dkv]
    float *dK, *dV;       // [T, dkv]
    // one chunk
    T *h1, *Q, *O, *h2, *g, *u, *m, *dr_s, *dO, *dk_s, *dv_s, *dm;
    float *fa, *r, *dr, *rstd1, *rstd2, *lse, *delta, *partials;
    size_t bytes;
    int slots;            // chunks per weight-gradient group
    std::vector<size_t> guards;   // debug mode: offsets of the guards behind the sub-buffers
};

// `wg` >= 1 is the number of consecutive chunks whose weight-gradient products are summed in ONE pass over the
// fp32 accumulators (a second partition size: K = wg * chunk for those products).  The operands of those products
// -- h1, dq (in Q's place), O, h2, dg, du (in g's and u's place), m, dr and dk, dv in storage type -- then exist once
// per chunk of a group ("slots", contiguous in row order, so a group's operand is one matrix of wg * chunk rows).
template <typename T>
LayerWs<T> plan(const streambp_layer_cfg &c, int64_t T_, int64_t chunk, void *base, int wg = 1) {
    const int64_t cn = chunk < T_ ? chunk : T_;
    const int64_t d = c.d_model, dq = (int64_t)c.n_q_heads * c.head_dim, dkv = (int64_t)c.n_kv_heads * c.head_dim;
    const int64_t I = c.d_ff, wide = dq > d ? dq : d;
    const int64_t D = (T_ + cn - 1) / cn;
    const int64_t slots = wg < 1 ? 1 : (wg > D ? D : wg);
    const int64_t gr = slots * cn;          // rows of a group's operand buffers
    Arena a(base);
    LayerWs<T> w;
    w.slots = (int)slots;
    w.hdr = reinterpret_cast<WsHeader *>(a.take_bytes(kHeaderBytes));
    w.cs = a.take<float>(T_ * c.head_dim);
    w.K = a.take<T>(T_ * dkv);
    w.V = a.take<T>(T_ * dkv);
    w.dK = a.take<float>(T_ * dkv);
    w.dV = a.take<float>(T_ * dkv);
    w.h1 = a.take<T>(gr * d);
    w.Q = a.take<T>(gr * dq);
    w.O = a.take<T>(gr * dq);
    w.h2 = a.take<T>(gr * d);
    w.g = a.take<T>(gr * I);
    w.u = a.take<T>(gr * I);
    w.m = a.take<T>(gr * I);
    if (slots > 1) {
        // group operands first (they outlive their chunk), then the buffers of the chunk in flight
        w.dr_s = a.take<T>(gr * d);
        w.dk_s = a.take<T>(gr * dkv);
        w.dv_s = a.take<T>(gr * dkv);
        w.dO = a.take<T>(cn * dq);
        w.fa = a.take<float>(cn * wide);
        w.dr = a.take<float>(sizeof(T) == 4 ? gr * d : cn * d);   // fp32 storage: dr itself is the product operand
        w.dm = a.take<T>(cn * I);
    } else {
        const size_t dead_begin = align_up(a.off, 256);
        w.dr_s = a.take<T>(cn * d);
        w.dO = a.take<T>(cn * dq);
        w.dk_s = a.take<T>(cn * dkv);
        w.dv_s = a.take<T>(cn * dkv);
        w.fa = a.take<float>(cn * wide);
        w.dr = a.take<float>(cn * d);
        // dm = dY Wd lives only from its product to the SwiGLU backward, while dr_s, dO, dk_s, dv_s, fa and dr are all
        // dead: it is laid over that span when it fits (it does for every LLM-shaped layer), else it gets its own block
        // (not in the guarded debug mode: the overlay would run over the guards of the buffers it covers)
        if (!a.guarded && a.off - dead_begin >= (size_t)(cn * I) * sizeof(T))
            w.dm = a.base ? reinterpret_cast<T *>(a.base + dead_begin) : nullptr;
        else
            w.dm = a.take<T>(cn * I);
    }
    w.r = a.take<float>(cn * d);
    w.rstd1 = a.take<float>(cn);
    w.rstd2 = a.take<float>(cn);
    w.lse = a.take<float>(cn * c.n_q_heads);
    w.delta = a.take<float>(cn * c.n_q_heads);
    // reduction partials: up to 64 row splits of the widest row reduced -- a gain gradient (d) or, with biases, the
    // three bias column sums of a chunk or group side by side (dq + 2 dkv)
    const int64_t bias_cols = c.qkv_bias ? dq + 2 * dkv : 0;
    w.partials = a.take<float>(64 * (bias_cols > wide ? bias_cols : wide));
    w.bytes = a.size();
    w.guards = a.guards;
    return w;
}

// The same plan with the group-operand pointers moved to the slot of the chunk that starts `row_off` rows into
// its group.
template <typename T>
LayerWs<T> at_slot(const LayerWs<T> &w, const streambp_layer_cfg &c, int64_t row_off) {
    if (row_off == 0 || w.h1 == nullptr) return w;
    const int64_t d = c.d_model, dq = (int64_t)c.n_q_heads * c.head_dim, dkv = (int64_t)c.n_kv_heads * c.head_dim;
    const int64_t I = c.d_ff;
    LayerWs<T> s = w;
    s.h1 += row_off * d; s.Q += row_off * dq; s.O += row_off * dq; s.h2 += row_off * d;
    s.g += row_off * I; s.u += row_off * I; s.m += row_off * I;
    s.dr_s += row_off * d; s.dk_s += row_off * dkv; s.dv_s += row_off * dkv;
    if (sizeof(T) == 4) s.dr += row_off * d;
    return s;
}

// K/V for all rows, chunk by chunk: h1 = RMSNorm1(X), K = RoPE(h1 Wk^T + bk), V = h1 Wv^T + bv
template <typename T>
int kv_prologue(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, int64_t T_, int64_t cn,
                int64_t pos0, const Segments &seg, LayerWs<T> &s, cudaStream_t st) {
    const int d = c.d_model, dh = c.head_dim, Hkv = c.n_kv_heads;
    const int64_t dkv = (int64_t)Hkv * dh;
    // rotary positions restart at every sequence of a packed batch
    SBP_TRY(seg.for_each(0, T_, [&](int64_t a, int64_t e, int64_t) {
        return rope_table(s.cs + a * dh, pos0, e - a, dh, c.rope_theta, st);
    }));
    for (int64_t r0 = 0; r0 < T_; r0 += cn) {
        const int64_t n = (T_ - r0 < cn) ? T_ - r0 : cn;
        SBP_TRY(rmsnorm_fwd<T>(X + r0 * d, nullptr, (const T *)w.g1, c.rms_eps, n, d, s.h1, s.rstd1, nullptr, st));
        // K = rotate(h1 Wk^T + bk) (the rotation in the product's epilogue where the kernel has it), V = h1 Wv^T + bv
        MmProb<T> kv[2] = {
            mm_prob<T>(OP_NT, n, dkv, d, s.h1, d, (const T *)w.wk, d, s.K + r0 * dkv, dkv, sizeof(T) == 4,
                       (const T *)w.bk, false),
            mm_prob<T>(OP_NT, n, dkv, d, s.h1, d, (const T *)w.wv, d, s.V + r0 * dkv, dkv, sizeof(T) == 4,
                       (const T *)w.bv, false)};
        mm_set_rope<T>(kv[0], s.cs + r0 * dh, Hkv, dh, s.fa);
        SBP_TRY(mm_group<T>(kv, 2, st));
    }
    return STREAMBP_OK;
}

// Re-forward of one chunk up to m = silu(g) * u. Leaves h1, rstd1, Q, O, lse, r, h2, rstd2, g, u, m.
template <typename T>
int chunk_forward(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, int64_t r0, int64_t n,
                  const Segments &seg, LayerWs<T> &s, cudaStream_t st) {
    const int d = c.d_model, dh = c.head_dim, Hq = c.n_q_heads, Hkv = c.n_kv_heads;
    const int64_t dq = (int64_t)Hq * dh, I = c.d_ff;
    const T *Xi = X + r0 * d;
    SBP_TRY(rmsnorm_fwd<T>(Xi, nullptr, (const T *)w.g1, c.rms_eps, n, d, s.h1, s.rstd1, nullptr, st));
    {   // Q = rotate(h1 Wq^T + bq)
        MmProb<T> qp = mm_prob<T>(OP_NT, n, dq, d, s.h1, d, (const T *)w.wq, d, s.Q, dq, sizeof(T) == 4,
                                  (const T *)w.bq, false);
        mm_set_rope<T>(qp, s.cs + r0 * dh, Hq, dh, s.fa);
        SBP_TRY(mm_group<T>(&qp, 1, st));
    }
    // the chunk's queries against the key / value prefix of their own sequence, one call per sequence the
    // chunk touches (a = first row, e = end row, q_seq = start of that sequence)
    SBP_TRY(seg.for_each(r0, r0 + n, [&](int64_t a, int64_t e, int64_t q_seq) {
        const int64_t m = e - a, off = a - r0, dkv = (int64_t)Hkv * dh;
        // causal pairs (query, key): m * (a - q_seq) + m (m + 1) / 2; two products forward
        const double pairs = (double)m * (double)(a - q_seq) + 0.5 * (double)m * (double)(m + 1);
        ProfScope prof(KC_ATTN_FWD, 2.0 * 2.0 * pairs * dh * Hq, st);
        return attn_fwd<T>(s.Q + off * dq, s.K + q_seq * dkv, s.V + q_seq * dkv, m, a - q_seq, Hq, Hkv, dh,
                           s.O + off * dq, s.lse + off * Hq, st);
    }));
    SBP_TRY((mm<T, float>(OP_NT, n, d, dq, s.O, dq, (const T *)w.wo, dq, s.fa, d, nullptr, false, st)));
    SBP_TRY(rmsnorm_fwd<T>(Xi, s.fa, (const T *)w.g2, c.rms_eps, n, d, s.h2, s.rstd2, s.r, st));
    SBP_TRY(mm_swiglu<T>(n, I, d, s.h2, d, (const T *)w.w_gate, (const T *)w.w_up, d, s.g, s.u, s.m, I, st));
    return STREAMBP_OK;
}

}  // namespace

template <typename T>
size_t layer_workspace(const streambp_layer_cfg &c, int64_t T_, int64_t chunk, int wgrad_group) {
    return plan<T>(c, T_, chunk, nullptr, wgrad_group).bytes;
}

template <typename T>
int layer_forward(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, int64_t T_, int64_t chunk,
                  int64_t pos0, T *Y, void *ws, cudaStream_t st, const int64_t *cu_seqlens, int n_seqs) {
    const Segments seg(cu_seqlens, n_seqs, T_);
    const int64_t cn = chunk < T_ ? chunk : T_;
    LayerWs<T> s = plan<T>(c, T_, chunk, ws);
    const SchedScope sched(s.hdr);
    const int d = c.d_model;
    const int64_t I = c.d_ff;
    SBP_TRY(ws_guards_arm(ws, s.guards, st));
    SBP_TRY(kv_prologue<T>(c, w, X, T_, cn, pos0, seg, s, st));
    for (int64_t r0 = 0; r0 < T_; r0 += cn) {
        const int64_t n = (T_ - r0 < cn) ? T_ - r0 : cn;
        SBP_TRY(chunk_forward<T>(c, w, X, r0, n, seg, s, st));
        SBP_TRY((mm<T, float>(OP_NT, n, d, I, s.m, I, (const T *)w.w_down, I, s.fa, d, nullptr, false, st)));
        SBP_TRY(add_cast<T>(s.r, s.fa, n * d, Y + r0 * d, st));
    }
    return ws_guards_check(ws, s.guards, s.hdr, st);
}

template <typename T>
int layer_backward(const streambp_layer_cfg &c, const streambp_layer_weights &w, const T *X, const T *dY, int64_t T_,
                   int64_t chunk, int64_t pos0, bool accumulate, const streambp_layer_grads &G, T *dX, void *ws,
                   cudaStream_t st, const int64_t *cu_seqlens, int n_seqs, int wgrad_group) {
    const NvtxRange call_range("streambp layer backward");
    const Segments seg(cu_seqlens, n_seqs, T_);
    const int64_t cn = chunk < T_ ? chunk : T_;
    LayerWs<T> base = plan<T>(c, T_, chunk, ws, wgrad_group);
    const SchedScope sched(base.hdr);
    const int d = c.d_model, dh = c.head_dim, Hq = c.n_q_heads, Hkv = c.n_kv_heads;
    const int64_t dq = (int64_t)Hq * dh, dkv = (int64_t)Hkv * dh, I = c.d_ff;
    constexpr bool kF32 = sizeof(T) == 4;

    SBP_TRY(ws_guards_arm(ws, base.guards, st));
    {
        const NvtxRange r("K/V prologue");
        SBP_TRY(kv_prologue<T>(c, w, X, T_, cn, pos0, seg, base, st));
    }
    SBP_TRY(fill_zero(base.dK, sizeof(float) * T_ * dkv, st));
    SBP_TRY(fill_zero(base.dV, sizeof(float) * T_ * dkv, st));
    if (!accumulate) {  // vectors are always added to; matrices are overwritten by the first group's product
        SBP_TRY(fill_zero(G.g1, sizeof(float) * d, st));
        SBP_TRY(fill_zero(G.g2, sizeof(float) * d, st));
        if (c.qkv_bias) {
            SBP_TRY(fill_zero(G.bq, sizeof(float) * dq, st));
            SBP_TRY(fill_zero(G.bk, sizeof(float) * dkv, st));
            SBP_TRY(fill_zero(G.bv, sizeof(float) * dkv, st));
        }
    }
    const int64_t D = (T_ + cn - 1) / cn;
    const int64_t k = base.slots;
    for (int64_t i = D - 1; i >= 0; i--) {
        // Chunks are grouped from the end: {D-1 .. D-k}, {D-k-1 .. D-2k}, ...  The weight-gradient products of a
        // group run once, when its first chunk (the last one processed) is done, over all the group's rows: the
        // operands of a group are contiguous in row order (X, dY in the caller's arrays, the rest in the slots).
        const NvtxRange chunk_range("chunk", i);
        const int64_t g_hi = D - 1 - ((D - 1 - i) / k) * k, g_lo = g_hi - k + 1 > 0 ? g_hi - k + 1 : 0;
        const bool group_done = i == g_lo;
        const int64_t r0 = i * cn, gr0 = g_lo * cn;
        const int64_t n = (T_ - r0 < cn) ? T_ - r0 : cn;
        const int64_t gn = ((g_hi + 1) * cn < T_ ? (g_hi + 1) * cn : T_) - gr0;      // rows of the group
        const bool acc = accumulate || g_hi != D - 1;
        const T *Xi = X + r0 * d, *dYi = dY + r0 * d, *dYg = dY + gr0 * d;
        LayerWs<T> s = at_slot<T>(base, c, r0 - gr0);
        {
            const NvtxRange r("re-forward");
            SBP_TRY(chunk_forward<T>(c, w, X, r0, n, seg, s, st));
        }
        const NvtxRange bwd_range("backward");

        // ---- MLP backward ----
        SBP_TRY((mm<T, T>(OP_NN, n, I, d, dYi, d, (const T *)w.w_down, I, s.dm, I, nullptr, false, st)));  // dm = dY Wd
        SBP_TRY(swiglu_bwd<T>(s.dm, s.g, s.u, n * I, st));                                            // g := dg, u := du
        {   // dh2 = dg Wg + du Wu, and with it (one launch) the group's dWd += dY^T m, dWg += dg^T h2, dWu += du^T h2:
            // the weight gradients are bound by the fp32 add into C at L2, the input gradient by the tensor pipe
            MmProb<T> pr[4];
            int np = 0;
            if (group_done) {
                pr[np++] = mm_prob<T>(OP_TN, d, I, gn, dYg, d, base.m, I, G.w_down, I, true, nullptr, acc);
                pr[np++] = mm_prob<T>(OP_TN, I, d, gn, base.g, I, base.h2, d, G.w_gate, d, true, nullptr, acc);
                pr[np++] = mm_prob<T>(OP_TN, I, d, gn, base.u, I, base.h2, d, G.w_up, d, true, nullptr, acc);
            }
            pr[np] = mm_prob<T>(OP_NN, n, d, I, s.g, I, (const T *)w.w_gate, d, s.fa, d, true, nullptr, false);
            mm_add_seg<T>(pr[np], I, s.u, I, (const T *)w.w_up, d);
            SBP_TRY(mm_group<T>(pr, np + 1, st));
        }
        // dr = dY + norm2_bwd(dh2)
        SBP_TRY(rmsnorm_bwd<T>(s.fa, nullptr, s.r, s.rstd2, (const T *)w.g2, dYi, nullptr, n, d, s.dr,
                               kF32 ? nullptr : s.dr_s, G.g2, s.partials, st));
        const T *dr_op = kF32 ? reinterpret_cast<const T *>(s.dr) : s.dr_s;
        const T *dr_grp = kF32 ? reinterpret_cast<const T *>(base.dr) : base.dr_s;

        // ---- attention output projection backward ----
        {   // dO = dr Wo, and the group's dWo += dr^T O
            MmProb<T> pr[2];
            int np = 0;
            if (group_done) pr[np++] = mm_prob<T>(OP_TN, d, dq, gn, dr_grp, d, base.O, dq, G.wo, dq, true, nullptr, acc);
            pr[np++] = mm_prob<T>(OP_NN, n, dq, d, dr_op, d, (const T *)w.wo, dq, s.dO, dq, sizeof(T) == 4, nullptr, false);
            SBP_TRY(mm_group<T>(pr, np, st));
        }

        // ---- partitioned attention backward: dQ (into fa), dK/dV prefix += ----
        SBP_TRY(seg.for_each(r0, r0 + n, [&](int64_t a, int64_t e, int64_t q_seq) {
            const int64_t m = e - a, off = a - r0;
            const double pairs = (double)m * (double)(a - q_seq) + 0.5 * (double)m * (double)(m + 1);
            ProfScope prof(KC_ATTN_BWD, 5.0 * 2.0 * pairs * dh * Hq, st);   // five products backward
            return attn_bwd<T>(s.Q + off * dq, s.K + q_seq * dkv, s.V + q_seq * dkv, s.O + off * dq, s.dO + off * dq,
                               s.lse + off * Hq, m, a - q_seq, Hq, Hkv, dh, s.delta + off * Hq, s.fa + off * dq,
                               s.dK + q_seq * dkv, s.dV + q_seq * dkv, st);
        }));

        // ---- Q, K, V projection backward (this chunk's dK/dV rows are final now) ----
        T *dq_s = s.Q;  // Q is dead after the attention backward
        SBP_TRY(rope_apply<T>(s.fa, s.cs + r0 * dh, n, Hq, dh, true, dq_s, st));
        SBP_TRY(rope_apply<T>(s.dK + r0 * dkv, s.cs + r0 * dh, n, Hkv, dh, true, s.dk_s, st));
        SBP_TRY(cast_from_f32<T>(s.dV + r0 * dkv, n * dkv, s.dv_s, st));
        {   // dh1 = dq Wq + dk Wk + dv Wv, and the group's dWq, dWk, dWv
            MmProb<T> pr[4];
            int np = 0;
            if (group_done) {
                pr[np++] = mm_prob<T>(OP_TN, dq, d, gn, base.Q, dq, base.h1, d, G.wq, d, true, nullptr, acc);
                pr[np++] = mm_prob<T>(OP_TN, dkv, d, gn, base.dk_s, dkv, base.h1, d, G.wk, d, true, nullptr, acc);
                pr[np++] = mm_prob<T>(OP_TN, dkv, d, gn, base.dv_s, dkv, base.h1, d, G.wv, d, true, nullptr, acc);
            }
            pr[np] = mm_prob<T>(OP_NN, n, d, dq, dq_s, dq, (const T *)w.wq, d, s.fa, d, true, nullptr, false);
            mm_add_seg<T>(pr[np], dkv, s.dk_s, dkv, (const T *)w.wk, d);
            mm_add_seg<T>(pr[np], dkv, s.dv_s, dkv, (const T *)w.wv, d);
            SBP_TRY(mm_group<T>(pr, np + 1, st));
        }
        if (c.qkv_bias && group_done)
            SBP_TRY(colsum3_add<T>(base.Q, (int)dq, G.bq, base.dk_s, (int)dkv, G.bk, base.dv_s, (int)dkv, G.bv, gn, s.partials, st));

        // ---- dX = dr + norm1_bwd(dh1) ----
        SBP_TRY(rmsnorm_bwd<T>(s.fa, Xi, nullptr, s.rstd1, (const T *)w.g1, nullptr, s.dr, n, d, nullptr, dX + r0 * d,
                               G.g1, s.partials, st));
    }
    return ws_guards_check(ws, base.guards, base.hdr, st);
}

template size_t layer_workspace<float>(const streambp_layer_cfg &, int64_t, int64_t, int);
template size_t layer_workspace<bf16>(const streambp_layer_cfg &, int64_t, int64_t, int);
template int layer_forward<float>(const streambp_layer_cfg &, const streambp_layer_weights &, const float *, int64_t,
                                  int64_t, int64_t, float *, void *, cudaStream_t, const int64_t *, int);
template int layer_forward<bf16>(const streambp_layer_cfg &, const streambp_layer_weights &, const bf16 *, int64_t,
                                 int64_t, int64_t, bf16 *, void *, cudaStream_t, const int64_t *, int);
template int layer_backward<float>(const streambp_layer_cfg &, const streambp_layer_weights &, const float *,
                                   const float *, int64_t, int64_t, int64_t, bool, const streambp_layer_grads &,
                                   float *, void *, cudaStream_t, const int64_t *, int, int);
template int layer_backward<bf16>(const streambp_layer_cfg &, const streambp_layer_weights &, const bf16 *,
                                  const bf16 *, int64_t, int64_t, int64_t, bool, const streambp_layer_grads &, bf16 *,
                                  void *, cudaStream_t, const int64_t *, int, int);

}  // namespace sbp
