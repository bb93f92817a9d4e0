// Host-side scheduler of the streamed final-norm + LM-head + cross-entropy backward
// (Sec. 3.2.1: logits are formed, used and dropped one sequence chunk at a time).
#include "common.cuh"

namespace sbp {

namespace {
template <typename T>
struct HeadWs {
    WsHeader *hdr;
    T *hn, *dz;
    float *z, *dhn, *rstd, *row_loss, *partials;
    int *chunk_valid;     // [number of chunks] unmasked labels per chunk: the device-side gate of each chunk
    int *group_valid;     // [number of groups] the same per weight-gradient group
    int slots;            // chunks per weight-gradient group
    size_t bytes;
    std::vector<size_t> guards;   // debug mode: offsets of the guards behind the sub-buffers
};

// `wg` >= 1: chunks per weight-gradient group (a second partition size, as in the layer): dW_vocab += dZ^T hn is formed
// once per group over all its rows, so hn and dlogits exist once per chunk of a group, contiguous in row order.
template <typename T>
HeadWs<T> plan(const streambp_head_cfg &c, int64_t T_, int64_t chunk, void *base, int wg = 1) {
    const int64_t cn = chunk < T_ ? chunk : T_;
    const int64_t d = c.d_model, V = c.vocab;
    const int64_t D = (T_ + cn - 1) / cn;
    const int64_t slots = wg < 1 ? 1 : (wg > D ? D : wg);
    const int64_t gr = slots * cn;
    Arena a(base);
    HeadWs<T> w;
    w.slots = (int)slots;
    w.hdr = reinterpret_cast<WsHeader *>(a.take_bytes(kHeaderBytes));
    w.hn = a.take<T>(gr * d);
    // fp32 storage: dlogits overwrite the logits in place (then the logits exist once per chunk of a group too)
    w.z = a.take<float>((sizeof(T) == 4 ? gr : cn) * V);
    w.dz = sizeof(T) == 4 ? reinterpret_cast<T *>(w.z) : a.take<T>(gr * V);
    w.dhn = a.take<float>(cn * d);
    w.rstd = a.take<float>(cn);
    w.row_loss = a.take<float>(cn);
    w.partials = a.take<float>(64 * d);
    w.chunk_valid = a.take<int>(D);
    w.group_valid = a.take<int>((D + slots - 1) / slots);
    w.bytes = a.size();
    w.guards = a.guards;
    return w;
}
}  // namespace

template <typename T>
size_t lmhead_workspace(const streambp_head_cfg &c, int64_t T_, int64_t chunk, int wgrad_group) {
    return plan<T>(c, T_, chunk, nullptr, wgrad_group).bytes;
}

template <typename T>
int lmhead_backward(const streambp_head_cfg &c, const T *g_final, const T *w_vocab, const T *H, const int64_t *labels,
                    int64_t T_, int64_t chunk, bool accumulate, float *loss, int64_t *n_valid, T *dH, float *d_w_vocab,
                    float *d_g_final, void *ws, cudaStream_t st, const RlRows *rl, float *ell, int wgrad_group) {
    const NvtxRange call_range(rl ? "streambp lm-head RL backward" : "streambp lm-head CE backward");
    const int64_t cn = chunk < T_ ? chunk : T_;
    HeadWs<T> s = plan<T>(c, T_, chunk, ws, wgrad_group);
    const SchedScope sched(s.hdr);
    const int d = c.d_model;
    const int64_t V = c.vocab;
    SBP_TRY(ws_guards_arm(ws, s.guards, st));
    // N is global: it is counted before the chunk loop so that every chunk scales by the same 1/N
    SBP_TRY(count_valid_labels(labels, T_, V, c.ignore_index, s.hdr, st));
    SBP_TRY(count_valid_per_chunk(labels, T_, cn, c.ignore_index, s.chunk_valid, st));
    const int64_t k = s.slots;
    if (k > 1) SBP_TRY(count_valid_per_chunk(labels, T_, k * cn, c.ignore_index, s.group_valid, st));
    if (!accumulate) {
        // chunks whose labels are all ignored are skipped on the device (their dlogits are exactly zero),
        // so no particular chunk can be relied on to overwrite the outputs: clear them and always add
        SBP_TRY(fill_zero(d_g_final, sizeof(float) * d, st));
        SBP_TRY(fill_zero(d_w_vocab, sizeof(float) * (size_t)V * d, st));
    }
    // rows of skipped chunks keep this zero
    if (rl && rl->logp_out) SBP_TRY(fill_zero(rl->logp_out, sizeof(float) * T_, st));
    const int64_t D = (T_ + cn - 1) / cn;
    struct GateScope {      // every launch of a chunk is gated by that chunk's count of unmasked labels
        explicit GateScope(const int *g) { call_state().gate = g; }
        ~GateScope() { call_state().gate = nullptr; }
    };
    for (int64_t i = 0; i < D; i++) {
        const NvtxRange chunk_range("chunk", i);
        // groups of k consecutive chunks; the group's weight-gradient product runs with its last chunk
        const int64_t g_lo = (i / k) * k, g_hi = g_lo + k - 1 < D - 1 ? g_lo + k - 1 : D - 1;
        const bool group_done = i == g_hi;
        const int64_t r0 = i * cn, gr0 = g_lo * cn, off = r0 - gr0;
        const int64_t n = (T_ - r0 < cn) ? T_ - r0 : cn;
        const int64_t gn = ((g_hi + 1) * cn < T_ ? (g_hi + 1) * cn : T_) - gr0;
        const bool acc = true;
        const T *Hi = H + r0 * d;
        // every launch is gated on the device by a count of unmasked labels: the chunk's own, or with groups the
        // group's (a masked chunk inside a live group is then processed like masked rows inside a live chunk: zero
        // dlogits, so it adds nothing anywhere)
        GateScope gate(k > 1 ? s.group_valid + i / k : s.chunk_valid + i);
        T *hn = s.hn + off * d, *dz = s.dz + off * V;
        float *z = sizeof(T) == 4 ? s.z + off * V : s.z;
        SBP_TRY(rmsnorm_fwd<T>(Hi, nullptr, g_final, c.rms_eps, n, d, hn, s.rstd, nullptr, st));
        SBP_TRY((mm<T, float>(OP_NT, n, V, d, hn, d, w_vocab, d, z, V, nullptr, false, st)));           // logits
        if (rl)
            SBP_TRY(rl_rows<T>(z, labels + r0, n, V, c.ignore_index, *rl, r0, dz, s.row_loss, st));
        else
            SBP_TRY(ce_rows<T>(z, labels + r0, n, V, c.ignore_index, s.hdr, dz, s.row_loss, st));
        SBP_TRY(loss_accumulate(s.row_loss, n, s.hdr, st));
        {   // dhn = dZ W needs only this chunk's dZ; dW += dZ^T hn runs over the group's rows, in the same launch, when
            // the group is complete (the few long dhn tiles first)
            const MmProb<T> pr[2] = {mm_prob<T>(OP_TN, V, d, gn, s.dz, V, s.hn, d, d_w_vocab, d, true, nullptr, acc),
                                     mm_prob<T>(OP_NN, n, d, V, dz, V, w_vocab, d, s.dhn, d, true, nullptr, false)};
            if (group_done) SBP_TRY(mm_group<T>(pr, 2, st));
            else SBP_TRY(mm_group<T>(pr + 1, 1, st));
        }
        SBP_TRY(rmsnorm_bwd<T>(s.dhn, Hi, nullptr, s.rstd, g_final, nullptr, nullptr, n, d, nullptr, dH + r0 * d,
                               d_g_final, s.partials, st));
    }
    if (!rl) {
        SBP_TRY(loss_finalize(s.hdr, loss, n_valid, st));
        return ws_guards_check(ws, s.guards, s.hdr, st);
    }
    SBP_TRY(rl_finalize(s.hdr, rl->objective, rl->beta, loss, ell, st));
    if (rl->objective == STREAMBP_OBJ_DPO) {
        // the running sums hold beta * sum_t d ell(t); the exact gradient is (sigmoid(beta ell) - 1) times that
        SBP_TRY(scale_by_factor<float>(d_w_vocab, V * d, s.hdr, st));
        SBP_TRY(scale_by_factor<float>(d_g_final, d, s.hdr, st));
        SBP_TRY(scale_by_factor<T>(dH, T_ * d, s.hdr, st));
    }
    return ws_guards_check(ws, s.guards, s.hdr, st);
}

template size_t lmhead_workspace<float>(const streambp_head_cfg &, int64_t, int64_t, int);
template size_t lmhead_workspace<bf16>(const streambp_head_cfg &, int64_t, int64_t, int);
template int lmhead_backward<float>(const streambp_head_cfg &, const float *, const float *, const float *,
                                    const int64_t *, int64_t, int64_t, bool, float *, int64_t *, float *, float *,
                                    float *, void *, cudaStream_t, const RlRows *, float *, int);
template int lmhead_backward<bf16>(const streambp_head_cfg &, const bf16 *, const bf16 *, const bf16 *,
                                   const int64_t *, int64_t, int64_t, bool, float *, int64_t *, bf16 *, float *,
                                   float *, void *, cudaStream_t, const RlRows *, float *, int);

}  // namespace sbp
