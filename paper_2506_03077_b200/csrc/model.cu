// Whole-model backward on layer-input checkpoints: embedding lookup, a chunked forward that keeps only
// each layer's input, the streamed head backward, the streamed layer backward from the last layer to
// the first, and the embedding scatter-add.
#include "common.cuh"

namespace sbp {

namespace {
template <typename T>
struct ModelWs {
    WsHeader *hdr;
    T *ckpt;      // [L + 1][T, d]: inputs of layers 0..L-1, then the last layer's output
    T *ga, *gb;   // [T, d] ping-pong buffers for the gradient travelling down the stack
    void *sub;    // workspace shared (in turn) by the layer forward, the head and the layer backward
    size_t sub_bytes, bytes;
    std::vector<size_t> guards;   // debug mode: offsets of the guards behind the sub-buffers
};

template <typename T>
ModelWs<T> plan(const streambp_model_cfg &c, int64_t T_, int64_t chunk_layer, int64_t chunk_head, void *base) {
    Arena a(base);
    ModelWs<T> w;
    const int64_t d = c.layer.d_model;
    w.hdr = reinterpret_cast<WsHeader *>(a.take_bytes(kHeaderBytes));
    w.ckpt = a.take<T>((int64_t)(c.n_layers + 1) * T_ * d);
    w.ga = a.take<T>(T_ * d);
    w.gb = a.take<T>(T_ * d);
    const size_t lb = layer_workspace<T>(c.layer, T_, chunk_layer), hb = lmhead_workspace<T>(c.head, T_, chunk_head);
    w.sub_bytes = lb > hb ? lb : hb;
    w.sub = a.take_bytes(w.sub_bytes);
    w.bytes = a.size();
    w.guards = a.guards;
    return w;
}

__global__ void merge_status_kernel(WsHeader *top, const WsHeader *sub) {
    pdl_enter();
    if (sub->status != 0 && top->status == 0) {
        top->status = sub->status;
        top->detail = sub->detail;
    }
}
int merge_status(WsHeader *top, const void *sub, cudaStream_t st) {
    SBP_LAUNCH(merge_status_kernel, 1, 1, 0, st, top, reinterpret_cast<const WsHeader *>(sub));
    return STREAMBP_OK;
}
}  // namespace

template <typename T>
size_t model_workspace(const streambp_model_cfg &c, int64_t T_, int64_t chunk_layer, int64_t chunk_head) {
    return plan<T>(c, T_, chunk_layer, chunk_head, nullptr).bytes;
}

template <typename T>
int model_backward(const streambp_model_cfg &c, const T *embed, const streambp_layer_weights *layers, const T *g_final,
                   const T *w_vocab, const int64_t *ids, const T *X0, const int64_t *labels, int64_t T_,
                   int64_t chunk_layer, int64_t chunk_head, bool accumulate, float *loss, float *d_embed,
                   const streambp_layer_grads *layer_grads, float *d_g_final, float *d_w_vocab, T *dX0, void *ws,
                   cudaStream_t st) {
    const NvtxRange call_range("streambp model backward");
    ModelWs<T> s = plan<T>(c, T_, chunk_layer, chunk_head, ws);
    const int d = c.layer.d_model;
    const int L = c.n_layers;
    const int64_t act = T_ * d;
    SBP_TRY(ws_guards_arm(ws, s.guards, st));
    // layer 0 input
    if (ids) {
        SBP_TRY(embedding_gather<T>(embed, ids, T_, d, c.head.vocab, s.ckpt, s.hdr, st));
    } else if (!cuda_ok(cudaMemcpyAsync(s.ckpt, X0, sizeof(T) * act, cudaMemcpyDeviceToDevice, st))) {
        return STREAMBP_E_CUDA;
    }
    // forward, storing only layer inputs
    for (int l = 0; l < L; l++) {
        const NvtxRange r("checkpointing forward, layer", l);
        SBP_TRY(fill_zero(s.sub, kHeaderBytes, st));
        SBP_TRY(layer_forward<T>(c.layer, layers[l], s.ckpt + (int64_t)l * act, T_, chunk_layer, 0,
                                 s.ckpt + (int64_t)(l + 1) * act, s.sub, st));
        SBP_TRY(merge_status(s.hdr, s.sub, st));
    }
    // head
    SBP_TRY(fill_zero(s.sub, kHeaderBytes, st));
    SBP_TRY(lmhead_backward<T>(c.head, g_final, w_vocab, s.ckpt + (int64_t)L * act, labels, T_, chunk_head, accumulate,
                               loss, nullptr, s.ga, d_w_vocab, d_g_final, s.sub, st));
    SBP_TRY(merge_status(s.hdr, s.sub, st));
    // layers, last to first
    T *gin = s.ga, *gout = s.gb;
    for (int l = L - 1; l >= 0; l--) {
        const NvtxRange r("layer", l);
        SBP_TRY(fill_zero(s.sub, kHeaderBytes, st));
        T *dst = (l == 0 && dX0 && !ids) ? dX0 : gout;
        SBP_TRY(layer_backward<T>(c.layer, layers[l], s.ckpt + (int64_t)l * act, gin, T_, chunk_layer, 0, accumulate,
                                  layer_grads[l], dst, s.sub, st));
        SBP_TRY(merge_status(s.hdr, s.sub, st));
        gout = gin;
        gin = dst;
    }
    // gin now holds dL/dX0
    if (ids && d_embed) {
        if (!accumulate) SBP_TRY(fill_zero(d_embed, sizeof(float) * c.head.vocab * d, st));
        SBP_TRY(embedding_scatter_add<T>(gin, ids, T_, d, c.head.vocab, d_embed, st));
    }
    if (dX0 && gin != dX0) {
        if (!cuda_ok(cudaMemcpyAsync(dX0, gin, sizeof(T) * act, cudaMemcpyDeviceToDevice, st))) return STREAMBP_E_CUDA;
    }
    return ws_guards_check(ws, s.guards, s.hdr, st);
}

template size_t model_workspace<float>(const streambp_model_cfg &, int64_t, int64_t, int64_t);
template size_t model_workspace<bf16>(const streambp_model_cfg &, int64_t, int64_t, int64_t);
template int model_backward<float>(const streambp_model_cfg &, const float *, const streambp_layer_weights *,
                                   const float *, const float *, const int64_t *, const float *, const int64_t *,
                                   int64_t, int64_t, int64_t, bool, float *, float *, const streambp_layer_grads *,
                                   float *, float *, float *, void *, cudaStream_t);
template int model_backward<bf16>(const streambp_model_cfg &, const bf16 *, const streambp_layer_weights *,
                                  const bf16 *, const bf16 *, const int64_t *, const bf16 *, const int64_t *, int64_t,
                                  int64_t, int64_t, bool, float *, float *, const streambp_layer_grads *, float *,
                                  float *, bf16 *, void *, cudaStream_t);

}  // namespace sbp
