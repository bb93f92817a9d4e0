/*
 * streambp.h -- C ABI of the B200 (sm_100a) streamed backward pass.
 *
 * The library computes the exact gradient of a decoder-only transformer by the
 * sequence-partitioned accumulation of the paper's Eq. (1):
 *     dL/dW = sum_i (dZ_out^(i)/dW)^T dL/dZ_out^(i)
 * over chunks i of `chunk` consecutive token rows (the paper's "partition size";
 * the last chunk may be shorter, and chunk >= T means a single chunk, i.e. the
 * ordinary un-partitioned backward, Sec. 4.3 "partition will not be performed if
 * it is larger than the sequence length").
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, row-major,
 *     16-byte aligned; `workspace` is device memory, 256-byte aligned.  Config and
 *     weight/grad pointer structs are HOST memory, read during the call only.
 *   - Matrices are stored [out_features, in_features] (y = x W^T).
 *   - `dtype` selects the storage type of activations and weights (X, dY, dX, H,
 *     dH, every weight): float or bf16.  Weight gradients, the loss and all
 *     accumulators are always float (fp32).  bf16 runs multiply bf16 operands and
 *     accumulate in fp32.
 *   - The library allocates no device memory and writes only to the outputs and the
 *     workspace; nothing a call computes survives it.  What the process does keep:
 *     per-device facts looked up once (SM count, kernel attributes, the address of
 *     the fixed scratch array of streambp_attention_backward_static), the per-thread
 *     record behind streambp_last_cuda_error / streambp_last_launch_count, a device
 *     flag a kernel raises when a bounded wait expires, and the event records of the
 *     optional profiling below.  Work is enqueued on `cuda_stream` (a cudaStream_t
 *     passed as void*, NULL = default stream) and the call returns without
 *     synchronising.
 *   - Return value: STREAMBP_OK (0) or a negative streambp_status.  Errors found
 *     on the host are returned before anything is enqueued.  Conditions only the
 *     device can see (a label outside [0, vocab), no unmasked label, an expired
 *     bounded wait inside a kernel) are recorded in the workspace header and read
 *     back with streambp_last_device_status().  Nothing aborts, traps or throws.
 *   - `accumulate` = 0 overwrites the weight-gradient outputs ("initialised from
 *     zero", text after Eq. (3)); 1 adds to what they hold.
 *   - Environment, read once per process: STREAMBP_GEMM_ENGINE = "simt" | "tc"
 *     forces the CUDA-core or the tcgen05 product kernels (default: tcgen05 for bf16,
 *     CUDA cores for fp32); STREAMBP_GEMM_SINGLE_CTA (any value) selects the
 *     single-CTA tcgen05 product kernel instead of the CTA-pair one, which is also
 *     what runs where a two-CTA cluster cannot be scheduled; STREAMBP_VERBOSE (any
 *     value) reports that choice on stderr; STREAMBP_WS_GUARD (any value) is a debug mode
 *     that puts a 256-byte guard after every sub-buffer of the workspaces (the size
 *     queries grow accordingly), fills the guards before and checks them after each
 *     call, and reports an overwritten guard as STREAMBP_E_WORKSPACE_GUARD through
 *     streambp_last_device_status; STREAMBP_PDL=0 launches every kernel with plain
 *     stream ordering instead of programmatic dependent launch (by default a kernel's
 *     blocks may become resident while the kernel before it in the stream is finishing;
 *     every kernel waits for that kernel's completion before it touches memory).  None of
 *     them changes a result beyond floating-point summation order.
 */
#ifndef STREAMBP_H_
#define STREAMBP_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STREAMBP_OK = 0,
    STREAMBP_E_NULL = -1,            /* a required pointer is NULL */
    STREAMBP_E_SHAPE = -2,           /* unsupported or inconsistent sizes */
    STREAMBP_E_ALIGN = -3,           /* pointer alignment */
    STREAMBP_E_WORKSPACE = -4,       /* workspace_bytes smaller than *_workspace_bytes() */
    STREAMBP_E_DTYPE = -5,           /* unknown dtype */
    STREAMBP_E_CUDA = -6,            /* a CUDA runtime / driver call failed */
    STREAMBP_E_BAD_LABEL = -7,       /* device: label not in [0, vocab) and != ignore_index */
    STREAMBP_E_NO_VALID_LABELS = -8, /* device: every label ignored; loss and grads are 0 */
    STREAMBP_E_DEVICE_TIMEOUT = -9,  /* device: a bounded wait inside a kernel ran out */
    STREAMBP_E_WORKSPACE_GUARD = -10 /* device, debug mode STREAMBP_WS_GUARD: a kernel wrote past a workspace sub-buffer */
} streambp_status;

typedef enum { STREAMBP_F32 = 0, STREAMBP_BF16 = 1 } streambp_dtype;

/* One pre-norm decoder layer: RMSNorm -> GQA causal attention with rotate-half RoPE
 * -> residual -> RMSNorm -> SwiGLU MLP -> residual (the attention / MLP transformation
 * of Sec. 3.2.2 with the normalisation, heads and residuals it leaves out restored). */
typedef struct {
    int32_t d_model;
    int32_t n_q_heads;
    int32_t n_kv_heads;   /* divides n_q_heads */
    int32_t head_dim;     /* 64 or 128 */
    int32_t d_ff;         /* SwiGLU intermediate width */
    int32_t qkv_bias;     /* 1: bq, bk, bv present */
    float rope_theta;
    float rms_eps;
    int32_t dtype;        /* streambp_dtype */
} streambp_layer_cfg;

/* Weights in storage dtype. g1,g2: [d_model]; wq: [Hq*dh, d]; wk,wv: [Hkv*dh, d];
 * wo: [d, Hq*dh]; w_gate,w_up: [d_ff, d]; w_down: [d, d_ff]; bq: [Hq*dh]; bk,bv: [Hkv*dh]
 * (biases NULL unless qkv_bias). */
typedef struct {
    const void *g1, *wq, *bq, *wk, *bk, *wv, *bv, *wo, *g2, *w_gate, *w_up, *w_down;
} streambp_layer_weights;

/* fp32 gradients, same shapes as the weights. */
typedef struct {
    float *g1, *wq, *bq, *wk, *bk, *wv, *bv, *wo, *g2, *w_gate, *w_up, *w_down;
} streambp_layer_grads;

/* Bytes of workspace streambp_layer_backward needs; 0 if the arguments are invalid. */
size_t streambp_layer_workspace_bytes(const streambp_layer_cfg *cfg, int64_t T, int64_t chunk);

/*
 * Streamed backward of one decoder layer (Sec. 3.2.2, partitioned attention / MLP
 * equations and the accumulation after them).
 *
 * Given the checkpointed layer input X [T, d_model], the upstream gradient dY [T, d_model]
 * and the weights, computes dX [T, d_model] and every weight gradient.  K and V (after
 * RoPE) are computed once for all T rows and cached in the workspace; then for each chunk
 * the library re-forwards that chunk (norm, Q, attention of the chunk's queries against
 * keys/values 0 .. chunk end only, output projection, norm, gate/up) and back-propagates
 * it, adding into the fp32 weight gradients and into fp32 dK/dV accumulators for the key
 * prefix.  `pos0` is the RoPE position of row 0.  The down-projection forward is never
 * computed: dY is given.  dX may not alias X or dY.
 */
int streambp_layer_backward(const streambp_layer_cfg *cfg, const streambp_layer_weights *w,
                            const void *X, const void *dY, int64_t T, int64_t chunk, int64_t pos0,
                            int accumulate, const streambp_layer_grads *grads, void *dX,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same streamed backward for a PACKED BATCH: X and dY hold n_seqs sequences back to back
 * (rows cu_seqlens[i] .. cu_seqlens[i+1]-1 are sequence i; cu_seqlens is a HOST array of n_seqs + 1
 * increasing entries from 0 to T).  Tokens attend only to earlier tokens of their own sequence and
 * rotary positions restart at pos0 in every sequence; every other step of the layer is row-wise, so a
 * chunk may span sequences and the products keep the chunk as their row dimension however short the
 * sequences are (the paper's transfer of sequence-length scaling to batch-size scaling, Sec. 4.1).
 * The result equals the sum over the sequences of streambp_layer_backward on each of them.
 * Workspace: streambp_layer_workspace_bytes(cfg, T, chunk).  Errors: additionally STREAMBP_E_SHAPE
 * for malformed cu_seqlens.
 */
int streambp_layer_backward_packed(const streambp_layer_cfg *cfg, const streambp_layer_weights *w,
                                   const void *X, const void *dY, int64_t T, int64_t chunk,
                                   const int64_t *cu_seqlens, int32_t n_seqs, int64_t pos0, int accumulate,
                                   const streambp_layer_grads *grads, void *dX,
                                   void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same streamed backward with a SECOND partition size for the weight gradients (Sec. 4.3, effect of the
 * partition size: every partition pays one read-modify-write pass over the fp32 gradient of every weight, which is
 * what makes small partitions slow).  The chunk loop is unchanged -- re-forward, attention and input gradients run per
 * `chunk` rows -- but the weight-gradient products g_W += (dZ_out/dW)^T dL/dZ_out of Eq. (1) are formed once per
 * `wgrad_group` consecutive chunks, as one product over wgrad_group * chunk rows, so the accumulators are passed over
 * D / wgrad_group times instead of D times.  The price is memory: the operands of those products (the chunk's
 * normalised inputs, attention output, gate / up / SwiGLU activations and their gradients) are kept for every chunk
 * of a group.  wgrad_group = 1 is streambp_layer_backward; values above the number of chunks act like that number.
 * The result is the same sum in a different association (equal within rounding of the fp32 accumulation).
 * cu_seqlens may be NULL (one sequence) or describe a packed batch as in streambp_layer_backward_packed.
 * Workspace: streambp_layer_workspace_bytes_grouped(cfg, T, chunk, wgrad_group).
 */
size_t streambp_layer_workspace_bytes_grouped(const streambp_layer_cfg *cfg, int64_t T, int64_t chunk,
                                              int32_t wgrad_group);
int streambp_layer_backward_grouped(const streambp_layer_cfg *cfg, const streambp_layer_weights *w, const void *X,
                                    const void *dY, int64_t T, int64_t chunk, int32_t wgrad_group,
                                    const int64_t *cu_seqlens, int32_t n_seqs, int64_t pos0, int accumulate,
                                    const streambp_layer_grads *grads, void *dX, void *workspace,
                                    size_t workspace_bytes, void *cuda_stream);

typedef struct {
    int32_t d_model;
    int64_t vocab;
    float rms_eps;
    int64_t ignore_index;
    int32_t dtype;        /* streambp_dtype */
} streambp_head_cfg;

size_t streambp_lmhead_workspace_bytes(const streambp_head_cfg *cfg, int64_t T, int64_t chunk);

/*
 * Streamed final-RMSNorm + LM head + cross-entropy backward (Sec. 3.2.1, SFT objective
 * Eq. (2) and the accumulation Eq. (3)), normalised to the MEAN over unmasked tokens.
 *
 * H [T, d] are the last layer's hidden states, w_vocab [vocab, d], g_final [d],
 * labels [T] (int64, already aligned to the logit rows; ignore_index marks masked rows).
 * The number N of unmasked labels is counted first; then per chunk the fp32 logits
 * [chunk, vocab] are formed, reduced to their log-sum-exp, turned into
 * dlogits = (softmax - onehot)/N (zero rows where ignored) and consumed by the two
 * gradient products, so that [T, vocab] never exists.
 * Outputs: *loss (device float), *n_valid (device int64), dH [T, d] storage dtype,
 * d_w_vocab [vocab, d] fp32, d_g_final [d] fp32.  `accumulate` applies to d_w_vocab and
 * d_g_final.  If N == 0 the loss and all gradients are written as 0 and the device
 * status becomes STREAMBP_E_NO_VALID_LABELS.
 */
int streambp_lmhead_ce_backward(const streambp_head_cfg *cfg, const void *g_final, const void *w_vocab,
                                const void *H, const int64_t *labels, int64_t T, int64_t chunk,
                                int accumulate, float *loss, int64_t *n_valid, void *dH,
                                float *d_w_vocab, float *d_g_final,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * The same streamed head under the reinforcement-learning objectives of Sec. 3.2.1.  Both depend on the
 * logits only through log pi_theta(t) = logits[t, token_t] - logsumexp(logits[t, :]), so each chunk's
 * dlogits are c_t * (onehot(token_t) - softmax(logits[t, :])) with a per-token coefficient c_t, and the
 * chunk loop, the two gradient products and the norm backward are those of the SFT head.
 *
 *   STREAMBP_OBJ_GRPO (Eq. (4)):  L = - sum_t weight_t f(t),
 *       f(t) = min(r_t A_t, clip(r_t, 1-clip_eps, 1+clip_eps) A_t) - beta (log pi_theta(t) - logp_ref[t]),
 *       r_t = exp(log pi_theta(t) - logp_old[t]).  weight_t carries the 1/(G T_o) of the objective
 *       (any per-token weighting is allowed); advantage[t] = A_t.
 *   STREAMBP_OBJ_DPO (Eq. (5)):   L = - log sigmoid(beta * ell),
 *       ell = sum_t weight_t (log pi_theta(t) - logp_ref[t]) with weight_t = +1 on the chosen response's
 *       tokens and -1 on the rejected one's.  As in the paper, ell and the un-corrected gradients
 *       beta * sum_t d ell(t) are accumulated over the chunks and the outputs are then multiplied in place
 *       by (sigmoid(beta ell) - 1); because of that in-place correction `accumulate` must be 0.
 *
 * tokens [T] int64 (ignore_index: the row takes no part); logp_old, logp_ref, advantage, weight: fp32 [T]
 * device arrays (logp_old and advantage are not read for DPO).  Outputs: *loss; logp [T] fp32 (optional,
 * log pi_theta of the given tokens, 0 on rows that take no part); *ell (optional, DPO); dH, d_w_vocab,
 * d_g_final as in streambp_lmhead_ce_backward.  Workspace: streambp_lmhead_workspace_bytes().
 */
typedef enum { STREAMBP_OBJ_GRPO = 1, STREAMBP_OBJ_DPO = 2 } streambp_objective;
typedef struct {
    int32_t objective;   /* streambp_objective */
    float beta;
    float clip_eps;      /* GRPO only */
} streambp_rl_cfg;

int streambp_lmhead_rl_backward(const streambp_head_cfg *cfg, const streambp_rl_cfg *rl, const void *g_final,
                                const void *w_vocab, const void *H, const int64_t *tokens, const float *logp_old,
                                const float *logp_ref, const float *advantage, const float *weight, int64_t T,
                                int64_t chunk, int accumulate, float *loss, float *logp, float *ell, void *dH,
                                float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                void *cuda_stream);

/*
 * The streamed LM-head backward with a SECOND partition size for the vocabulary weight gradient (Sec. 4.3, effect of
 * the partition size; Sec. 3.2.1 for the step itself).  Logits, loss rows and dL/dH still run per `chunk` rows, but
 * d_w_vocab += dlogits^T hn is formed once per `wgrad_group` consecutive chunks, as one product over
 * wgrad_group * chunk rows: the [vocab, d_model] fp32 accumulator is read and written D / wgrad_group times instead of
 * D times.  The price is memory: the normalised hidden rows and the dlogits are kept for every chunk of a group (the
 * fp32 logits still exist for one chunk only when storage is bf16).  A group whose labels are all ignored is skipped
 * on the device; a masked chunk inside a live group is processed (its dlogits are zero).  wgrad_group = 1 is the plain
 * entry point; values above the number of chunks act like that number.  Same sums in a different association.
 * All other arguments, outputs and errors as in streambp_lmhead_ce_backward / streambp_lmhead_rl_backward;
 * STREAMBP_E_SHAPE also for wgrad_group < 1.  Workspace: streambp_lmhead_workspace_bytes_grouped().
 */
size_t streambp_lmhead_workspace_bytes_grouped(const streambp_head_cfg *cfg, int64_t T, int64_t chunk,
                                               int32_t wgrad_group);
int streambp_lmhead_ce_backward_grouped(const streambp_head_cfg *cfg, const void *g_final, const void *w_vocab,
                                        const void *H, const int64_t *labels, int64_t T, int64_t chunk,
                                        int32_t wgrad_group, int accumulate, float *loss, int64_t *n_valid, void *dH,
                                        float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream);
int streambp_lmhead_rl_backward_grouped(const streambp_head_cfg *cfg, const streambp_rl_cfg *rl, const void *g_final,
                                        const void *w_vocab, const void *H, const int64_t *tokens,
                                        const float *logp_old, const float *logp_ref, const float *advantage,
                                        const float *weight, int64_t T, int64_t chunk, int32_t wgrad_group,
                                        int accumulate, float *loss, float *logp, float *ell, void *dH,
                                        float *d_w_vocab, float *d_g_final, void *workspace, size_t workspace_bytes,
                                        void *cuda_stream);

typedef struct {
    int32_t n_layers;
    streambp_layer_cfg layer;
    streambp_head_cfg head;
} streambp_model_cfg;

/* Includes the [n_layers][T, d] layer-input checkpoints (storage dtype). */
size_t streambp_model_workspace_bytes(const streambp_model_cfg *cfg, int64_t T,
                                      int64_t chunk_layer, int64_t chunk_head);

/*
 * Whole-model backward with layer-input checkpoints only (Sec. 2 / Sec. 3.1: the
 * substrate the streamed backward sits on): embedding lookup (or X0 given), a chunked
 * forward that stores each layer's input, the streamed head backward, then the streamed
 * layer backward for l = L..1 with dY := dX of the layer above, and the embedding
 * scatter-add.  `layers` and `layer_grads` are host arrays of n_layers structs.
 * ids [T] int64 index `embed` [vocab, d]; if ids is NULL, X0 [T, d] is the first layer's
 * input (then embed / d_embed may be NULL).  dX0 [T, d] (storage dtype) may be NULL.
 */
int streambp_model_backward(const streambp_model_cfg *cfg, const void *embed,
                            const streambp_layer_weights *layers, const void *g_final, const void *w_vocab,
                            const int64_t *ids, const void *X0, const int64_t *labels, int64_t T,
                            int64_t chunk_layer, int64_t chunk_head, int accumulate,
                            float *loss, float *d_embed, const streambp_layer_grads *layer_grads,
                            float *d_g_final, float *d_w_vocab, void *dX0,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Partition size for a memory budget (Sec. 4.3, "Effect of partition size": a partition that is too small
 * pays for re-loading the weights and for the fp32 read-modify-write of every weight gradient once per
 * partition, while a larger one costs only marginally more memory).  Returns the largest chunk, a multiple
 * of 128 rows (or T itself when T fits), whose workspace as reported by streambp_layer_workspace_bytes /
 * streambp_lmhead_workspace_bytes does not exceed budget_bytes; 0 if even one 128-row chunk does not fit or
 * an argument is invalid.  Host-only: no GPU work, no allocation.
 */
int64_t streambp_layer_suggest_chunk(const streambp_layer_cfg *cfg, int64_t T, size_t budget_bytes);
int64_t streambp_lmhead_suggest_chunk(const streambp_head_cfg *cfg, int64_t T, size_t budget_bytes);

/* Synchronises `cuda_stream` and returns the status the kernels of the last call using
 * this workspace recorded (STREAMBP_OK, E_BAD_LABEL, E_NO_VALID_LABELS, E_DEVICE_TIMEOUT),
 * or STREAMBP_E_CUDA if the stream reports an error. */
int streambp_last_device_status(void *workspace, void *cuda_stream);

const char *streambp_status_string(int status);

/* The last CUDA error code (cudaError_t / CUresult as int) behind a STREAMBP_E_CUDA
 * returned on the calling thread; 0 if none. */
int streambp_last_cuda_error(void);

/* Number of kernel launches the last call on the calling thread enqueued. */
int64_t streambp_last_launch_count(void);

/*
 * Building block exposed for tests and profiling: C = A * B (+ bias) with the operand
 * layouts the three gradient products of Eq. (1) need.  op: 0 = "NT" C[M,N] = A[M,K] B[N,K]^T
 * (forward y = x W^T), 1 = "NN" C[M,N] = A[M,K] B[K,N] (input gradient dY W),
 * 2 = "TN" C[M,N] = A[K,M]^T B[K,N] (weight gradient dY^T X).  A and B have `in_dtype`
 * (row-major, leading dimensions lda/ldb in elements), C has `out_dtype`, leading dimension
 * ldc; accumulate = 1 adds to C (fp32 C only).  engine: 0 = automatic, 1 = fp32 CUDA-core
 * kernel, 2 = tcgen05 tensor-core kernel (bf16 operands only).
 */
int streambp_gemm(int op, int64_t M, int64_t N, int64_t K, const void *A, int64_t lda,
                  const void *B, int64_t ldb, void *C, int64_t ldc, int32_t in_dtype,
                  int32_t out_dtype, int accumulate, int engine, void *cuda_stream);

/*
 * Building block exposed for tests and profiling: several independent products in ONE launch of the
 * tensor-core kernel (bf16 operands).  The per-chunk gradients of Eq. (1) that become ready together
 * (e.g. dWg += dg^T h2, dWu += du^T h2 and dh2 = dg Wg + du Wu after the partitioned MLP of
 * Sec. 3.2.2) share a launch so that their tiles fill the GPU together.  Problem i computes
 * C_i (+)= sum over its n_segments K segments of op(A_s, B_s), `op` and layouts as in streambp_gemm;
 * all segments of a problem share M, N and C.  n <= 4 problems, 8 segments in total, 1..3 per problem.
 * out_dtype STREAMBP_F32 (accumulate allowed) or STREAMBP_BF16 (the sum over segments is formed in fp32
 * and rounded once; accumulate not allowed).
 * sched: NULL, or two int32 of device memory that are zero when the launch starts; the kernel then
 * hands tiles to CTAs dynamically (longest first) and leaves the two ints zero again.  The result does
 * not depend on the schedule.  Returns STREAMBP_E_SHAPE if a problem does not meet the tensor-core
 * kernel's alignment rules (leading dimensions multiples of 8 elements, 16-byte aligned pointers).
 */
typedef struct {
    int32_t op;
    int32_t n_segments;
    int64_t M, N;
    const void *A[3];
    int64_t lda[3];
    const void *B[3];
    int64_t ldb[3];
    int64_t K[3];
    void *C;
    int64_t ldc;
    int32_t out_dtype;
    int32_t accumulate;
} streambp_gemm_problem;
int streambp_gemm_grouped(const streambp_gemm_problem *problems, int32_t n, int32_t *sched, void *cuda_stream);

/*
 * The MLP's first half as the layer runs it (Sec. 3.2.2, the partitioned MLP): g = A W_gate^T, u = A W_up^T and
 * m = silu(g) * u, with silu taken of the values ROUNDED to the storage type (the ones the backward reads).
 * A: [M, K] (lda), W_gate, W_up: [N, K] (ldb), g, u, m: [M, N] dense; all of `dtype` (float or bf16), device.
 * bf16 on the CTA-pair product kernel is ONE launch (the even CTA of a pair fetches W_gate rows, the odd one
 * W_up rows, so g and u of the same columns meet in one accumulator row); otherwise two products and an
 * element-wise kernel.  Same results either way up to the summation order of the products.
 */
int streambp_gemm_swiglu(const void *A, int64_t lda, const void *w_gate, const void *w_up, int64_t ldb, int64_t M,
                         int64_t N, int64_t K, void *g, void *u, void *m, int32_t dtype, void *cuda_stream);

/*
 * Building blocks exposed for tests and profiling: the partitioned attention of Sec. 3.2.2
 * (S^(i) = Q^(i) K^(:i)T, causal softmax, O^(i) = P^(i) V^(:i)) for one chunk of n query rows that
 * sit at absolute rows q0 .. q0+n-1 and attend to keys 0 .. q0+n-1, and its backward.
 * q, o, d_o: [n, n_q_heads, head_dim]; k, v: [q0+n, n_kv_heads, head_dim] (storage dtype);
 * lse: [n_q_heads, n] fp32 (natural log of the row sums of exp(score / sqrt(head_dim)));
 * delta: scratch [n_q_heads, n] fp32; dq: [n, n_q_heads, head_dim] fp32, overwritten;
 * dk, dv: [q0+n, n_kv_heads, head_dim] fp32, ADDED to (the key-prefix accumulators).
 * engine: 0 automatic, 1 CUDA cores, 2 tensor cores (bf16, head_dim 128 only); the forward also takes 3 / 4 =
 * tensor cores with one / two 128-query tiles per CTA (2 picks between them from the grid size); the backward also
 * takes 5 = the five-product tensor-core kernel: one CTA role, the key-tile owners also form dQ and add their
 * shares into it in global memory (dq is cleared by the call), so S and dP are not recomputed by a second role.
 * Its dQ is not bit-reproducible from run to run (the order of those adds is not fixed; dK and dV are), which is
 * why the deterministic two-role kernel stays the default.  Environment STREAMBP_ATTN_BWD=five makes the
 * five-product kernel the choice of the schedulers (layer / model entry points) in this process.
 */
int streambp_attention_forward(const void *q, const void *k, const void *v, int64_t n, int64_t q0,
                               int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                               void *o, float *lse, int engine, void *cuda_stream);
int streambp_attention_backward(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                const float *lse, int64_t n, int64_t q0, int32_t n_q_heads, int32_t n_kv_heads,
                                int32_t head_dim, int32_t dtype, float *delta, float *dq, float *dk, float *dv,
                                int engine, void *cuda_stream);

/*
 * (No counterpart in the paper.)  streambp_attention_backward for callers that have no device buffer
 * to offer for `delta` and cannot obtain one when they call: host code in a latency-critical loop
 * where cudaMalloc / cudaFree would stall the whole device, a plug-in whose host framework already owns
 * all device memory, a process whose memory budget is frozen after start-up.  Same arguments and results
 * as streambp_attention_backward minus `delta` (engine 0, 1 or 2 only): the row sums live in a fixed array inside the library
 * image, STREAMBP_STATIC_DELTA_MAX_FLOATS floats (4 MiB) that every GPU loading the library holds until
 * the process exits.  The call performs no device-memory allocation of any kind.
 *   - Limit: n * n_q_heads <= STREAMBP_STATIC_DELTA_MAX_FLOATS, else STREAMBP_E_WORKSPACE is returned
 *     and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  Its previous contents are irrelevant (every row sum
 *     used by a call is rewritten by that call first), but two calls whose kernels overlap on the GPU
 *     (different streams, or several host threads) race on it: serialise them on one stream.
 */
#define STREAMBP_STATIC_DELTA_MAX_FLOATS (1 << 20)
int streambp_attention_backward_static(const void *q, const void *k, const void *v, const void *o, const void *d_o,
                                       const float *lse, int64_t n, int64_t q0, int32_t n_q_heads,
                                       int32_t n_kv_heads, int32_t head_dim, int32_t dtype, float *dq, float *dk,
                                       float *dv, int engine, void *cuda_stream);

/*
 * Optional device timing by kernel class (0 = linear products, 1 = attention forward,
 * 2 = attention backward).  While enabled, each launch of those classes is bracketed by CUDA
 * events on the caller's stream.  streambp_profile_enable(1) also clears earlier records;
 * streambp_profile_read() waits for the recorded events and returns, for one class, the summed
 * device time, the number of bracketed launches and their algorithmic FLOPs (products: 2MNK;
 * attention: 2 * head_dim per causal (query, key) pair and product).  Not thread-safe; meant for
 * benchmarks.
 */
void streambp_profile_enable(int on);
int streambp_profile_read(int kernel_class, double *milliseconds, int64_t *calls, double *flops);

/*
 * Which tcgen05 product kernel bf16 products run on the current device: 2 = CTA pairs
 * (cta_group::2, 256 x 256 tiles), 1 = single CTA (128 x 256 tiles; a two-CTA cluster cannot be
 * scheduled, or STREAMBP_GEMM_SINGLE_CTA is set), 0 = none (no tensor-map support: bf16 products
 * fall back to the CUDA-core kernels).  Host-only query; launches nothing.
 */
int streambp_product_kernel(void);

/*
 * Test hooks (no counterpart in the paper; not part of the method).
 *
 * streambp_test_expire_wait: launches a one-CTA kernel that runs the library's bounded mbarrier wait -- the
 * same device function every tensor-core kernel waits in -- on a barrier nothing arrives at, with `limit_ns`
 * (1 us .. 100 ms) in place of the kernels' two seconds, and then winds down as those kernels do (abort flag,
 * drain, tensor memory freed).  The GPU is not hung and the context stays usable; afterwards
 * streambp_last_device_status() on that stream returns STREAMBP_E_DEVICE_TIMEOUT once and clears the flag.
 *
 * streambp_test_per_device_value: the library caches per-device facts (SM count, shared-memory opt-in, product
 * kernel choice) by device ordinal.  This runs that cache with `ordinal` in place of the current device and a
 * value to remember on first use: it returns the value cached for that ordinal.  Host-only.
 *
 * streambp_test_workspace_guard: plans three sub-buffers with guards in `workspace` (>= 4096 bytes, 256-byte
 * aligned; guards are used here whether or not STREAMBP_WS_GUARD is set), fills the guards, has a kernel write
 * `overrun` floats past the end of the second sub-buffer (0: none), checks the guards and records the outcome in the
 * workspace header: afterwards streambp_last_device_status is STREAMBP_OK or STREAMBP_E_WORKSPACE_GUARD.
 */
int streambp_test_expire_wait(uint64_t limit_ns, void *cuda_stream);
int streambp_test_workspace_guard(void *workspace, size_t workspace_bytes, int32_t overrun, void *cuda_stream);
int streambp_test_per_device_value(int ordinal, int value);

#ifdef __cplusplus
}
#endif
#endif /* STREAMBP_H_ */
