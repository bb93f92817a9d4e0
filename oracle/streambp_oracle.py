"""CPU oracle for the streamed backward pass -- TEST INFRASTRUCTURE ONLY.

The paper's method is exact: accumulating the per-partition terms of Eq. (1)
over any partition of the sequence gives the ordinary gradient (Eq. (1), the
text after Eq. (3), and the text after Eq. (5)).  The oracle is therefore the
plain definition that the streamed path must reach: an ordinary, NON-streamed,
full-sequence forward and backward of

  * one pre-norm decoder layer (RMSNorm, GQA causal attention with RoPE,
    residual, RMSNorm, SwiGLU MLP, residual) -- the attention / MLP skeleton of
    Sec. 3.2.2 with the normalisation, heads and residuals the paper leaves out
    "without loss of generality" put back in the usual Llama/Qwen form;
  * the final RMSNorm + language-modelling head + mean cross-entropy over the
    unmasked tokens (Sec. 3.2.1, SFT objective, Eq. (2)), and the same head under
    the GRPO (Eq. (4)) and DPO (Eq. (5)) objectives;
  * a stack of such layers between an embedding lookup and that head.

Everything is numpy float64.  `numpy.matmul`, `exp`, `log`, `cos`, `sin` are the
only library steps.  Loops over row blocks exist only to bound memory: every
row of a softmax, a norm or a matrix product is independent of the others by
definition, so a row block computes exactly the rows it holds against the
complete set of keys / vocabulary entries those rows see.  There is no chunked
accumulation logic, no online softmax, no tiling of a reduction.

Pinned (tests/test_oracle_*.py) by central finite differences, by an
independent PyTorch-autograd restatement, and by closed forms (zero head
weights, single-token attention, RMSNorm orthogonality, RoPE isometry).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module; it shares no code with the CUDA path.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np

F64 = np.float64


@dataclass(frozen=True)
class LayerCfg:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    qkv_bias: bool
    rope_theta: float
    rms_eps: float = 1e-6


@dataclass(frozen=True)
class HeadCfg:
    d_model: int
    vocab: int
    rms_eps: float = 1e-6
    ignore_index: int = -100


def _f64(a):
    return None if a is None else np.asarray(a, dtype=F64)


# ---------------------------------------------------------------------------
# RMSNorm
# ---------------------------------------------------------------------------

def rmsnorm_forward(x, gain, eps):
    """h = x / sqrt(mean_j x_j^2 + eps) * gain, row by row. Returns (h, xhat, rms)."""
    rms = np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    xhat = x / rms
    return xhat * gain, xhat, rms


def rmsnorm_backward(dh, xhat, rms, gain):
    """Gradient of rmsnorm_forward: with w = dh * gain,
    dx = (w - xhat * mean_j(w_j xhat_j)) / rms and dgain = sum_t dh_t * xhat_t."""
    w = dh * gain
    dx = (w - xhat * np.mean(w * xhat, axis=-1, keepdims=True)) / rms
    dgain = np.sum(dh * xhat, axis=0)
    return dx, dgain


# ---------------------------------------------------------------------------
# Rotary position embedding (rotate-half pairing)
# ---------------------------------------------------------------------------

def rope_tables(positions, head_dim, theta):
    """cos/sin of angle p * theta^(-2j/head_dim), j < head_dim/2. Shapes [T, head_dim/2]."""
    half = head_dim // 2
    j = np.arange(half, dtype=F64)
    inv_freq = np.power(F64(theta), -2.0 * j / head_dim)
    ang = np.asarray(positions, dtype=F64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def rope_apply(u, cos, sin):
    """u: [T, H, dh]. Pair (j, j+dh/2) is rotated by the angle of position t, frequency j."""
    half = u.shape[-1] // 2
    a, b = u[..., :half], u[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def rope_apply_transpose(du, cos, sin):
    """Gradient through rope_apply: the rotation by the negative angle."""
    half = du.shape[-1] // 2
    a, b = du[..., :half], du[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    return np.concatenate([a * c + b * s, b * c - a * s], axis=-1)


# ---------------------------------------------------------------------------
# Causal grouped-query attention (Sec. 3.2.2 attention equations, scaled, causal mask)
# ---------------------------------------------------------------------------

def _causal_probs(q_rows, k_all, t0, scale):
    """softmax over keys s <= t for query rows t0.. against keys 0..t1-1."""
    n = q_rows.shape[0]
    t1 = t0 + n
    s = (q_rows @ k_all[:t1].T) * scale
    key = np.arange(t1)[None, :]
    row = (t0 + np.arange(n))[:, None]
    s = np.where(key <= row, s, -np.inf)
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention_forward(q, k, v, row_block=1024, q_start=0):
    """q: [T - q_start, Hq, dh], the query rows q_start .. T-1; k, v: [T, Hkv, dh]; query head h reads KV head
    h // (Hq/Hkv).  q_start > 0 only restricts which rows are evaluated (rows are independent)."""
    n, Hq, dh = q.shape
    T = q_start + n
    G = Hq // k.shape[1]
    scale = 1.0 / np.sqrt(F64(dh))
    o = np.empty_like(q)
    for h in range(Hq):
        kh, vh = k[:, h // G, :], v[:, h // G, :]
        for t0 in range(q_start, T, row_block):
            t1 = min(T, t0 + row_block)
            p = _causal_probs(q[t0 - q_start:t1 - q_start, h, :], kh, t0, scale)
            o[t0 - q_start:t1 - q_start, h, :] = p @ vh[:t1]
    return o


def attention_backward(q, k, v, do, row_block=1024, q_start=0):
    """Returns (dq, dk, dv). dk, dv are summed over the query heads of each KV group.  q, do: the query rows
    q_start .. T-1 (as in attention_forward); dk, dv: [T, Hkv, dh], the contribution of those rows."""
    n, Hq, dh = q.shape
    T = q_start + n
    G = Hq // k.shape[1]
    scale = 1.0 / np.sqrt(F64(dh))
    dq = np.empty_like(q)
    dk = np.zeros_like(k[:T])
    dv = np.zeros_like(v[:T])
    for h in range(Hq):
        g = h // G
        kh, vh = k[:, g, :], v[:, g, :]
        for t0 in range(q_start, T, row_block):
            t1 = min(T, t0 + row_block)
            a, b = t0 - q_start, t1 - q_start
            p = _causal_probs(q[a:b, h, :], kh, t0, scale)
            doh = do[a:b, h, :]
            dv[:t1, g, :] += p.T @ doh
            dp = doh @ vh[:t1].T
            ds = p * (dp - np.sum(p * dp, axis=-1, keepdims=True))
            dq[a:b, h, :] = (ds @ kh[:t1]) * scale
            dk[:t1, g, :] += (ds.T @ q[a:b, h, :]) * scale
    return dq, dk, dv


# ---------------------------------------------------------------------------
# SwiGLU
# ---------------------------------------------------------------------------

def _sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def silu(z):
    return z * _sigmoid(z)


def silu_grad(z):
    s = _sigmoid(z)
    return s * (1.0 + z * (1.0 - s))


# ---------------------------------------------------------------------------
# Decoder layer
# ---------------------------------------------------------------------------

def _layer_forward_full(cfg: LayerCfg, W: Dict[str, np.ndarray], X, pos0, row_block):
    T = X.shape[0]
    Hq, Hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    h1, xhat1, rms1 = rmsnorm_forward(X, W["g1"], cfg.rms_eps)
    q = h1 @ W["wq"].T
    k = h1 @ W["wk"].T
    v = h1 @ W["wv"].T
    if cfg.qkv_bias:
        q, k, v = q + W["bq"], k + W["bk"], v + W["bv"]
    cos, sin = rope_tables(pos0 + np.arange(T), dh, cfg.rope_theta)
    qr = rope_apply(q.reshape(T, Hq, dh), cos, sin)
    kr = rope_apply(k.reshape(T, Hkv, dh), cos, sin)
    vh = v.reshape(T, Hkv, dh)
    o = attention_forward(qr, kr, vh, row_block).reshape(T, Hq * dh)
    r = X + o @ W["wo"].T
    h2, xhat2, rms2 = rmsnorm_forward(r, W["g2"], cfg.rms_eps)
    g = h2 @ W["w_gate"].T
    u = h2 @ W["w_up"].T
    m = silu(g) * u
    y = r + m @ W["w_down"].T
    cache = dict(h1=h1, xhat1=xhat1, rms1=rms1, qr=qr, kr=kr, vh=vh, cos=cos, sin=sin, o=o,
                 xhat2=xhat2, rms2=rms2, h2=h2, g=g, u=u, m=m)
    return y, cache


def layer_forward(cfg: LayerCfg, W, X, pos0=0, row_block=1024):
    """Y = layer(X): pre-norm attention block then pre-norm SwiGLU block, both residual."""
    W = {k: _f64(v) for k, v in W.items()}
    return _layer_forward_full(cfg, W, _f64(X), pos0, row_block)[0]


def layer_backward(cfg: LayerCfg, W, X, dY, pos0=0, row_block=1024):
    """Ordinary full-sequence backward of one decoder layer.

    Given the layer input X [T, d], its weights and dL/dY [T, d], returns
    (dX, grads) with grads keyed like the weights (biases only if cfg.qkv_bias).
    """
    W = {k: _f64(v) for k, v in W.items()}
    X, dY = _f64(X), _f64(dY)
    T = X.shape[0]
    Hq, Hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    _, c = _layer_forward_full(cfg, W, X, pos0, row_block)
    G: Dict[str, np.ndarray] = {}
    # MLP
    dm = dY @ W["w_down"]
    G["w_down"] = dY.T @ c["m"]
    du = dm * silu(c["g"])
    dg = dm * c["u"] * silu_grad(c["g"])
    G["w_gate"] = dg.T @ c["h2"]
    G["w_up"] = du.T @ c["h2"]
    dh2 = dg @ W["w_gate"] + du @ W["w_up"]
    dr_norm, G["g2"] = rmsnorm_backward(dh2, c["xhat2"], c["rms2"], W["g2"])
    dr = dY + dr_norm
    # attention output projection
    G["wo"] = dr.T @ c["o"]
    do = (dr @ W["wo"]).reshape(T, Hq, dh)
    dqr, dkr, dvh = attention_backward(c["qr"], c["kr"], c["vh"], do, row_block)
    dq = rope_apply_transpose(dqr, c["cos"], c["sin"]).reshape(T, Hq * dh)
    dk = rope_apply_transpose(dkr, c["cos"], c["sin"]).reshape(T, Hkv * dh)
    dv = dvh.reshape(T, Hkv * dh)
    G["wq"] = dq.T @ c["h1"]
    G["wk"] = dk.T @ c["h1"]
    G["wv"] = dv.T @ c["h1"]
    if cfg.qkv_bias:
        G["bq"], G["bk"], G["bv"] = dq.sum(0), dk.sum(0), dv.sum(0)
    dh1 = dq @ W["wq"] + dk @ W["wk"] + dv @ W["wv"]
    dx_norm, G["g1"] = rmsnorm_backward(dh1, c["xhat1"], c["rms1"], W["g1"])
    dX = dr + dx_norm
    return dX, G


def layer_backward_packed(cfg: LayerCfg, W, X, dY, cu_seqlens, pos0=0, row_block=1024):
    """A packed batch is a set of independent sequences that share the weights: the input gradient of
    each sequence is that of the sequence alone, the weight gradients are the sums over the sequences."""
    X, dY = _f64(X), _f64(dY)
    dX = np.empty_like(X)
    G: Dict[str, np.ndarray] = {}
    for a, e in zip(cu_seqlens[:-1], cu_seqlens[1:]):
        dX[a:e], Gi = layer_backward(cfg, W, X[a:e], dY[a:e], pos0=pos0, row_block=row_block)
        for k, v in Gi.items():
            G[k] = v if k not in G else G[k] + v
    return dX, G


# ---------------------------------------------------------------------------
# LM head + cross-entropy (SFT objective of Sec. 3.2.1, normalised by the number
# of unmasked labels)
# ---------------------------------------------------------------------------

def lmhead_ce_forward(cfg: HeadCfg, g_final, w_vocab, H, labels, row_block=512):
    """Mean over unmasked rows of logsumexp(z_t) - z_t[y_t], z = RMSNorm(H) W_vocab^T."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    labels = np.asarray(labels, dtype=np.int64)
    valid = labels != cfg.ignore_index
    N = int(valid.sum())
    if N == 0:
        return 0.0, 0
    total = 0.0
    for t0 in range(0, H.shape[0], row_block):
        t1 = min(H.shape[0], t0 + row_block)
        hn, _, _ = rmsnorm_forward(H[t0:t1], g_final, cfg.rms_eps)
        z = hn @ w_vocab.T
        zmax = z.max(axis=-1, keepdims=True)
        lse = zmax[:, 0] + np.log(np.exp(z - zmax).sum(axis=-1))
        vb = valid[t0:t1]
        idx = np.nonzero(vb)[0]
        total += float(np.sum(lse[idx] - z[idx, labels[t0:t1][idx]]))
    return total / N, N


def lmhead_ce_backward(cfg: HeadCfg, g_final, w_vocab, H, labels, row_block=512):
    """Returns (loss, N, dH, dW_vocab, dg_final) for the mean cross-entropy."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    labels = np.asarray(labels, dtype=np.int64)
    T = H.shape[0]
    valid = labels != cfg.ignore_index
    N = int(valid.sum())
    dH = np.zeros_like(H)
    dW = np.zeros_like(w_vocab)
    dg = np.zeros_like(g_final)
    if N == 0:
        return 0.0, 0, dH, dW, dg
    total = 0.0
    for t0 in range(0, T, row_block):
        t1 = min(T, t0 + row_block)
        hn, xhat, rms = rmsnorm_forward(H[t0:t1], g_final, cfg.rms_eps)
        z = hn @ w_vocab.T
        zmax = z.max(axis=-1, keepdims=True)
        e = np.exp(z - zmax)
        se = e.sum(axis=-1, keepdims=True)
        lse = zmax[:, 0] + np.log(se[:, 0])
        idx = np.nonzero(valid[t0:t1])[0]
        yl = labels[t0:t1][idx]
        total += float(np.sum(lse[idx] - z[idx, yl]))
        dz = e / se
        dz[idx, yl] -= 1.0
        dz[~valid[t0:t1]] = 0.0
        dz /= N
        dW += dz.T @ hn
        dhn = dz @ w_vocab
        dH[t0:t1], dgi = rmsnorm_backward(dhn, xhat, rms, g_final)
        dg += dgi
    return total / N, N, dH, dW, dg


# ---------------------------------------------------------------------------
# LM head under the RL objectives of Sec. 3.2.1 (GRPO Eq. (4), DPO Eq. (5)).
# Both depend on the logits only through log pi_theta(t) = z_t[o_t] - logsumexp(z_t) of the given
# token o_t, so the gradient wrt the logits of row t is c_t * (e_{o_t} - softmax(z_t)) with a
# per-token coefficient c_t = dL / dlog pi_theta(t).  Rows whose token equals ignore_index do not
# take part.
# ---------------------------------------------------------------------------

def _token_logprobs(cfg: HeadCfg, g_final, w_vocab, H, tokens, row_block):
    """log softmax(RMSNorm(H) W^T)[t, tokens[t]] for rows that take part (0 elsewhere)."""
    T = H.shape[0]
    part = tokens != cfg.ignore_index
    logp = np.zeros(T)
    for t0 in range(0, T, row_block):
        t1 = min(T, t0 + row_block)
        hn, _, _ = rmsnorm_forward(H[t0:t1], g_final, cfg.rms_eps)
        z = hn @ w_vocab.T
        zmax = z.max(axis=-1, keepdims=True)
        lse = zmax[:, 0] + np.log(np.exp(z - zmax).sum(axis=-1))
        idx = np.nonzero(part[t0:t1])[0]
        logp[t0 + idx] = z[idx, tokens[t0:t1][idx]] - lse[idx]
    return logp


def _backprop_token_coefficients(cfg: HeadCfg, g_final, w_vocab, H, tokens, coef, row_block):
    """Given c_t = dL/dlog pi(t), returns (dH, dW_vocab, dg_final): dz_t = c_t (e_{o_t} - softmax(z_t))."""
    T = H.shape[0]
    part = tokens != cfg.ignore_index
    dH, dW, dg = np.zeros_like(H), np.zeros_like(w_vocab), np.zeros_like(g_final)
    for t0 in range(0, T, row_block):
        t1 = min(T, t0 + row_block)
        hn, xhat, rms = rmsnorm_forward(H[t0:t1], g_final, cfg.rms_eps)
        z = hn @ w_vocab.T
        z = z - z.max(axis=-1, keepdims=True)
        p = np.exp(z)
        p /= p.sum(axis=-1, keepdims=True)
        dz = -p
        idx = np.nonzero(part[t0:t1])[0]
        dz[idx, tokens[t0:t1][idx]] += 1.0
        dz *= np.where(part[t0:t1], coef[t0:t1], 0.0)[:, None]
        dW += dz.T @ hn
        dH[t0:t1], dgi = rmsnorm_backward(dz @ w_vocab, xhat, rms, g_final)
        dg += dgi
    return dH, dW, dg


def grpo_token_terms(logp, logp_old, logp_ref, advantage, beta, clip_eps):
    """f(t) of Eq. (4) and df/dlog pi_theta(t):
    f = min(r A, clip(r, 1-eps, 1+eps) A) - beta (log pi_theta - log pi_ref), r = pi_theta / pi_old.

    The min / clip is a branch; it is decided here, in float64, from this function's own arguments only.
    A comparison with a lower-precision implementation is meaningful for tokens whose ratio keeps a margin
    from 1 +- eps (see `grpo_branch_margin`): the caller builds its inputs that way."""
    r = np.exp(logp - logp_old)
    unclipped = r * advantage
    clipped = np.clip(r, 1.0 - clip_eps, 1.0 + clip_eps) * advantage
    inside = (r > 1.0 - clip_eps) & (r < 1.0 + clip_eps)
    takes_unclipped = unclipped <= clipped
    # d(r A)/dlog pi = r A; the clipped branch is constant in log pi wherever the clip is active
    keeps = takes_unclipped | inside
    f = np.where(keeps, unclipped, clipped) - beta * (logp - logp_ref)
    df = np.where(keeps, unclipped, 0.0) - beta
    return f, df


def grpo_branch_margin(logp, logp_old, clip_eps):
    """Per token, the distance in log pi_theta to the nearest point where the min / clip branch of Eq. (4)
    changes: |log r - log(1 - eps)| and |log r - log(1 + eps)| (the only places where the derivative of
    min(r A, clip(r) A) jumps for A != 0).  An implementation whose log-probabilities are within less than
    this margin of the exact ones takes the same branch."""
    x = _f64(logp) - _f64(logp_old)
    return np.minimum(np.abs(x - np.log1p(-clip_eps)), np.abs(x - np.log1p(clip_eps)))


def lmhead_grpo_forward(cfg: HeadCfg, g_final, w_vocab, H, tokens, logp_old, logp_ref, advantage, weight,
                        beta, clip_eps, row_block=512):
    """L = - sum_t weight_t f(t); weight_t carries the 1/(G T_o) of Eq. (4)."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    tokens = np.asarray(tokens, dtype=np.int64)
    part = tokens != cfg.ignore_index
    logp = _token_logprobs(cfg, g_final, w_vocab, H, tokens, row_block)
    f, _ = grpo_token_terms(logp, _f64(logp_old), _f64(logp_ref), _f64(advantage), beta, clip_eps)
    return float(-np.sum(np.where(part, _f64(weight) * f, 0.0)))


def lmhead_grpo_backward(cfg: HeadCfg, g_final, w_vocab, H, tokens, logp_old, logp_ref, advantage, weight,
                         beta, clip_eps, row_block=512):
    """Returns (loss, logp, dH, dW_vocab, dg_final) for the GRPO objective."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    tokens = np.asarray(tokens, dtype=np.int64)
    part = tokens != cfg.ignore_index
    logp = _token_logprobs(cfg, g_final, w_vocab, H, tokens, row_block)
    f, df = grpo_token_terms(logp, _f64(logp_old), _f64(logp_ref), _f64(advantage), beta, clip_eps)
    w = _f64(weight)
    loss = float(-np.sum(np.where(part, w * f, 0.0)))
    dH, dW, dg = _backprop_token_coefficients(cfg, g_final, w_vocab, H, tokens, -w * df, row_block)
    return loss, logp, dH, dW, dg


def lmhead_dpo_forward(cfg: HeadCfg, g_final, w_vocab, H, tokens, logp_ref, sign, beta, row_block=512):
    """L = -log sigmoid(beta * ell), ell = sum_t sign_t (log pi_theta(t) - log pi_ref(t)) with sign +1 on the
    chosen response's tokens and -1 on the rejected one's (Eq. (5))."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    tokens = np.asarray(tokens, dtype=np.int64)
    part = tokens != cfg.ignore_index
    logp = _token_logprobs(cfg, g_final, w_vocab, H, tokens, row_block)
    ell = float(np.sum(np.where(part, _f64(sign) * (logp - _f64(logp_ref)), 0.0)))
    return float(np.log1p(np.exp(-beta * ell))), ell


def lmhead_dpo_backward(cfg: HeadCfg, g_final, w_vocab, H, tokens, logp_ref, sign, beta, row_block=512):
    """Returns (loss, ell, dH, dW_vocab, dg_final): dL/dlog pi(t) = (sigmoid(beta ell) - 1) beta sign_t (Eq. (6))."""
    g_final, w_vocab, H = _f64(g_final), _f64(w_vocab), _f64(H)
    tokens = np.asarray(tokens, dtype=np.int64)
    loss, ell = lmhead_dpo_forward(cfg, g_final, w_vocab, H, tokens, logp_ref, sign, beta, row_block)
    factor = 1.0 / (1.0 + np.exp(-beta * ell)) - 1.0
    dH, dW, dg = _backprop_token_coefficients(cfg, g_final, w_vocab, H, tokens, factor * beta * _f64(sign), row_block)
    return loss, ell, dH, dW, dg


# ---------------------------------------------------------------------------
# Whole model: embedding -> L layers -> head
# ---------------------------------------------------------------------------

def model_forward_loss(layer_cfg: LayerCfg, head_cfg: HeadCfg, layers: List[Dict], g_final, w_vocab,
                       labels, embed=None, ids=None, X0=None, row_block=1024):
    X = _f64(embed)[np.asarray(ids)] if ids is not None else _f64(X0)
    for W in layers:
        X = layer_forward(layer_cfg, W, X, 0, row_block)
    return lmhead_ce_forward(head_cfg, g_final, w_vocab, X, labels)[0]


def model_backward(layer_cfg: LayerCfg, head_cfg: HeadCfg, layers: List[Dict], g_final, w_vocab,
                   labels, embed=None, ids=None, X0=None, row_block=1024):
    """Returns dict(loss, n_valid, d_embed or None, layers=[grads...], g_final, w_vocab, dX0)."""
    X = _f64(embed)[np.asarray(ids)] if ids is not None else _f64(X0)
    inputs = []
    for W in layers:
        inputs.append(X)
        X = layer_forward(layer_cfg, W, X, 0, row_block)
    loss, N, dX, dWv, dgf = lmhead_ce_backward(head_cfg, g_final, w_vocab, X, labels)
    layer_grads: List[Optional[Dict]] = [None] * len(layers)
    for l in range(len(layers) - 1, -1, -1):
        dX, layer_grads[l] = layer_backward(layer_cfg, layers[l], inputs[l], dX, 0, row_block)
    d_embed = None
    if ids is not None:
        d_embed = np.zeros_like(_f64(embed))
        np.add.at(d_embed, np.asarray(ids), dX)
    return dict(loss=loss, n_valid=N, d_embed=d_embed, layers=layer_grads, g_final=dgf, w_vocab=dWv, dX0=dX)


# ---------------------------------------------------------------------------
# Error metrics
# ---------------------------------------------------------------------------

def rel_frobenius(a, ref):
    """||a - ref||_F / ||ref||_F (0 when both vanish)."""
    a, ref = _f64(a), _f64(ref)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(a - ref)
    if den == 0.0:
        return 0.0 if num == 0.0 else np.inf
    return float(num / den)


def paper_errors(a, ref):
    """The two error measures of the paper's correctness table (App. B.1):
    mean |ref - a| and mean |ref - a| / |ref + 1e-10|."""
    a, ref = _f64(a), _f64(ref)
    d = np.abs(ref - a)
    return float(d.mean()), float((d / np.abs(ref + 1e-10)).mean())
