"""Second opinion on the oracle: the same layer and loss stated with PyTorch CPU
float64 library ops (scaled_dot_product_attention, cross_entropy, silu) and
differentiated by autograd.  Nothing here calls or copies the oracle's formulas.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import synth


def torch_rmsnorm(x, g, eps):
    return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + eps) * g


def torch_rope(u, pos, theta):
    # u: [T, H, dh]; library-style rotate_half formulation
    dh = u.shape[-1]
    inv = theta ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = pos.to(torch.float64)[:, None] * inv[None, :]
    emb = torch.cat([ang, ang], dim=-1)
    cos, sin = emb.cos()[:, None, :], emb.sin()[:, None, :]
    rot = torch.cat([-u[..., dh // 2:], u[..., : dh // 2]], dim=-1)
    return u * cos + rot * sin


def torch_layer(cfg, W, X, pos0):
    T = X.shape[0]
    Hq, Hkv, dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    h1 = torch_rmsnorm(X, W["g1"], cfg.rms_eps)
    q = F.linear(h1, W["wq"], W.get("bq")).view(T, Hq, dh)
    k = F.linear(h1, W["wk"], W.get("bk")).view(T, Hkv, dh)
    v = F.linear(h1, W["wv"], W.get("bv")).view(T, Hkv, dh)
    pos = pos0 + torch.arange(T)
    q, k = torch_rope(q, pos, cfg.rope_theta), torch_rope(k, pos, cfg.rope_theta)
    rep = Hq // Hkv
    k = k.repeat_interleave(rep, dim=1)
    v = v.repeat_interleave(rep, dim=1)
    o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None],
                                       v.transpose(0, 1)[None], is_causal=True)[0]
    o = o.transpose(0, 1).reshape(T, Hq * dh)
    r = X + F.linear(o, W["wo"])
    h2 = torch_rmsnorm(r, W["g2"], cfg.rms_eps)
    m = F.silu(F.linear(h2, W["w_gate"])) * F.linear(h2, W["w_up"])
    return r + F.linear(m, W["w_down"])


def make(cfg, seed, T):
    s = synth.LayerShape(cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff,
                         cfg.qkv_bias, cfg.rope_theta, cfg.rms_eps)
    W = {k: synth.normal(seed, "w." + k, shp, 1.0 if k in ("g1", "g2") else 0.0, 0.2).astype(np.float64)
         for k, shp in synth.layer_weight_shapes(s).items()}
    X = synth.normal(seed, "X", (T, cfg.d_model)).astype(np.float64)
    dY = synth.normal(seed, "dY", (T, cfg.d_model)).astype(np.float64)
    return W, X, dY


@pytest.mark.parametrize("bias,Hq,Hkv,dh,theta,pos0", [
    (False, 4, 2, 16, 1e4, 0), (True, 6, 2, 8, 1e6, 100), (True, 4, 4, 8, 5e5, 7), (False, 4, 1, 8, 1e4, 3)])
def test_layer_matches_autograd(bias, Hq, Hkv, dh, theta, pos0):
    cfg = O.LayerCfg(32, Hq, Hkv, dh, 56, bias, theta, 1e-6)
    T = 33
    W, X, dY = make(cfg, 10 + Hq, T)
    tW = {k: torch.tensor(v, requires_grad=True) for k, v in W.items()}
    tX = torch.tensor(X, requires_grad=True)
    Y = torch_layer(cfg, tW, tX, pos0)
    (Y * torch.tensor(dY)).sum().backward()
    assert O.rel_frobenius(O.layer_forward(cfg, W, X, pos0), Y.detach().numpy()) < 1e-13
    dX, G = O.layer_backward(cfg, W, X, dY, pos0=pos0, row_block=8)
    assert O.rel_frobenius(dX, tX.grad.numpy()) < 1e-12
    for k in W:
        assert O.rel_frobenius(G[k], tW[k].grad.numpy()) < 1e-12, k


def test_lmhead_matches_autograd():
    T, d, V = 37, 24, 101
    cfg = O.HeadCfg(d, V, 1e-6, -100)
    g = synth.normal(3, "g", (d,), 1.0, 0.1).astype(np.float64)
    Wv = synth.normal(3, "wv", (V, d), 0.0, 0.3).astype(np.float64)
    H = synth.normal(3, "H", (T, d)).astype(np.float64)
    labels = synth.integers(3, "labels", (T,), V)
    labels[:9] = -100
    labels[20] = -100
    tg, tW, tH = (torch.tensor(a, requires_grad=True) for a in (g, Wv, H))
    loss = F.cross_entropy(F.linear(torch_rmsnorm(tH, tg, 1e-6), tW), torch.tensor(labels),
                           ignore_index=-100, reduction="mean")
    loss.backward()
    l, N, dH, dW, dg = O.lmhead_ce_backward(cfg, g, Wv, H, labels, row_block=8)
    assert N == T - 10
    assert abs(l - loss.item()) < 1e-13
    assert O.rel_frobenius(dH, tH.grad.numpy()) < 1e-12
    assert O.rel_frobenius(dW, tW.grad.numpy()) < 1e-12
    assert O.rel_frobenius(dg, tg.grad.numpy()) < 1e-12


def test_model_matches_autograd():
    lc = O.LayerCfg(16, 4, 2, 4, 24, True, 1e4, 1e-6)
    hc = O.HeadCfg(16, 29, 1e-6, -100)
    T, L = 15, 3
    layers = [make(lc, 40 + l, T)[0] for l in range(L)]
    E = synth.normal(7, "E", (29, 16)).astype(np.float64)
    g = synth.normal(7, "g", (16,), 1.0, 0.1).astype(np.float64)
    Wv = synth.normal(7, "wv", (29, 16), 0.0, 0.3).astype(np.float64)
    ids, labels = synth.make_model_tokens(29, 7, T, 0.3)
    assert labels[-1] == -100 and (labels[:3] == -100).all() and labels[3] == ids[4]
    tl = [{k: torch.tensor(v, requires_grad=True) for k, v in W.items()} for W in layers]
    tE, tg, tW = (torch.tensor(a, requires_grad=True) for a in (E, g, Wv))
    x = tE[torch.tensor(ids)]
    for W in tl:
        x = torch_layer(lc, W, x, 0)
    loss = F.cross_entropy(F.linear(torch_rmsnorm(x, tg, 1e-6), tW), torch.tensor(labels), ignore_index=-100)
    loss.backward()
    res = O.model_backward(lc, hc, layers, g, Wv, labels, embed=E, ids=ids)
    assert abs(res["loss"] - loss.item()) < 1e-12
    assert O.rel_frobenius(res["d_embed"], tE.grad.numpy()) < 1e-11
    assert O.rel_frobenius(res["w_vocab"], tW.grad.numpy()) < 1e-11
    assert O.rel_frobenius(res["g_final"], tg.grad.numpy()) < 1e-11
    for l in range(L):
        for k in layers[l]:
            assert O.rel_frobenius(res["layers"][l][k], tl[l][k].grad.numpy()) < 1e-11, (l, k)
