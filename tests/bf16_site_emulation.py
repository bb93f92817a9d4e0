"""Numerical emulation of where the CUDA path rounds to bf16 -- TEST INFRASTRUCTURE ONLY.

A restatement of the model's forward and backward in plain PyTorch CPU float32 in which every place where the CUDA
path stores or feeds a bf16 value is a named SITE that can be switched on alone or left out.  It answers one
question the oracle cannot: which of those roundings carry the error of a gradient against an un-rounded run.  It is
neither the oracle (fp64, no rounding, plain definition) nor the product; it shares code with neither.

Sites: ckpt (layer-input checkpoints), h1, qk (rotated Q and K), v, p (probabilities as a product operand), o, h2,
gu (gate / up), m, hn, dz, dH / dX (inter-layer gradients), dm, dgdu, dr, dO, ds, dq, dkv, delta_bf (delta taken from
the rounded O and dO instead of sum_s P dP).  OPERAND_SITES are operands of a tensor-core product (what "bf16 with
fp32 accumulation" means); STORAGE_SITES are roundings an implementation could avoid without changing that.

    python tests/bf16_site_emulation.py          # the full widths of the model configuration, 2 layers x 1024
                                                 # tokens: about ten minutes of CPU and 30 GB of memory
"""
import json
import math
import os
import sys
import time

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
import numpy as np
import torch

from paper_2506_03077_b200 import synth

F = torch.float32

ALL = ["ckpt", "h1", "qk", "v", "p", "o", "h2", "gu", "m", "hn", "dz", "dH", "dm", "dgdu", "dr", "dO", "ds", "dq", "dkv", "dX",
       "delta_bf"]
STORAGE_SITES = ["ckpt", "dH", "dX", "delta_bf"]
OPERAND_SITES = [x for x in ALL if x not in STORAGE_SITES]
class Emu:
    def __init__(self, sites):
        self.sites = set(sites)
    def r(self, site, x):
        return x.bfloat16().to(F) if site in self.sites else x

def rms_fwd(x, g, eps=1e-6):
    rms = torch.sqrt((x * x).mean(-1, keepdim=True) + eps)
    xh = x / rms
    return xh * g, xh, rms
def rms_bwd(dh, xh, rms, g):
    w = dh * g
    return (w - xh * (w * xh).mean(-1, keepdim=True)) / rms, (dh * xh).sum(0)
def rope(u, cos, sin, tr=False):
    half = u.shape[-1] // 2
    a, b = u[..., :half], u[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    if tr: s = -s
    return torch.cat([a * c - b * s, b * c + a * s], -1)

def layer_fwd(E, s, W, X, cos, sin):
    T = X.shape[0]; Hq, Hkv, dh = s.n_q_heads, s.n_kv_heads, s.head_dim; G = Hq // Hkv
    h1, xh1, rms1 = rms_fwd(X, W["g1"]); h1 = E.r("h1", h1)
    q = h1 @ W["wq"].T + W["bq"]; k = h1 @ W["wk"].T + W["bk"]; v = h1 @ W["wv"].T + W["bv"]
    qr = E.r("qk", rope(q.view(T, Hq, dh), cos, sin)); kr = E.r("qk", rope(k.view(T, Hkv, dh), cos, sin)); vh = E.r("v", v.view(T, Hkv, dh))
    kx = kr.repeat_interleave(G, 1); vx = vh.repeat_interleave(G, 1)
    S = torch.einsum("thd,shd->hts", qr, kx) / math.sqrt(dh)
    mask = torch.ones(T, T, dtype=torch.bool).tril()
    S = S.masked_fill(~mask, float("-inf"))
    lse = torch.logsumexp(S, -1, keepdim=True)
    P = torch.exp(S - lse)
    l = P.sum(-1, keepdim=True)  # = 1; the kernel divides the fp32 row sum of UNROUNDED p
    o = torch.einsum("hts,shd->thd", E.r("p", P), vx)
    o = E.r("o", o.reshape(T, Hq * dh))
    r = X + o @ W["wo"].T
    h2, xh2, rms2 = rms_fwd(r, W["g2"]); h2 = E.r("h2", h2)
    g = E.r("gu", h2 @ W["w_gate"].T); u = E.r("gu", h2 @ W["w_up"].T)
    m = E.r("m", torch.nn.functional.silu(g) * u)
    y = r + m @ W["w_down"].T
    c = dict(h1=h1, xh1=xh1, rms1=rms1, qr=qr, kr=kr, vh=vh, P=P, o=o, r=r, xh2=xh2, rms2=rms2, h2=h2, g=g, u=u, m=m)
    return y, c

def layer_bwd(E, s, W, X, dY, cos, sin):
    T = X.shape[0]; Hq, Hkv, dh = s.n_q_heads, s.n_kv_heads, s.head_dim; G = Hq // Hkv
    _, c = layer_fwd(E, s, W, X, cos, sin)
    Gd = {}
    dm = E.r("dm", dY @ W["w_down"])
    Gd["w_down"] = dY.T @ c["m"]
    sg = torch.sigmoid(c["g"])
    du = E.r("dgdu", dm * c["g"] * sg); dg = E.r("dgdu", dm * c["u"] * sg * (1 + c["g"] * (1 - sg)))
    Gd["w_gate"] = dg.T @ c["h2"]; Gd["w_up"] = du.T @ c["h2"]
    dh2 = dg @ W["w_gate"] + du @ W["w_up"]
    drn, Gd["g2"] = rms_bwd(dh2, c["xh2"], c["rms2"], W["g2"])
    dr = dY + drn
    dr_s = E.r("dr", dr)
    Gd["wo"] = dr_s.T @ c["o"]
    dO = E.r("dO", dr_s @ W["wo"]).view(T, Hq, dh)
    P = c["P"]
    kx = c["kr"].repeat_interleave(G, 1); vx = c["vh"].repeat_interleave(G, 1)
    o3 = c["o"].view(T, Hq, dh)
    dP = torch.einsum("thd,shd->hts", dO, vx)
    if "delta_bf" in E.sites:   # as the kernels do: from the stored (rounded) O and dO
        delta = (dO * o3).sum(-1).T[:, :, None]
    else:                        # consistent with the probabilities actually used
        delta = (P * dP).sum(-1, keepdim=True)
    dS = P * (dP - delta) / math.sqrt(dh)
    dSr = E.r("ds", dS)
    Pr = E.r("p", P)
    dvx = torch.einsum("hts,thd->shd", Pr, dO)
    dqr = torch.einsum("hts,shd->thd", dSr, kx)
    dkx = torch.einsum("hts,thd->shd", dSr, c["qr"])
    dkr = dkx.view(T, Hkv, G, dh).sum(2); dvh = dvx.view(T, Hkv, G, dh).sum(2)
    dq = E.r("dq", rope(dqr, cos, sin, True).reshape(T, Hq * dh))
    dk = E.r("dkv", rope(dkr, cos, sin, True).reshape(T, Hkv * dh)); dv = E.r("dkv", dvh.reshape(T, Hkv * dh))
    Gd["wq"] = dq.T @ c["h1"]; Gd["wk"] = dk.T @ c["h1"]; Gd["wv"] = dv.T @ c["h1"]
    Gd["bq"], Gd["bk"], Gd["bv"] = dq.sum(0), dk.sum(0), dv.sum(0)
    dh1 = dq @ W["wq"] + dk @ W["wk"] + dv @ W["wv"]
    dxn, Gd["g1"] = rms_bwd(dh1, c["xh1"], c["rms1"], W["g1"])
    return dr + dxn, Gd

def model(E, s, hshape, layers, Emb, gf, Wv, ids, labels):
    T = ids.shape[0]
    j = torch.arange(s.head_dim // 2, dtype=torch.float64)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * torch.pow(torch.tensor(s.rope_theta, dtype=torch.float64), -2 * j / s.head_dim)[None]
    cos, sin = torch.cos(ang).to(F), torch.sin(ang).to(F)
    X = Emb[ids]
    inputs = []
    for W in layers:
        X = E.r("ckpt", X)
        inputs.append(X)
        X, _ = layer_fwd(E, s, W, X, cos, sin)
    X = E.r("ckpt", X)
    hn, xh, rms = rms_fwd(X, gf); hnr = E.r("hn", hn)
    z = hnr @ Wv.T
    valid = labels != -100
    N = int(valid.sum())
    p = torch.softmax(z, -1)
    dz = p.clone()
    idx = torch.nonzero(valid)[:, 0]
    dz[idx, labels[idx]] -= 1
    dz[~valid] = 0
    dz = E.r("dz", dz / N)
    dWv = dz.T @ hnr
    dhn = dz @ Wv
    dH, dgf = rms_bwd(dhn, xh, rms, gf)
    dX = E.r("dH", dH)
    out = {"w_vocab": dWv, "g_final": dgf}
    for l in range(len(layers) - 1, -1, -1):
        dX, Gd = layer_bwd(E, s, layers[l], inputs[l], dX, cos, sin)
        dX = E.r("dX", dX)
        for k, v in Gd.items(): out[f"L{l}.{k}"] = v
    return out



def build_case(s, hs, seed, T, L, V):
    tt = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(F)
    layers = [{k: tt(v) for k, v in synth.make_layer_weights(s, seed, True, prefix=f"layer{l}").items()} for l in range(L)]
    Emb = tt(synth.round_bf16(synth.normal(seed, "embed", (V, s.d_model), 0.0, 0.02)))
    gf = tt(synth.round_bf16(synth.normal(seed, "g_final", (s.d_model,), 1.0, 0.02)))
    Wv = tt(synth.round_bf16(synth.normal(seed, "w_vocab", (V, s.d_model), 0.0, 0.02)))
    ids, labels = synth.make_model_tokens(V, seed, T, 0.1)
    return layers, Emb, gf, Wv, torch.from_numpy(ids), torch.from_numpy(labels)


def errors(s, hs, case, sites, exact, keys):
    got = model(Emu(sites), s, hs, *case)
    return {k: float((got[k] - exact[k]).norm() / exact[k].norm()) for k in keys}


def main():
    c = synth.CONFIGS["qwen7b_model"]
    s, hs = c.layer, c.head
    T = int(os.environ.get("EMU_T", 1024)); L = int(os.environ.get("EMU_L", 2)); V = int(os.environ.get("EMU_V", hs.vocab))
    case = build_case(s, hs, c.seed, T, L, V)
    t = time.time()
    exact = model(Emu([]), s, hs, *case)
    print("un-rounded run", round(time.time() - t, 1), "s", flush=True)
    keys = ["w_vocab"] + [f"L{l}.{k}" for l in (0, L - 1) for k in ("wq", "wk", "bq", "g1", "wv", "wo", "w_down", "w_gate")]
    def report(name, sites):
        e = errors(s, hs, case, sites, exact, keys)
        print(f"{name:28s}", " ".join(f"{k}={v:.2e}" for k, v in e.items()), flush=True)
    report("all sites", ALL)
    report("operand sites only", OPERAND_SITES)
    report("storage sites only", STORAGE_SITES)
    for site in ALL:
        report("only " + site, [site])


if __name__ == "__main__":
    main()
