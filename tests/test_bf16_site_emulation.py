"""Which bf16 roundings carry the error of the model's gradients against an un-rounded run (CPU, small widths).

The GPU path at the full model widths misses the 2e-2 stated for bf16 runs on the softmax-path gradients of the last
layer (2.5e-2; tests/test_gpu_model.py bounds them by a documented 3e-2).  The emulation in bf16_site_emulation.py
(run as a script for the full widths: it reproduces 2.47e-2) attributes that error site by site.  Here its structure
is pinned at widths the CPU suite can afford:
  * the emulation with no site on is an exact model (it agrees with the oracle);
  * rounding only what is NOT an operand of a tensor-core product (checkpoints, inter-layer gradients, delta from the
    rounded O / dO) explains a small part of the error; rounding only the operands explains nearly all of it;
  * the softmax-path gradients (W_q, W_k) are the most sensitive ones, and the most sensitive site is the normalised
    activation that feeds the Q / K / V products -- an operand of the configuration's bf16 products (at the full widths
    the rotated Q / K come second: 1.38e-2 and 1.24e-2 of the 2.47e-2).
"""
import numpy as np
import torch

import bf16_site_emulation as E
from oracle import streambp_oracle as O
from paper_2506_03077_b200 import synth


def small_case():
    s = synth.LayerShape(256, 4, 2, 64, 688, True, 1e6)
    hs = synth.HeadShape(256, 4096)
    return s, hs, E.build_case(s, hs, 4, 192, 2, hs.vocab)


def test_emulation_without_rounding_is_the_model():
    s, hs, case = small_case()
    layers, Emb, gf, Wv, ids, labels = case
    got = E.model(E.Emu([]), s, hs, *case)
    ref = O.model_backward(O.LayerCfg(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta,
                                      s.rms_eps), O.HeadCfg(hs.d_model, hs.vocab),
                           [{k: v.numpy() for k, v in W.items()} for W in layers], gf.numpy(), Wv.numpy(), labels.numpy(),
                           embed=Emb.numpy(), ids=ids.numpy())
    assert O.rel_frobenius(got["w_vocab"].numpy(), ref["w_vocab"]) < 2e-5
    for l in (0, 1):
        for k in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g1", "g2", "bq", "bk", "bv"):
            assert O.rel_frobenius(got[f"L{l}.{k}"].numpy(), ref["layers"][l][k]) < 5e-5, (l, k)


def test_operand_roundings_carry_the_error():
    s, hs, case = small_case()
    exact = E.model(E.Emu([]), s, hs, *case)
    keys = ["w_vocab", "L0.wq", "L1.wq", "L1.wk", "L1.w_down"]
    err = lambda sites: E.errors(s, hs, case, sites, exact, keys)
    full, operands, storage = err(E.ALL), err(E.OPERAND_SITES), err(E.STORAGE_SITES)
    for k in keys:
        assert operands[k] > 0.85 * full[k], (k, operands[k], full[k])      # operands alone: nearly all of it
        assert storage[k] < 0.5 * full[k], (k, storage[k], full[k])         # everything avoidable: the small part
    # in quadrature the two parts make up the whole (independent roundings)
    for k in keys:
        assert abs(np.hypot(operands[k], storage[k]) / full[k] - 1.0) < 0.15, k
    # delta from the rounded O, dO instead of sum_s P dP changes nothing measurable
    assert max(err(["delta_bf"]).values()) < 1e-5
    # the softmax path is the sensitive one, and its largest single contributor is an operand of the forward pass:
    # the normalised activations that feed the Q / K / V products (at the full widths the rotated Q / K come second)
    assert full["L1.wq"] > full["L1.w_down"]
    single = {site: err([site])["L1.wq"] for site in ("h1", "qk", "ckpt", "ds", "dq", "gu", "o", "v", "p")}
    assert single["h1"] == max(single.values())
