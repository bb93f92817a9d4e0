"""Pins for the oracle's GRPO and DPO LM-head objectives (Sec. 3.2.1): finite differences, an independent
PyTorch-autograd statement, and closed-form special cases."""
import numpy as np
import torch
import torch.nn.functional as F

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import synth


def setup(seed, T=23, d=12, V=37, masked=5):
    cfg = O.HeadCfg(d, V, 1e-6, -100)
    g = synth.normal(seed, "g", (d,), 1.0, 0.1).astype(np.float64)
    W = synth.normal(seed, "w", (V, d), 0.0, 0.4).astype(np.float64)
    H = synth.normal(seed, "H", (T, d)).astype(np.float64)
    tok = synth.integers(seed, "tok", (T,), V)
    tok[:masked] = -100
    tok[11] = -100
    lp = O._token_logprobs(cfg, g, W, H, tok, 7)
    old = lp + synth.normal(seed, "old", (T,), 0.0, 0.25)        # ratios on both sides of the clip range
    ref = lp + synth.normal(seed, "ref", (T,), 0.0, 0.3)
    adv = synth.normal(seed, "adv", (T,)).astype(np.float64)
    wt = np.full(T, 1.0 / (T - masked - 1))
    return cfg, g, W, H, tok, old.astype(np.float64), ref.astype(np.float64), adv, wt


def fd(f, x, u, h=1e-6):
    return (f(x + h * u) - f(x - h * u)) / (2 * h)


def test_grpo_matches_finite_differences_and_visits_every_branch():
    cfg, g, W, H, tok, old, ref, adv, wt = setup(3)
    beta, eps = 0.04, 0.2
    loss, logp, dH, dW, dg = O.lmhead_grpo_backward(cfg, g, W, H, tok, old, ref, adv, wt, beta, eps, row_block=6)
    r = np.exp(logp - old)[tok != -100]
    a = adv[tok != -100]
    # the four (clip side, advantage sign) cases must all occur, else the test proves little
    assert ((r > 1 + eps) & (a > 0)).any() and ((r > 1 + eps) & (a < 0)).any()
    assert ((r < 1 - eps) & (a > 0)).any() and ((r < 1 - eps) & (a < 0)).any()
    assert abs(loss - O.lmhead_grpo_forward(cfg, g, W, H, tok, old, ref, adv, wt, beta, eps)) < 1e-14
    for name, val, grad, f in (
            ("H", H, dH, lambda v: O.lmhead_grpo_forward(cfg, g, W, v, tok, old, ref, adv, wt, beta, eps)),
            ("W", W, dW, lambda v: O.lmhead_grpo_forward(cfg, g, v, H, tok, old, ref, adv, wt, beta, eps)),
            ("g", g, dg, lambda v: O.lmhead_grpo_forward(cfg, v, W, H, tok, old, ref, adv, wt, beta, eps))):
        u = synth.normal(9, "dir" + name, val.shape).astype(np.float64)
        num, an = fd(f, val, u), float(np.sum(grad * u))
        assert abs(num - an) <= 1e-6 * max(abs(num), abs(an)) + 1e-10, (name, num, an)
    assert np.all(dH[:5] == 0.0) and np.all(dH[11] == 0.0)


def test_dpo_matches_finite_differences():
    cfg, g, W, H, tok, old, ref, adv, wt = setup(4)
    sign = np.where(np.arange(len(tok)) < 14, 1.0, -1.0)
    beta = 0.3
    loss, ell, dH, dW, dg = O.lmhead_dpo_backward(cfg, g, W, H, tok, ref, sign, beta, row_block=5)
    for name, val, grad, f in (
            ("H", H, dH, lambda v: O.lmhead_dpo_forward(cfg, g, W, v, tok, ref, sign, beta)[0]),
            ("W", W, dW, lambda v: O.lmhead_dpo_forward(cfg, g, v, H, tok, ref, sign, beta)[0]),
            ("g", g, dg, lambda v: O.lmhead_dpo_forward(cfg, v, W, H, tok, ref, sign, beta)[0])):
        u = synth.normal(8, "dir" + name, val.shape).astype(np.float64)
        num, an = fd(f, val, u), float(np.sum(grad * u))
        assert abs(num - an) <= 1e-6 * max(abs(num), abs(an)) + 1e-10, (name, num, an)


def torch_logp(g, W, H, tok):
    hn = H * torch.rsqrt(H.pow(2).mean(-1, keepdim=True) + 1e-6) * g
    logits = F.linear(hn, W)
    idx = torch.tensor(np.where(tok < 0, 0, tok))
    return torch.log_softmax(logits, dim=-1).gather(1, idx[:, None])[:, 0]


def test_grpo_and_dpo_match_autograd():
    cfg, g, W, H, tok, old, ref, adv, wt = setup(5)
    part = torch.tensor(tok != -100)
    tg, tW, tH = (torch.tensor(a, requires_grad=True) for a in (g, W, H))
    lp = torch_logp(tg, tW, tH, tok)
    r = torch.exp(lp - torch.tensor(old))
    A = torch.tensor(adv)
    f = torch.minimum(r * A, torch.clamp(r, 0.8, 1.2) * A) - 0.04 * (lp - torch.tensor(ref))
    loss = -(torch.tensor(wt) * f)[part].sum()
    loss.backward()
    o = O.lmhead_grpo_backward(cfg, g, W, H, tok, old, ref, adv, wt, 0.04, 0.2)
    assert abs(o[0] - loss.item()) < 1e-13
    assert O.rel_frobenius(o[2], tH.grad.numpy()) < 1e-12
    assert O.rel_frobenius(o[3], tW.grad.numpy()) < 1e-12
    assert O.rel_frobenius(o[4], tg.grad.numpy()) < 1e-12
    # DPO
    sign = np.where(np.arange(len(tok)) % 2 == 0, 1.0, -1.0)
    tg, tW, tH = (torch.tensor(a, requires_grad=True) for a in (g, W, H))
    lp = torch_logp(tg, tW, tH, tok)
    ell = (torch.tensor(sign) * (lp - torch.tensor(ref)))[part].sum()
    loss = -F.logsigmoid(0.3 * ell)
    loss.backward()
    o = O.lmhead_dpo_backward(cfg, g, W, H, tok, ref, sign, 0.3)
    assert abs(o[0] - loss.item()) < 1e-13 and abs(o[1] - ell.item()) < 1e-13
    assert O.rel_frobenius(o[2], tH.grad.numpy()) < 1e-12
    assert O.rel_frobenius(o[3], tW.grad.numpy()) < 1e-12
    assert O.rel_frobenius(o[4], tg.grad.numpy()) < 1e-12


def test_special_cases_reduce_to_cross_entropy():
    cfg, g, W, H, tok, old, ref, adv, wt = setup(6)
    sft = O.lmhead_ce_backward(cfg, g, W, H, tok)
    N = sft[1]
    lp = O._token_logprobs(cfg, g, W, H, tok, 64)
    # GRPO on-policy (pi_old = pi_theta, so r = 1: never clipped), beta = 0, advantage 1, weight 1/N:
    # f = r, df/dlog pi = 1, so the gradient is that of the mean cross-entropy
    o = O.lmhead_grpo_backward(cfg, g, W, H, tok, lp, ref, np.ones_like(adv), np.full(len(tok), 1.0 / N), 0.0, 0.2)
    assert abs(o[0] + 1.0) < 1e-12                               # L = -sum w * 1
    for a, b in zip(o[2:], sft[2:]):
        assert O.rel_frobenius(a, b) < 1e-12
    # DPO with every token "chosen" and pi_ref = pi_theta: ell = 0, L = ln 2, gradient = -(beta/2) sum_t dlog pi
    d = O.lmhead_dpo_backward(cfg, g, W, H, tok, lp, np.ones(len(tok)), 0.5)
    assert abs(d[0] - np.log(2.0)) < 1e-12 and abs(d[1]) < 1e-12
    for a, b in zip(d[2:], sft[2:]):
        assert O.rel_frobenius(a, 0.25 * N * b) < 1e-12          # (sigma(0) - 1) * beta = -1/4 per token vs -(-1/N)
    # clip is active and selected for every token: no policy-gradient term, only the KL term remains
    far = lp - 1.0                                               # r = e > 1 + eps, positive advantage -> clipped
    o2 = O.lmhead_grpo_backward(cfg, g, W, H, tok, far, ref, np.abs(adv) + 0.1, wt, 0.1, 0.2)
    kl_only = O._backprop_token_coefficients(cfg, g, W, H, tok, 0.1 * wt, 64)
    for a, b in zip(o2[2:], kl_only):
        assert O.rel_frobenius(a, b) < 1e-12


def test_branch_margin_is_the_distance_to_a_change_of_branch():
    # moving one token's log-probability by less than its margin leaves its (f, df) branch unchanged; moving it
    # by more than the margin towards the nearest boundary changes df for a token whose advantage makes the clip bind
    cfg, g, W, H, tok, old, ref, adv, wt = setup(7)
    lp = O._token_logprobs(cfg, g, W, H, tok, 7)
    margin = O.grpo_branch_margin(lp, old, 0.2)
    _, df0 = O.grpo_token_terms(lp, old, ref, adv, 0.04, 0.2)
    r = np.exp(lp - old)
    for t in np.nonzero(tok != -100)[0]:
        for sgn in (-1.0, 1.0):
            near = lp.copy()
            near[t] += sgn * 0.9 * margin[t]
            _, df1 = O.grpo_token_terms(near, old, ref, adv, 0.04, 0.2)
            # same branch: df is either r A - beta on both sides or -beta on both sides
            assert (df1[t] == -0.04) == (df0[t] == -0.04)
    # a token inside the range with positive advantage: crossing 1 + eps switches the policy-gradient term off
    t = int(np.argmax((tok != -100) & (r > 1.0) & (r < 1.2) & (adv > 0)))
    far = lp.copy()
    far[t] = old[t] + np.log(1.2) + 1e-9
    _, df2 = O.grpo_token_terms(far, old, ref, adv, 0.04, 0.2)
    assert df0[t] != -0.04 and df2[t] == -0.04
    assert abs(margin[t] - (np.log(1.2) - (lp[t] - old[t]))) < 1e-12
