"""GPU parity: streambp_lmhead_rl_backward (GRPO and DPO objectives, Sec. 3.2.1) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth
from helpers import TOL, assert_close, to_dev

pytestmark = pytest.mark.gpu


# Every GRPO token keeps this distance (in log pi_theta) from the points where the min / clip branch of Eq. (4)
# changes, so the oracle (float64) and the kernel (float32 from bf16 products) take the same branch without
# either side seeing the other's numbers; the kernel's own log-probabilities are checked to be closer than that.
CLIP_EPS = 0.2
BRANCH_MARGIN = 0.08
LOGP_TOL = {torch.float32: 2e-5, torch.bfloat16: 3e-2}


def make_case(seed, T, d, V, dtype, masked):
    bf = dtype == torch.bfloat16
    hs = synth.HeadShape(d, V)
    g, W, H, tok = synth.make_head_inputs(hs, seed, T, bf, masked)
    W = W * 4.0                                   # sharper policies: ratios and clip branches vary more
    if bf:
        W = synth.round_bf16(W)
    cfg = O.HeadCfg(d, V)
    lp = O._token_logprobs(cfg, g.astype(np.float64), W.astype(np.float64), H.astype(np.float64), tok, 256)
    x = -synth.normal(seed, "old", (T,), 0.0, 0.3)              # log r = log pi_theta - log pi_old
    for edge in (np.log1p(-CLIP_EPS), np.log1p(CLIP_EPS)):         # push ratios near a clip edge away from it
        near = np.abs(x - edge) < BRANCH_MARGIN
        x = np.where(near, edge + np.where(x >= edge, 1.0, -1.0) * BRANCH_MARGIN * 1.25, x)
    old = (lp - x).astype(np.float32)
    ref = (lp + synth.normal(seed, "ref", (T,), 0.0, 0.3)).astype(np.float32)
    adv = synth.normal(seed, "adv", (T,)).astype(np.float32)
    return hs, cfg, g, W, H, tok, old, ref, adv


def run_rl(hs, objective, beta, eps, g, W, H, tok, old, ref, adv, wt, chunk, dtype, accumulate=False, check=True,
           wgrad_group=1):
    cfg = B.HeadConfig(hs.d_model, hs.vocab, hs.rms_eps, hs.ignore_index, dtype)
    T = H.shape[0]
    f32 = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    loss = torch.full((1,), float("nan"), device="cuda")
    ell = torch.full((1,), float("nan"), device="cuda")
    logp = torch.full((T,), float("nan"), device="cuda")
    dH = torch.full((T, hs.d_model), float("nan"), device="cuda", dtype=dtype)
    dW = torch.full((hs.vocab, hs.d_model), float("nan"), device="cuda")
    dg = torch.full((hs.d_model,), float("nan"), device="cuda")
    ws = B.alloc_workspace(B.lmhead_workspace_bytes(cfg, T, chunk, wgrad_group))
    st = B.lmhead_rl_backward(cfg, objective, beta, eps, to_dev(g, dtype), to_dev(W, dtype), to_dev(H, dtype),
                              torch.from_numpy(tok).cuda(), f32(old), f32(ref), f32(adv), f32(wt), chunk, loss, dH, dW,
                              dg, ws, logp=logp, ell=ell, accumulate=accumulate, check=check,
                              wgrad_group=wgrad_group)
    if st != B.OK:
        return st
    assert B.last_device_status(ws) == B.OK
    return loss.item(), ell.item(), logp, dH, dW, dg


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T,V,chunk", [(200, 1000, 64), (96, 1003, 96)])
def test_grpo_matches_oracle(dtype, T, V, chunk):
    masked = T // 5
    hs, cfg, g, W, H, tok, old, ref, adv = make_case(40 + T, T, 128, V, dtype, masked)
    tok[T // 2] = -100
    wt = np.full(T, 1.0 / (T - masked - 1), dtype=np.float32)
    beta, eps = 0.04, CLIP_EPS
    # the oracle decides alone; its own float64 log-probabilities confirm the margin the inputs were built with
    ref_out = O.lmhead_grpo_backward(cfg, g, W, H, tok, old, ref, adv, wt, beta, eps)
    part = tok != -100
    margin = O.grpo_branch_margin(ref_out[1], old, eps)[part]
    assert margin.min() >= BRANCH_MARGIN and LOGP_TOL[dtype] < 0.5 * BRANCH_MARGIN
    r = np.exp(ref_out[1] - old)[part]
    assert (r > 1 + eps).any() and (r < 1 - eps).any() and ((r > 1 - eps) & (r < 1 + eps)).any()
    assert np.abs(adv[part]).min() > 0.0
    for ch, grp in ((chunk, 1), (23, 1), (23, 3)):     # chunk invariance, ragged; vocabulary gradient per 3 chunks
        loss, _, logp, dH, dW, dg = run_rl(hs, B.OBJ_GRPO, beta, eps, g, W, H, tok, old, ref, adv, wt, ch, dtype,
                                           wgrad_group=grp)
        assert np.abs(logp.cpu().numpy()[part] - ref_out[1][part]).max() < LOGP_TOL[dtype]
        assert torch.count_nonzero(logp[torch.from_numpy(~part).cuda()]) == 0
        assert abs(loss - ref_out[0]) <= (2e-5 if dtype == torch.float32 else 2e-2) * max(1.0, abs(ref_out[0]))
        assert_close("dH", dH, ref_out[2], TOL[dtype])
        assert_close("dW", dW, ref_out[3], TOL[dtype])
        assert_close("dg", dg, ref_out[4], TOL[dtype])
        assert torch.count_nonzero(dH[:masked]) == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dpo_matches_oracle(dtype):
    T, V, chunk = 192, 1536, 64
    hs, cfg, g, W, H, tok, old, ref, adv = make_case(77, T, 128, V, dtype, 0)
    tok[:40] = -100                                # shared prompt; then chosen (+1) and rejected (-1) responses
    tok[64:128] = -100                             # a whole chunk that takes no part
    sign = np.where(np.arange(T) < 128, 1.0, -1.0).astype(np.float32)
    beta = 0.25
    ref_out = O.lmhead_dpo_backward(cfg, g, W, H, tok, ref, sign, beta)
    for ch, grp in ((chunk, 1), (T, 1), (50, 1), (32, 2)):
        # the last case forms the vocabulary gradient per 2 chunks; rows 64..127 are then one whole skipped group
        loss, ell, logp, dH, dW, dg = run_rl(hs, B.OBJ_DPO, beta, 0.0, g, W, H, tok, None, ref, None, sign, ch, dtype,
                                             wgrad_group=grp)
        # bf16: ell sums 152 log-probabilities whose errors (up to 6e-3 each, from the bf16 operands of the logits
        # product) add up to 0.04; the correction factor sigmoid(beta ell) - 1 moves by beta * 0.04 / 2 < 1e-2
        assert abs(ell - ref_out[1]) <= (1e-4 if dtype == torch.float32 else 0.1)
        assert abs(loss - ref_out[0]) <= (1e-5 if dtype == torch.float32 else 1.5e-2)
        assert_close("dH", dH, ref_out[2], TOL[dtype])
        assert_close("dW", dW, ref_out[3], TOL[dtype])
        assert_close("dg", dg, ref_out[4], TOL[dtype])
        assert torch.count_nonzero(dH[64:128]) == 0


def test_rl_head_special_cases_and_errors():
    T, V = 64, 512
    hs, cfg, g, W, H, tok, old, ref, adv = make_case(5, T, 64, V, torch.float32, 8)
    N = T - 8
    lp = O._token_logprobs(cfg, g.astype(np.float64), W.astype(np.float64), H.astype(np.float64), tok, 64)
    sft = O.lmhead_ce_backward(cfg, g, W, H, tok)
    # on-policy, beta = 0, advantage 1, weight 1/N: the gradient of the mean cross-entropy (Eq. (2))
    out = run_rl(hs, B.OBJ_GRPO, 0.0, 0.2, g, W, H, tok, lp, ref, np.ones(T), np.full(T, 1.0 / N), 16, torch.float32)
    assert abs(out[0] + 1.0) < 1e-5
    assert_close("dW", out[4], sft[3], 1e-4)
    assert_close("dH", out[3], sft[2], 1e-4)
    # DPO with pi_ref = pi_theta: ell = 0, loss = ln 2, factor -1/2
    out = run_rl(hs, B.OBJ_DPO, 0.5, 0.0, g, W, H, tok, None, lp, None, np.ones(T), 16, torch.float32)
    assert abs(out[0] - np.log(2.0)) < 1e-5 and abs(out[1]) < 1e-4
    assert_close("dW", out[4], 0.25 * N * sft[3], 1e-4)
    # DPO cannot accumulate (the correction is applied in place); unknown objectives are refused
    assert run_rl(hs, B.OBJ_DPO, 0.5, 0.0, g, W, H, tok, None, lp, None, np.ones(T), 16, torch.float32,
                  accumulate=True, check=False) == B.E_SHAPE
    assert run_rl(hs, 7, 0.5, 0.0, g, W, H, tok, None, lp, None, np.ones(T), 16, torch.float32, check=False) == B.E_SHAPE
