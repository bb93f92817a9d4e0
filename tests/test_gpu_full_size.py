"""Parity at the benchmark's full sizes and launch configuration.

The oracle cannot be run on every full-size case inside a test run, so full-size cases use what holds at
any size and what the oracle can produce cheaply:
  * prefix window: with the upstream gradient zero beyond row P, causality makes every gradient equal to
    that of the P-row truncated problem, which the oracle computes directly;
  * chunk invariance (Eq. (1)) between two partition sizes at full T;
  * LM head: rows of dH depend on their own row only (given the global N), so sampled rows come from the
    oracle; the vocabulary sum of dW vanishes; masked rows are exactly zero.
Full oracle runs at full size are opt-in (STREAMBP_FULL_ORACLE=1): minutes of CPU time each.
"""
import os

import numpy as np
import pytest
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth
from helpers import TOL, assert_close, to_dev

pytestmark = pytest.mark.gpu
FULL_ORACLE = os.environ.get("STREAMBP_FULL_ORACLE") == "1"
BF = torch.bfloat16


def _cfgs(s):
    oc = O.LayerCfg(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta, s.rms_eps)
    bc = B.LayerConfig(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta, s.rms_eps, BF)
    return oc, bc


def _run(bc, Wd, Xd, dYd, chunk, wgrad_group=1):
    grads = B.alloc_layer_grads(bc)
    dX = torch.empty_like(Xd)
    ws = B.alloc_workspace(B.layer_workspace_bytes(bc, Xd.shape[0], chunk, wgrad_group))
    B.layer_backward(bc, Wd, Xd, dYd, chunk, grads, dX, ws, wgrad_group=wgrad_group)
    assert B.last_device_status(ws) == B.OK
    return dX, grads


@pytest.mark.parametrize("name", ["qwen7b_layer", "llama8b_layer"])
def test_layer_full_size_prefix_window_and_chunk_invariance(name):
    c = synth.CONFIGS[name]
    s, T, chunk = c.layer, c.T, c.chunk
    oc, bc = _cfgs(s)
    W = synth.make_layer_weights(s, c.seed, True)
    X, dY = synth.make_layer_io(s, c.seed, T, True)
    Wd = {k: to_dev(v, BF) for k, v in W.items()}
    Xd = to_dev(X, BF)
    # (1) prefix window: upstream gradient only in the first P rows (P is not a multiple of the chunk)
    P = chunk + 384
    dYw = dY.copy()
    dYw[P:] = 0.0
    dX, grads = _run(bc, Wd, Xd, to_dev(dYw, BF), chunk)
    assert torch.count_nonzero(dX[P:]) == 0                      # causality, exactly
    dX_ref, G_ref = O.layer_backward(oc, W, X[:P], dY[:P])
    tol = TOL[BF]
    assert_close("dX[:P]", dX[:P], dX_ref, tol)
    for k, v in G_ref.items():
        assert_close(k, grads[k], v, tol)
    del dX, grads
    # (2) chunk invariance at full T on the full upstream gradient, in the benchmark's configuration
    dYd = to_dev(dY, BF)
    dX_a, g_a = _run(bc, Wd, Xd, dYd, chunk)
    dX_b, g_b = _run(bc, Wd, Xd, dYd, 2 * chunk)
    assert O.rel_frobenius(dX_b.float().cpu().numpy(), dX_a.float().cpu().numpy()) <= tol
    for k in g_a:
        assert O.rel_frobenius(g_b[k].cpu().numpy(), g_a[k].cpu().numpy()) <= tol, k
    del dX_b, g_b
    # (3) the second partition size: weight gradients summed over groups of 3 chunks (the last group is shorter) --
    # dX is the same chunk loop bit for bit, the weight gradients the same sums in another association
    dX_c, g_c = _run(bc, Wd, Xd, dYd, chunk, wgrad_group=3)
    assert torch.equal(dX_c, dX_a)
    for k in g_a:
        assert O.rel_frobenius(g_c[k].cpu().numpy(), g_a[k].cpu().numpy()) <= 2e-3, k
    del dX_c, g_c
    if FULL_ORACLE:
        dX_ref, G_ref = O.layer_backward(oc, W, X, dY)
        errs = {"dX": assert_close("dX", dX_a, dX_ref, tol)}
        for k, v in G_ref.items():
            errs[k] = assert_close(k, g_a[k], v, tol)
        print(name, "full-size errors vs oracle:", {k: f"{e:.2e}" for k, e in errs.items()})


def test_head_full_width():
    """qwen7b head: full hidden width and vocabulary.  A 2048-row problem against the oracle, then the
    full T = 32768 / chunk 1024 launch checked on sampled rows and invariants."""
    c = synth.CONFIGS["qwen7b_head"]
    h, T = c.head, c.T
    g, Wv, H, labels = synth.make_head_inputs(h, c.seed, T, True, c.masked_prefix)
    cfg = B.HeadConfig(h.d_model, h.vocab, h.rms_eps, h.ignore_index, BF)
    gd, Wd = to_dev(g, BF), to_dev(Wv, BF)
    ocfg = O.HeadCfg(h.d_model, h.vocab)

    def run(Hn, lab, chunk):
        Hd, ld = to_dev(Hn, BF), torch.from_numpy(lab).cuda()
        n = Hn.shape[0]
        loss = torch.zeros(1, device="cuda")
        nv = torch.zeros(1, dtype=torch.int64, device="cuda")
        dH = torch.empty_like(Hd)
        dW = torch.empty(h.vocab, h.d_model, device="cuda")
        dg = torch.empty(h.d_model, device="cuda")
        ws = B.alloc_workspace(B.lmhead_workspace_bytes(cfg, n, chunk))
        B.lmhead_ce_backward(cfg, gd, Wd, Hd, ld, chunk, loss, nv, dH, dW, dg, ws)
        assert B.last_device_status(ws) == B.OK
        return loss.item(), int(nv.item()), dH, dW, dg

    # reduced T, full widths, ragged chunking (2048 = 1000 + 1000 + 48), rows 7168.. so that some are masked
    sl = slice(7168, 7168 + 2048)
    loss, nv, dH, dW, dg = run(H[sl], labels[sl], 1000)
    ref = O.lmhead_ce_backward(ocfg, g, Wv, H[sl], labels[sl])
    assert nv == ref[1] == 1024
    assert abs(loss - ref[0]) <= 2e-3 * ref[0]
    tol = TOL[BF]
    assert_close("dH", dH, ref[2], tol)
    assert_close("dW", dW, ref[3], tol)
    assert_close("dg", dg, ref[4], tol)
    del dH, dW, dg
    # full size, benchmark launch configuration
    loss, nv, dH, dW, dg = run(H, labels, c.chunk)
    assert nv == T - c.masked_prefix
    assert 11.9 < loss < 13.5                                     # ~ ln V + var(z)/2 at random init
    assert torch.count_nonzero(dH[: c.masked_prefix]) == 0
    rows = np.array([8192, 8193, 12345, 20000, 31000, 32767])
    sub = O.lmhead_ce_backward(ocfg, g, Wv, H[rows], labels[rows])
    expect = sub[2] * (sub[1] / nv)                               # same rows, global N instead of the subset's
    assert_close("dH[sampled rows]", dH[torch.from_numpy(rows).cuda()], expect, tol)
    col = dW.double().sum(0).abs().max().item()
    assert col <= 1e-2 * dW.double().abs().sum(0).max().item()    # rows of softmax - onehot sum to zero
