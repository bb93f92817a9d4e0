"""GPU parity: streambp_lmhead_ce_backward against the CPU oracle, closed forms and invariants."""
import numpy as np
import pytest
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth
from helpers import TOL, assert_close, to_dev

pytestmark = pytest.mark.gpu


def run_head(hs: synth.HeadShape, g, W, H, labels, chunk, dtype, accumulate=False, prior=None, wgrad_group=1):
    cfg = B.HeadConfig(hs.d_model, hs.vocab, hs.rms_eps, hs.ignore_index, dtype)
    gd, Wd, Hd = to_dev(g, dtype), to_dev(W, dtype), to_dev(H, dtype)
    ld = torch.from_numpy(labels).cuda()
    T = H.shape[0]
    loss = torch.full((1,), float("nan"), device="cuda")
    nv = torch.full((1,), -1, dtype=torch.int64, device="cuda")
    dH = torch.full_like(Hd, float("nan"))
    if prior is None:
        dW = torch.full((hs.vocab, hs.d_model), float("nan"), device="cuda")
        dg = torch.full((hs.d_model,), float("nan"), device="cuda")
    else:
        dW, dg = prior
    ws = B.alloc_workspace(B.lmhead_workspace_bytes(cfg, T, chunk, wgrad_group))
    B.lmhead_ce_backward(cfg, gd, Wd, Hd, ld, chunk, loss, nv, dH, dW, dg, ws, accumulate=accumulate,
                         wgrad_group=wgrad_group)
    return loss, nv, dH, dW, dg, B.last_device_status(ws)


def test_tiny_config_head_fp32():
    c = synth.CONFIGS["tiny"]
    g, W, H, labels = synth.make_head_inputs(c.head, c.seed, c.T, False, c.masked_prefix)
    loss, nv, dH, dW, dg, st = run_head(c.head, g, W, H, labels, c.chunk_head, torch.float32)
    assert st == B.OK
    ref = O.lmhead_ce_backward(O.HeadCfg(c.head.d_model, c.head.vocab), g, W, H, labels)
    assert int(nv.item()) == ref[1] == c.T - c.masked_prefix
    assert abs(loss.item() - ref[0]) <= 1e-5 * abs(ref[0])
    assert_close("dH", dH, ref[2], TOL[torch.float32])
    assert_close("dW", dW, ref[3], TOL[torch.float32])
    assert_close("dg", dg, ref[4], TOL[torch.float32])
    assert torch.count_nonzero(dH[: c.masked_prefix]) == 0       # ignored rows: exactly zero


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("V,T,chunk", [(1000, 150, 64), (1003, 90, 32), (2048, 64, 64)])
def test_head_shapes_and_chunk_invariance(dtype, V, T, chunk):
    hs = synth.HeadShape(128, V)
    g, W, H, labels = synth.make_head_inputs(hs, 11, T, dtype == torch.bfloat16, T // 4)
    labels[T // 2] = -100
    ref = O.lmhead_ce_backward(O.HeadCfg(128, V), g, W, H, labels)
    for ch in (chunk, T, 1 if T <= 64 else 17):
        loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, labels, ch, dtype)
        assert st == B.OK and int(nv.item()) == ref[1]
        assert abs(loss.item() - ref[0]) <= (1e-5 if dtype == torch.float32 else 2e-3) * abs(ref[0])
        assert_close("dH", dH, ref[2], TOL[dtype])
        assert_close("dW", dW, ref[3], TOL[dtype])
        assert_close("dg", dg, ref[4], TOL[dtype])


def test_zero_head_weights_closed_form():
    # W = 0: loss = ln V, dH = 0, dW[v] = (1/N) sum_t (1/V - [v = y_t]) hn_t
    hs = synth.HeadShape(64, 4096)
    g, W, H, labels = synth.make_head_inputs(hs, 2, 40, False, 8)
    W[:] = 0.0
    loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, labels, 16, torch.float32)
    assert abs(loss.item() - 8.317766166719343) < 2e-6
    assert torch.count_nonzero(dH) == 0 and torch.count_nonzero(dg) == 0
    hn = H / np.sqrt((H.astype(np.float64) ** 2).mean(-1, keepdims=True) + 1e-6) * g
    N = 32
    expect = np.tile(hn[8:].sum(0) / (4096 * N), (4096, 1))
    for t in range(8, 40):
        expect[labels[t]] -= hn[t] / N
    assert_close("dW", dW, expect, 1e-5)


def test_vocab_sum_of_weight_gradient_vanishes():
    hs = synth.HeadShape(128, 3000)
    g, W, H, labels = synth.make_head_inputs(hs, 5, 96, True, 10)
    _, _, _, dW, _, _ = run_head(hs, g, W, H, labels, 32, torch.bfloat16)
    col = dW.double().sum(0).abs().max().item()
    scale = dW.double().abs().sum(0).max().item()
    assert col <= 1e-2 * scale


def test_device_status_bad_label_and_no_valid_label():
    hs = synth.HeadShape(64, 500)
    g, W, H, labels = synth.make_head_inputs(hs, 1, 32, False, 0)
    bad = labels.copy()
    bad[5] = 500
    *_, st = run_head(hs, g, W, H, bad, 16, torch.float32)
    assert st == B.E_BAD_LABEL
    none = np.full_like(labels, -100)
    loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, none, 16, torch.float32)
    assert st == B.E_NO_VALID_LABELS
    assert loss.item() == 0.0 and int(nv.item()) == 0
    assert torch.count_nonzero(dH) == 0 and torch.count_nonzero(dW) == 0 and torch.count_nonzero(dg) == 0


def test_head_accumulate():
    hs = synth.HeadShape(64, 512)
    g, W, H, labels = synth.make_head_inputs(hs, 3, 48, False, 4)
    _, _, _, dW, dg, _ = run_head(hs, g, W, H, labels, 16, torch.float32)
    prior = (dW.clone(), dg.clone())
    run_head(hs, g, W, H, labels, 16, torch.float32, accumulate=True, prior=prior)
    assert O.rel_frobenius(prior[0].cpu().numpy(), 2 * dW.cpu().numpy()) < 1e-6
    assert O.rel_frobenius(prior[1].cpu().numpy(), 2 * dg.cpu().numpy()) < 1e-6


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_fully_masked_chunks_are_skipped_exactly(dtype):
    """Chunks whose labels are all ignored are gated off on the device; the result must still be the
    oracle's, with exactly-zero dH rows there, also when the first chunk is one of them."""
    hs = synth.HeadShape(128, 1536)
    T, chunk = 256, 64
    g, W, H, labels = synth.make_head_inputs(hs, 21, T, dtype == torch.bfloat16, 0)
    labels[0:64] = -100        # chunk 0
    labels[128:192] = -100     # chunk 2
    labels[200] = -100         # a single ignored row inside a live chunk
    ref = O.lmhead_ce_backward(O.HeadCfg(128, 1536), g, W, H, labels)
    loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, labels, chunk, dtype)
    assert st == B.OK and int(nv.item()) == ref[1] == 127
    assert abs(loss.item() - ref[0]) <= (1e-5 if dtype == torch.float32 else 2e-3) * abs(ref[0])
    assert_close("dH", dH, ref[2], TOL[dtype])
    assert_close("dW", dW, ref[3], TOL[dtype])
    assert_close("dg", dg, ref[4], TOL[dtype])
    for rows in (slice(0, 64), slice(128, 192), slice(200, 201)):
        assert torch.count_nonzero(dH[rows]) == 0


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("group", [2, 3, 100])
def test_vocab_gradient_summed_over_groups_of_chunks(dtype, group):
    """The second partition size: dW_vocab formed once per `group` chunks (ragged last chunk, ragged last group,
    a group larger than the number of chunks) equals the oracle and changes nothing but dW's summation order."""
    hs = synth.HeadShape(128, 1003)
    T, chunk = 330, 48                       # 7 chunks, the last of 42 rows
    g, W, H, labels = synth.make_head_inputs(hs, 31, T, dtype == torch.bfloat16, 20)
    labels[100] = -100
    ref = O.lmhead_ce_backward(O.HeadCfg(128, 1003), g, W, H, labels)
    base = run_head(hs, g, W, H, labels, chunk, dtype)
    loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, labels, chunk, dtype, wgrad_group=group)
    assert st == B.OK and int(nv.item()) == ref[1]
    assert abs(loss.item() - ref[0]) <= (1e-5 if dtype == torch.float32 else 2e-3) * abs(ref[0])
    assert_close("dH", dH, ref[2], TOL[dtype])
    assert_close("dW", dW, ref[3], TOL[dtype])
    assert_close("dg", dg, ref[4], TOL[dtype])
    # everything but dW is computed by the same launches on the same operands
    assert torch.equal(dH, base[2]) and torch.equal(dg, base[4]) and loss.item() == base[0].item()
    assert O.rel_frobenius(dW.cpu().numpy(), base[3].cpu().numpy().astype(np.float64)) < 1e-5


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_grouped_head_with_masked_chunks_and_groups(dtype):
    """Groups of 2 chunks: group 0 fully masked (skipped on the device), group 1 half masked (its masked chunk is
    processed and contributes exact zeros), accumulate on top of a prior value."""
    hs = synth.HeadShape(128, 1536)
    T, chunk = 384, 64
    g, W, H, labels = synth.make_head_inputs(hs, 23, T, dtype == torch.bfloat16, 0)
    labels[0:128] = -100       # chunks 0, 1 = group 0
    labels[192:256] = -100     # chunk 3, second half of group 1
    ref = O.lmhead_ce_backward(O.HeadCfg(128, 1536), g, W, H, labels)
    prior = (torch.full((1536, 128), 0.5, device="cuda"), torch.full((128,), -0.25, device="cuda"))
    loss, nv, dH, dW, dg, st = run_head(hs, g, W, H, labels, chunk, dtype, accumulate=True, prior=prior,
                                        wgrad_group=2)
    assert st == B.OK and int(nv.item()) == ref[1] == 192
    assert_close("dH", dH, ref[2], TOL[dtype])
    assert_close("dW", dW - 0.5, ref[3], TOL[dtype])
    assert_close("dg", dg + 0.25, ref[4], TOL[dtype])
    for rows in (slice(0, 128), slice(192, 256)):
        assert torch.count_nonzero(dH[rows]) == 0
