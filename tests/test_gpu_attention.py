"""GPU parity of the partitioned-attention building blocks (CUDA-core and tensor-core engines)
against the CPU oracle's attention."""
import numpy as np
import pytest
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth
from helpers import assert_close

pytestmark = pytest.mark.gpu


def make_qkv(seed, n, q0, Hq, Hkv, dh, dtype, scale=1.0):
    kv = q0 + n
    q = synth.normal(seed, "q", (kv, Hq, dh), 0.0, scale)
    k = synth.normal(seed, "k", (kv, Hkv, dh), 0.0, scale)
    v = synth.normal(seed, "v", (kv, Hkv, dh))
    do = synth.normal(seed, "do", (kv, Hq, dh))
    if dtype == torch.bfloat16:
        q, k, v, do = (synth.round_bf16(a) for a in (q, k, v, do))
    return q, k, v, do


def oracle_chunk(q, k, v, do, q0):
    """Oracle attention on the whole prefix; the rows of the chunk are those from q0 on.
    Upstream gradient is zero outside the chunk, so dk/dv hold the chunk's contribution only."""
    o = O.attention_forward(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64))
    do_chunk = do.astype(np.float64).copy()
    do_chunk[:q0] = 0.0
    dq, dk, dv = O.attention_backward(q.astype(np.float64), k.astype(np.float64), v.astype(np.float64), do_chunk)
    return o[q0:], dq[q0:], dk, dv


def oracle_window(q, k, v, do, q0):
    """The same for a long prefix: only the chunk's query rows are evaluated (q, do hold rows q0.. only)."""
    f = lambda a: a.astype(np.float64)
    o = O.attention_forward(f(q), f(k), f(v), q_start=q0)
    dq, dk, dv = O.attention_backward(f(q), f(k), f(v), f(do), q_start=q0)
    return o, dq, dk, dv


def oracle_lse(q, k, q0, dh):
    T, Hq, _ = q.shape
    G = Hq // k.shape[1]
    out = np.empty((Hq, T - q0))
    for h in range(Hq):
        s = (q[q0:, h].astype(np.float64) @ k[:, h // G].astype(np.float64).T) / np.sqrt(dh)
        for i in range(T - q0):
            row = s[i, : q0 + i + 1]
            out[h, i] = row.max() + np.log(np.exp(row - row.max()).sum())
    return out


CASES = [
    # n, q0, Hq, Hkv
    (128, 0, 2, 1),        # one tile, diagonal only
    (256, 0, 4, 2),        # two query tiles
    (128, 384, 2, 2),      # chunk deep inside the sequence: full tiles then the diagonal
    (200, 300, 4, 1),      # ragged chunk, offset not a tile multiple
    (77, 1000, 2, 1),      # short chunk against a long prefix
    (640, 0, 2, 1),        # un-partitioned
    (384, 200, 2, 1),      # two-tile forward CTAs: the last CTA has one tile only; offset not a tile multiple
    (130, 126, 4, 2),      # the second tile of the CTA has two rows
]


@pytest.mark.parametrize("engine", [1, 2, 3, 4])      # CUDA cores; tensor cores: automatic, one tile, two tiles per CTA
@pytest.mark.parametrize("n,q0,Hq,Hkv", CASES)
def test_attention_forward_bf16(engine, n, q0, Hq, Hkv):
    dh, dt = 128, torch.bfloat16
    q, k, v, do = make_qkv(n + q0, n, q0, Hq, Hkv, dh, dt, scale=1.5)
    o_ref, _, _, _ = oracle_chunk(q, k, v, do, q0)
    qd = torch.from_numpy(q[q0:]).to("cuda", dt).contiguous()
    kd, vd = torch.from_numpy(k).to("cuda", dt), torch.from_numpy(v).to("cuda", dt)
    o = torch.full((n, Hq, dh), float("nan"), device="cuda", dtype=dt)
    lse = torch.full((Hq, n), float("nan"), device="cuda")
    B.attention_forward(qd, kd, vd, q0, o, lse, engine=engine)
    torch.cuda.synchronize()
    got = o.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert O.rel_frobenius(got, o_ref) < 6e-3
    assert np.abs(got - o_ref).max() < 0.06
    lse_ref = oracle_lse(q, k, q0, dh)
    assert np.abs(lse.cpu().numpy() - lse_ref).max() < 2e-3


@pytest.mark.parametrize("engine", [1, 2, 5])          # CUDA cores; tensor cores: two-role kernel, five-product kernel
@pytest.mark.parametrize("n,q0,Hq,Hkv", CASES)
def test_attention_backward_bf16(engine, n, q0, Hq, Hkv):
    dh, dt = 128, torch.bfloat16
    q, k, v, do = make_qkv(n + q0 + 1, n, q0, Hq, Hkv, dh, dt, scale=1.5)
    o_ref, dq_ref, dk_ref, dv_ref = oracle_chunk(q, k, v, do, q0)
    qd = torch.from_numpy(q[q0:]).to("cuda", dt).contiguous()
    dod = torch.from_numpy(do[q0:]).to("cuda", dt).contiguous()
    kd, vd = torch.from_numpy(k).to("cuda", dt), torch.from_numpy(v).to("cuda", dt)
    o = torch.empty((n, Hq, dh), device="cuda", dtype=dt)
    lse = torch.empty((Hq, n), device="cuda")
    B.attention_forward(qd, kd, vd, q0, o, lse, engine=1)
    dq = torch.full((n, Hq, dh), float("nan"), device="cuda")
    dk = torch.ones((q0 + n, Hkv, dh), device="cuda")       # accumulated into: start from a known value
    dv = torch.ones((q0 + n, Hkv, dh), device="cuda")
    B.attention_backward(qd, kd, vd, o, dod, lse, q0, dq, dk, dv, engine=engine)
    torch.cuda.synchronize()
    assert_close("dq", dq, dq_ref, 1.5e-2, heads=Hq)
    assert_close("dk", dk - 1.0, dk_ref, 1.5e-2, heads=Hkv)
    assert_close("dv", dv - 1.0, dv_ref, 1.5e-2, heads=Hkv)


# The prefix lengths of the T = 32768 layer configuration: the last chunk (2048 queries against 32768 keys, 256 key
# tiles per CTA: lazy rescale, the K/V rings and the merged dK/dV + dQ grid all in their long-run regime) and a ragged
# 200-row chunk that ends at the same row.  Four query heads on one KV head keep the oracle (numpy, float64) at a few
# seconds.  Every (128-row block, head) of every output is bounded, not only the whole tensor.
@pytest.mark.parametrize("n,q0", [(2048, 30720), (200, 32768 - 200)])
def test_attention_full_prefix_bf16(n, q0):
    Hq, Hkv, dh, dt = 4, 1, 128, torch.bfloat16
    kv = q0 + n
    f = lambda name, shape, s=1.0: synth.round_bf16(synth.normal(900 + n, name, shape, 0.0, s))
    q, do = f("q", (n, Hq, dh), 1.5), f("do", (n, Hq, dh))
    k, v = f("k", (kv, Hkv, dh), 1.5), f("v", (kv, Hkv, dh))
    o_ref, dq_ref, dk_ref, dv_ref = oracle_window(q, k, v, do, q0)
    qd, dod = (torch.from_numpy(a).to("cuda", dt).contiguous() for a in (q, do))
    kd, vd = torch.from_numpy(k).to("cuda", dt), torch.from_numpy(v).to("cuda", dt)
    o = torch.empty((n, Hq, dh), device="cuda", dtype=dt)
    lse = torch.empty((Hq, n), device="cuda")
    for engine in (3, 4):                  # one and two query tiles per CTA
        o.fill_(float("nan")); lse.fill_(float("nan"))
        B.attention_forward(qd, kd, vd, q0, o, lse, engine=engine)
        torch.cuda.synchronize()
        assert_close(f"o (engine {engine})", o, o_ref, 6e-3, heads=Hq)
        assert torch.isfinite(lse).all()
    for engine in (2, 5):                  # the two-role kernel and the five-product kernel
        dq = torch.full((n, Hq, dh), float("nan"), device="cuda")
        dk = torch.zeros((kv, Hkv, dh), device="cuda")
        dv = torch.zeros((kv, Hkv, dh), device="cuda")
        B.attention_backward(qd, kd, vd, o, dod, lse, q0, dq, dk, dv, engine=engine)
        torch.cuda.synchronize()
        assert_close(f"dq (engine {engine})", dq, dq_ref, 1.5e-2, heads=Hq)
        assert_close(f"dk (engine {engine})", dk, dk_ref, 1.5e-2, heads=Hkv)
        assert_close(f"dv (engine {engine})", dv, dv_ref, 1.5e-2, heads=Hkv)


@pytest.mark.parametrize("dh,dtype", [(64, torch.float32), (128, torch.float32), (64, torch.bfloat16)])
def test_attention_cuda_core_variants(dh, dtype):
    n, q0, Hq, Hkv = 100, 60, 4, 2
    q, k, v, do = make_qkv(5, n, q0, Hq, Hkv, dh, dtype)
    o_ref, dq_ref, dk_ref, dv_ref = oracle_chunk(q, k, v, do, q0)
    qd = torch.from_numpy(q[q0:]).to("cuda", dtype).contiguous()
    dod = torch.from_numpy(do[q0:]).to("cuda", dtype).contiguous()
    kd, vd = torch.from_numpy(k).to("cuda", dtype), torch.from_numpy(v).to("cuda", dtype)
    o = torch.empty((n, Hq, dh), device="cuda", dtype=dtype)
    lse = torch.empty((Hq, n), device="cuda")
    B.attention_forward(qd, kd, vd, q0, o, lse, engine=1)
    tol = 1e-5 if dtype == torch.float32 else 6e-3
    assert O.rel_frobenius(o.float().cpu().numpy(), o_ref) < tol
    dq = torch.empty((n, Hq, dh), device="cuda")
    dk = torch.zeros((q0 + n, Hkv, dh), device="cuda")
    dv = torch.zeros((q0 + n, Hkv, dh), device="cuda")
    B.attention_backward(qd, kd, vd, o, dod, lse, q0, dq, dk, dv, engine=1)
    tol = 2e-5 if dtype == torch.float32 else 1.5e-2
    assert O.rel_frobenius(dq.cpu().numpy(), dq_ref) < tol
    assert O.rel_frobenius(dk.cpu().numpy(), dk_ref) < tol
    assert O.rel_frobenius(dv.cpu().numpy(), dv_ref) < tol


def test_attention_growing_maxima_tensor_core():
    """Scores that grow with the key index: the running row maximum rises by more than the lazy-rescale threshold
    (2^8) from one 128-key tile to the next, so the forward kernel has to rescale its output accumulator at every
    tile and the backward sees probabilities concentrated at the end of each row.  Pins the exactness of the lazy
    rescale (output and log-sum-exp) against the oracle's plain softmax."""
    n, q0, Hq, Hkv, dh, dt = 256, 768, 2, 1, 128, torch.bfloat16
    kv = q0 + n
    q, k, v, do = make_qkv(31, n, q0, Hq, Hkv, dh, dt, scale=0.25)
    # a common direction e: q gets +4 e, key j gets +(j / 128) * 3.5 e  ->  score += 14 * (tile index) / sqrt(128) * ...
    e = np.zeros(dh); e[:8] = 1.0
    q = synth.round_bf16(q + 4.0 * e)
    k = synth.round_bf16(k + (np.arange(kv)[:, None, None] / 128.0) * 3.5 * e)
    tile_step = 4.0 * 3.5 * 8 / np.sqrt(dh) * 1.4426950408889634      # rise of the score per tile, in log2 units
    assert tile_step > 8.0
    o_ref, dq_ref, dk_ref, dv_ref = oracle_chunk(q, k, v, do, q0)
    qd = torch.from_numpy(q[q0:]).to("cuda", dt).contiguous()
    dod = torch.from_numpy(do[q0:]).to("cuda", dt).contiguous()
    kd, vd = torch.from_numpy(k).to("cuda", dt), torch.from_numpy(v).to("cuda", dt)
    o = torch.full((n, Hq, dh), float("nan"), device="cuda", dtype=dt)
    lse = torch.full((Hq, n), float("nan"), device="cuda")
    lse_ref = oracle_lse(q, k, q0, dh)
    for engine in (3, 4):                  # one and two query tiles per CTA: both forward kernels
        o.fill_(float("nan")); lse.fill_(float("nan"))
        B.attention_forward(qd, kd, vd, q0, o, lse, engine=engine)
        got = o.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all()
        assert O.rel_frobenius(got, o_ref) < 6e-3
        assert np.abs(lse.cpu().numpy() - lse_ref).max() < 2e-3 * max(1.0, np.abs(lse_ref).max() / 10)
    # backward: dK and dV are well conditioned.  dQ = sum_j dS_j K_j is not, here: the rows of dS sum to zero, which
    # cancels the large common component of these keys only as exactly as delta = rowsum(dO * O) is known, and O is
    # stored in bf16.  The fp32 CUDA-core engine, fed the same bf16 O, shows the same loss; the tensor-core engine
    # must stay within a small factor of it.
    errs = {}
    for engine in (1, 2):
        dq = torch.full((n, Hq, dh), float("nan"), device="cuda")
        dk = torch.zeros((kv, Hkv, dh), device="cuda")
        dv = torch.zeros((kv, Hkv, dh), device="cuda")
        B.attention_backward(qd, kd, vd, o, dod, lse, q0, dq, dk, dv, engine=engine)
        torch.cuda.synchronize()
        errs[engine] = (O.rel_frobenius(dq.cpu().numpy(), dq_ref), O.rel_frobenius(dk.cpu().numpy(), dk_ref),
                        O.rel_frobenius(dv.cpu().numpy(), dv_ref))
    assert errs[2][1] < 1e-2 and errs[2][2] < 1e-2
    assert errs[2][0] < 2.5 * errs[1][0] + 1e-2
    assert errs[2][0] < DQ_GROWING_MAXIMA_TOL, errs


# dQ against the oracle in the ill-conditioned case above: measured 5.7e-2 (CUDA-core engine) and 7.0e-2 (tensor-core
# engine) on the same bf16 O -- the conditioning of the case (see the comment in the test), not a property of an engine
DQ_GROWING_MAXIMA_TOL = 0.1
