"""GPU parity: streambp_layer_backward (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth
from helpers import TOL, assert_close, compare_layer, layer_case, run_layer, to_dev

pytestmark = pytest.mark.gpu


def test_tiny_config_layer_fp32_matches_oracle():
    # configuration "tiny": d 256, 4 query / 2 KV heads of 64, d_ff 688, T 512, chunk 128, fp32
    cfgs = synth.CONFIGS["tiny"]
    ocfg, bcfg, W, X, dY = layer_case(cfgs.layer, cfgs.seed, cfgs.T, torch.float32)
    dX, grads = run_layer(bcfg, W, X, dY, cfgs.chunk)
    compare_layer(ocfg, W, X, dY, dX, grads, TOL[torch.float32])


@pytest.mark.parametrize("bias,Hq,Hkv,dh,T,chunk,pos0", [
    (True, 4, 2, 64, 200, 64, 0),        # ragged last chunk (200 = 3*64 + 8), bias
    (False, 2, 1, 128, 96, 40, 17),      # head_dim 128, ragged, position offset
    (True, 6, 2, 64, 130, 1, 0),         # chunk of one row
    (True, 4, 4, 64, 77, 1000, 5),       # chunk >= T: un-partitioned mode
])
def test_layer_fp32_shapes(bias, Hq, Hkv, dh, T, chunk, pos0):
    shape = synth.LayerShape(64 * 2, Hq, Hkv, dh, 168, bias, 1e4)
    ocfg, bcfg, W, X, dY = layer_case(shape, 7, T, torch.float32, dy_std=1.0, wstd=0.05)
    dX, grads = run_layer(bcfg, W, X, dY, chunk, pos0=pos0)
    compare_layer(ocfg, W, X, dY, dX, grads, TOL[torch.float32], pos0=pos0)


def test_chunk_invariance_fp32():
    # Eq. (1): any partition gives the same gradient -- divisors and non-divisors of T
    shape = synth.LayerShape(128, 4, 2, 64, 168, True, 1e4)
    ocfg, bcfg, W, X, dY = layer_case(shape, 3, 192, torch.float32, dy_std=1.0, wstd=0.05)
    base_dX, base = run_layer(bcfg, W, X, dY, 192)
    for chunk in (96, 64, 48, 32, 50, 7):
        dX, grads = run_layer(bcfg, W, X, dY, chunk)
        assert O.rel_frobenius(dX.cpu().numpy(), base_dX.cpu().numpy()) < 1e-5, chunk
        for k in base:
            assert O.rel_frobenius(grads[k].cpu().numpy(), base[k].cpu().numpy()) < 1e-5, (chunk, k)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T,chunk,group", [(200, 32, 2), (200, 32, 3), (192, 64, 2), (150, 40, 16), (96, 96, 2)])
def test_weight_gradients_summed_over_groups_of_chunks(dtype, T, chunk, group):
    """The second partition size (Sec. 4.3): weight-gradient products formed once per `group` chunks over all their
    rows.  Same sum, different association: against the oracle at the usual tolerance, dX bit-identical to the
    ungrouped call (the chunk loop itself is unchanged), ragged last chunk and a last group of fewer chunks included,
    a group larger than the number of chunks, bias sums, and accumulation into existing gradients."""
    shape = synth.LayerShape(128, 4, 2, 64, 168, True, 1e4) if dtype == torch.float32 else \
        synth.LayerShape(256, 4, 2, 128, 512, True, 1e6)
    ocfg, bcfg, W, X, dY = layer_case(shape, 11, T, dtype, dy_std=1.0 if dtype == torch.float32 else 1e-3,
                                      wstd=0.05 if dtype == torch.float32 else 0.02)
    dX, grads = run_layer(bcfg, W, X, dY, chunk, pos0=3, wgrad_group=group)
    compare_layer(ocfg, W, X, dY, dX, grads, TOL[dtype], pos0=3)
    dX1, g1 = run_layer(bcfg, W, X, dY, chunk, pos0=3)
    assert torch.equal(dX, dX1)
    for k in g1:
        assert O.rel_frobenius(grads[k].cpu().numpy(), g1[k].cpu().numpy()) < (1e-5 if dtype == torch.float32 else 2e-3), k
    twice = {k: v.clone() for k, v in grads.items()}
    run_layer(bcfg, W, X, dY, chunk, pos0=3, wgrad_group=group, accumulate=True, grads=twice)
    for k in grads:
        assert O.rel_frobenius(twice[k].cpu().numpy(), 2.0 * grads[k].cpu().numpy()) < 1e-6, k
    assert B.layer_workspace_bytes(bcfg, T, chunk, group) > B.layer_workspace_bytes(bcfg, T, chunk) or chunk >= T
    # the operands kept per extra chunk of a group: a fixed number of bytes per row
    if chunk * 3 <= T:
        w1, w2, w3 = (B.layer_workspace_bytes(bcfg, T, chunk, g) for g in (1, 2, 3))
        assert w3 - w2 <= w2 - w1 + 4096 and w3 > w2


def test_bias_column_sums_with_many_row_splits():
    """Biases with dq + 2 dkv wider than the model width and a chunk long enough for the column sums to be split over
    many row blocks: the reduction partials are (row splits) x (dq + 2 dkv) floats.  (The workspace plan once sized them
    by the model width; the guarded debug mode found the overrun.  tests/test_gpu_gemm.py runs this case under guards.)"""
    shape = synth.LayerShape(256, 2, 2, 128, 512, True, 1e6)
    ocfg, bcfg, W, X, dY = layer_case(shape, 13, 1100, torch.bfloat16)
    for chunk, group in ((1024, 1), (512, 2)):
        dX, grads = run_layer(bcfg, W, X, dY, chunk, wgrad_group=group)
        compare_layer(ocfg, W, X, dY, dX, grads, TOL[torch.bfloat16])


def test_grouped_packed_batch_matches_packed():
    shape = synth.LayerShape(256, 4, 2, 128, 512, False, 1e6)
    ocfg, bcfg, W, X, dY = layer_case(shape, 12, 300, torch.bfloat16)
    cu = [0, 70, 71, 230, 300]
    dX, grads = run_layer(bcfg, W, X, dY, 64, wgrad_group=2, cu_seqlens=cu)
    dX_ref, G_ref = O.layer_backward_packed(ocfg, W, X, dY, cu)
    assert_close("dX", dX, dX_ref, TOL[torch.bfloat16])
    for k in G_ref:
        assert_close(k, grads[k], G_ref[k], TOL[torch.bfloat16])


def test_accumulate_adds_to_existing_gradients():
    shape = synth.LayerShape(128, 4, 2, 64, 168, True, 1e4)
    ocfg, bcfg, W, X, dY = layer_case(shape, 4, 100, torch.float32, dy_std=1.0, wstd=0.05)
    _, once = run_layer(bcfg, W, X, dY, 32)
    grads = {k: v.clone() for k, v in once.items()}
    run_layer(bcfg, W, X, dY, 32, accumulate=True, grads=grads)
    for k in once:
        assert O.rel_frobenius(grads[k].cpu().numpy(), 2.0 * once[k].cpu().numpy()) < 1e-6, k


def test_reruns_are_bit_identical():
    shape = synth.LayerShape(128, 4, 2, 64, 168, True, 1e4)
    ocfg, bcfg, W, X, dY = layer_case(shape, 5, 150, torch.bfloat16)
    dX1, g1 = run_layer(bcfg, W, X, dY, 64)
    dX2, g2 = run_layer(bcfg, W, X, dY, 64)
    assert torch.equal(dX1, dX2)
    for k in g1:
        assert torch.equal(g1[k], g2[k]), k


def test_causality_zero_upstream_tail():
    shape = synth.LayerShape(128, 4, 2, 64, 168, False, 1e4)
    ocfg, bcfg, W, X, dY = layer_case(shape, 6, 160, torch.float32, dy_std=1.0, wstd=0.05)
    dY[100:] = 0.0
    dX, _ = run_layer(bcfg, W, X, dY, 48)
    assert torch.count_nonzero(dX[100:]) == 0
    assert torch.count_nonzero(dX[:100]) > 0


@pytest.mark.parametrize("shape,T,chunk", [
    (synth.LayerShape(512, 8, 2, 64, 1376, True, 1e6), 640, 256),
    (synth.LayerShape(1024, 8, 2, 128, 2816, False, 5e5), 1100, 512),     # several tiles, ragged tail
    # three query heads of 128: the second 256-column tile of the Q product holds one head only (rotation in the
    # product's epilogue), one KV head, biases, ragged chunks
    (synth.LayerShape(384, 3, 1, 128, 688, True, 1e6), 300, 128),
])
def test_layer_bf16_matches_oracle(shape, T, chunk):
    ocfg, bcfg, W, X, dY = layer_case(shape, 8, T, torch.bfloat16)
    dX, grads = run_layer(bcfg, W, X, dY, chunk)
    errs = compare_layer(ocfg, W, X, dY, dX, grads, TOL[torch.bfloat16])
    print({k: f"{v:.2e}" for k, v in errs.items()})
    # chunk invariance in bf16 within the same tolerance
    dX2, grads2 = run_layer(bcfg, W, X, dY, T)
    compare_layer(ocfg, W, X, dY, dX2, grads2, TOL[torch.bfloat16])


def test_layer_bf16_long_prefix_small_width():
    """Few query tiles and heads against a long prefix (long key loops in few CTAs, many key-tile owners in the
    backward): results must match the oracle and stay bit-reproducible from run to run."""
    shape = synth.LayerShape(256, 2, 1, 128, 688, True, 1e6)
    T, chunk = 4096 + 200, 512
    ocfg, bcfg, W, X, dY = layer_case(shape, 12, T, torch.bfloat16)
    dX, grads = run_layer(bcfg, W, X, dY, chunk)
    compare_layer(ocfg, W, X, dY, dX, grads, TOL[torch.bfloat16])
    dX2, grads2 = run_layer(bcfg, W, X, dY, chunk)
    assert torch.equal(dX, dX2)
    for k in grads:
        assert torch.equal(grads[k], grads2[k]), k


@pytest.mark.parametrize("dtype,dh,cu", [
    (torch.float32, 64, [0, 70, 71, 200, 333]),          # sequences shorter and longer than the chunk, one of length 1
    (torch.bfloat16, 128, [0, 300, 1100, 1101, 1500]),   # tensor-core attention on per-sequence prefixes
])
def test_packed_batch_matches_sum_over_sequences(dtype, dh, cu):
    """Packed batch (several sequences back to back): attention and rotary positions stay inside each
    sequence; the result is the sum over the sequences of the single-sequence backward."""
    shape = synth.LayerShape(256, 4, 2, dh, 344, True, 1e4)
    T, chunk = cu[-1], 128
    wstd, dystd = (0.05, 1.0) if dtype == torch.float32 else (0.02, 1e-3)
    ocfg, bcfg, W, X, dY = layer_case(shape, 17, T, dtype, dy_std=dystd, wstd=wstd)
    Wd = {k: to_dev(v, dtype) for k, v in W.items()}
    Xd, dYd = to_dev(X, dtype), to_dev(dY, dtype)
    grads = B.alloc_layer_grads(bcfg)
    for g in grads.values():
        g.fill_(float("nan"))
    dX = torch.full_like(Xd, float("nan"))
    ws = B.alloc_workspace(B.layer_workspace_bytes(bcfg, T, chunk))
    B.layer_backward_packed(bcfg, Wd, Xd, dYd, chunk, cu, grads, dX, ws, pos0=3)
    assert B.last_device_status(ws) == B.OK
    dX_ref, G_ref = O.layer_backward_packed(ocfg, W, X, dY, cu, pos0=3)
    tol = TOL[dtype]
    assert_close("dX", dX, dX_ref, tol)
    for k, v in G_ref.items():
        assert_close(k, grads[k], v, tol)
    # malformed boundaries are refused on the host
    bad = B.layer_backward_packed(bcfg, Wd, Xd, dYd, chunk, [0, 50, 50, T], grads, dX, ws, check=False)
    assert bad == B.E_SHAPE
    assert B.layer_backward_packed(bcfg, Wd, Xd, dYd, chunk, [0, 50, T - 1], grads, dX, ws, check=False) == B.E_SHAPE


def test_host_fed_runner_matches_direct_calls():
    """Three sequences fed from pinned host memory through the two-buffer runner (copies on a second stream,
    overlapping the kernels of the neighbouring steps) give, bit for bit, the dX and the accumulated weight
    gradients of three direct calls on device-resident inputs."""
    shape = synth.LayerShape(256, 4, 2, 128, 512, True, 1e6)
    T, chunk, dt = 384, 128, torch.bfloat16
    _, bcfg, W, _, _ = layer_case(shape, 5, T, dt)
    Wd = {k: to_dev(v, dt) for k, v in W.items()}
    ios = [synth.make_layer_io(shape, 50 + i, T, True) for i in range(3)]
    ws = B.alloc_workspace(B.layer_workspace_bytes(bcfg, T, chunk))
    # direct calls
    g_ref = B.alloc_layer_grads(bcfg)
    dX_ref = []
    for i, (X, dY) in enumerate(ios):
        dX = torch.empty(T, shape.d_model, dtype=dt, device="cuda")
        B.layer_backward(bcfg, Wd, to_dev(X, dt), to_dev(dY, dt), chunk, g_ref, dX, ws, accumulate=i > 0)
        dX_ref.append(dX.cpu())
    assert B.last_device_status(ws) == B.OK
    # host-fed
    g = B.alloc_layer_grads(bcfg)
    fed = B.HostFedLayerBackward(bcfg, Wd, g, T, chunk, ws)
    host = [(torch.from_numpy(X).to(dt).pin_memory(), torch.from_numpy(dY).to(dt).pin_memory()) for X, dY in ios]
    out = [torch.empty(T, shape.d_model, dtype=dt).pin_memory() for _ in ios]
    fed.prefetch(*host[0])
    for i in range(3):
        if i + 1 < 3:
            fed.prefetch(*host[i + 1])
        fed.step(out[i], accumulate=i > 0)
    fed.drain()
    torch.cuda.synchronize()
    assert B.last_device_status(ws) == B.OK
    for i in range(3):
        assert torch.equal(out[i], dX_ref[i])
    for k in g:
        assert torch.equal(g[k], g_ref[k])


def test_data_parallel_runner_single_rank_matches_direct_call():
    """World size 1: the data-parallel runner (gradients accumulated into views of one flat bucket, exchange on a
    second stream) returns the gradients of the direct call, bit for bit, and its shard is the whole bucket."""
    from paper_2506_03077_b200 import dp
    shape = synth.LayerShape(256, 4, 2, 128, 512, True, 1e6)
    T, chunk, dt = 320, 128, torch.bfloat16
    _, bcfg, W, X, dY = layer_case(shape, 11, T, dt)
    dX_ref, g_ref = run_layer(bcfg, W, X, dY, chunk)
    Wd = {k: to_dev(v, dt) for k, v in W.items()}
    r = dp.DataParallelLayerBackward(bcfg, Wd, T, chunk)
    dX = torch.empty(T, shape.d_model, dtype=dt, device="cuda")
    for v in r.bucket.views.values():
        v.fill_(float("nan"))            # the call must overwrite
    r.step(to_dev(X, dt), to_dev(dY, dt), dX)
    r.wait()
    torch.cuda.synchronize()
    assert B.last_device_status(r.ws) == B.OK
    assert torch.equal(dX, dX_ref)
    full = dp.gather_full_gradients(r.bucket, r.shard)
    for k in g_ref:
        assert torch.equal(full[k], g_ref[k])
    assert r.shard.numel() == r.bucket.total



class _Fenced:
    """A device tensor with sentinel-filled fences of `pad` elements before and after it in the same allocation."""

    def __init__(self, shape, dtype, pad=512, fill=float("nan")):
        n = int(np.prod(shape))
        self.pad, self.n = pad, n
        self.sentinel = 12345.0 if dtype != torch.int64 else 12345
        self.buf = torch.full((n + 2 * pad,), self.sentinel, dtype=dtype, device="cuda")
        self.t = self.buf[pad:pad + n].view(*shape)
        self.t.fill_(fill)
        assert self.t.data_ptr() % 16 == 0

    def intact(self):
        return bool((self.buf[:self.pad] == self.sentinel).all()) and bool((self.buf[self.pad + self.n:] == self.sentinel).all())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_no_write_outside_the_outputs(dtype):
    """Every output of the layer, the head and the attention building blocks sits between sentinel fences; ragged
    sizes (rows, chunk and vocabulary not multiples of any tile).  Nothing outside the outputs may change."""
    shape = synth.LayerShape(256, 4, 2, 128, 520, True, 1e6) if dtype == torch.bfloat16 else \
        synth.LayerShape(128, 4, 2, 64, 168, True, 1e4)
    T, chunk = 333, 100
    ocfg, bcfg, W, X, dY = layer_case(shape, 21, T, dtype)
    Wd = {k: to_dev(v, dtype) for k, v in W.items()}
    dX = _Fenced((T, shape.d_model), dtype)
    G = {k: _Fenced(shp, torch.float32) for k, shp in B.layer_grad_shapes(bcfg).items()}
    Xd, dYd = to_dev(X, dtype), to_dev(dY, dtype)
    before = {k: v.clone() for k, v in dict(Wd, X=Xd, dY=dYd).items()}
    for group in (1, 2):
        ws = B.alloc_workspace(B.layer_workspace_bytes(bcfg, T, chunk, group))
        B.layer_backward(bcfg, Wd, Xd, dYd, chunk, {k: g.t for k, g in G.items()}, dX.t, ws, wgrad_group=group)
        assert B.last_device_status(ws) == B.OK
        assert all(torch.equal(v, dict(Wd, X=Xd, dY=dYd)[k]) for k, v in before.items())      # inputs are read only
        assert dX.intact() and all(g.intact() for g in G.values()), [k for k, g in G.items() if not g.intact()]
        assert torch.isfinite(dX.t.float()).all() and all(torch.isfinite(g.t).all() for g in G.values())
    # head: vocabulary and rows ragged
    hs = synth.HeadShape(shape.d_model, 1003)
    g, Wv, H, labels = synth.make_head_inputs(hs, 22, 211, dtype == torch.bfloat16, 40)
    hc = B.HeadConfig(hs.d_model, hs.vocab, hs.rms_eps, hs.ignore_index, dtype)
    dH, dWv, dg = _Fenced((211, hs.d_model), dtype), _Fenced((hs.vocab, hs.d_model), torch.float32), _Fenced((hs.d_model,), torch.float32)
    loss, nv = _Fenced((1,), torch.float32), _Fenced((1,), torch.int64, fill=0)
    ws = B.alloc_workspace(B.lmhead_workspace_bytes(hc, 211, 64))
    B.lmhead_ce_backward(hc, to_dev(g, dtype), to_dev(Wv, dtype), to_dev(H, dtype), torch.from_numpy(labels).cuda(), 64,
                         loss.t, nv.t, dH.t, dWv.t, dg.t, ws)
    assert B.last_device_status(ws) == B.OK
    assert all(f.intact() for f in (dH, dWv, dg, loss, nv))
    assert torch.isfinite(dWv.t).all() and torch.isfinite(dH.t.float()).all()
    # attention building blocks (both tensor-core backward kernels in bf16)
    n, q0, Hq, Hkv, dh = 150, 139, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    mk = lambda *s: torch.randn(*s, device="cuda").to(dtype)
    q, do, k, v = mk(n, Hq, dh), mk(n, Hq, dh), mk(q0 + n, Hkv, dh), mk(q0 + n, Hkv, dh)
    o, lse = _Fenced((n, Hq, dh), dtype), _Fenced((Hq, n), torch.float32)
    for engine in ((1, 3, 4) if dtype == torch.bfloat16 else (1,)):
        B.attention_forward(q, k, v, q0, o.t, lse.t, engine=engine)
        torch.cuda.synchronize()
        assert o.intact() and lse.intact(), engine
    for engine in ((1, 2, 5) if dtype == torch.bfloat16 else (1,)):
        dq, dk, dv = _Fenced((n, Hq, dh), torch.float32), _Fenced((q0 + n, Hkv, dh), torch.float32, fill=0.0), \
            _Fenced((q0 + n, Hkv, dh), torch.float32, fill=0.0)
        B.attention_backward(q, k, v, o.t, do, lse.t, q0, dq.t, dk.t, dv.t, engine=engine)
        torch.cuda.synchronize()
        assert dq.intact() and dk.intact() and dv.intact(), engine
        assert torch.isfinite(dq.t).all() and torch.isfinite(dk.t).all()
