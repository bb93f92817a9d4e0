"""GPU parity of the exposed product building block in its three operand layouts."""
import numpy as np
import pytest
import torch

from paper_2506_03077_b200 import binding as B

pytestmark = pytest.mark.gpu


def ref_product(op, A, Bm):
    a, b = A.double().cpu(), Bm.double().cpu()
    if op == B.OP_NT:
        return a @ b.T
    if op == B.OP_NN:
        return a @ b
    return a.T @ b


def shapes(op, M, N, K):
    if op == B.OP_NT:
        return (M, K), (N, K)
    if op == B.OP_NN:
        return (M, K), (K, N)
    return (K, M), (K, N)


@pytest.mark.parametrize("op", [B.OP_NT, B.OP_NN, B.OP_TN])
@pytest.mark.parametrize("M,N,K", [(64, 64, 16), (130, 70, 45), (257, 129, 300)])
@pytest.mark.parametrize("dtype,out", [(torch.float32, torch.float32), (torch.bfloat16, torch.float32),
                                       (torch.bfloat16, torch.bfloat16)])
def test_cuda_core_product(op, M, N, K, dtype, out):
    gen = torch.Generator(device="cpu").manual_seed(M * 7 + N * 3 + K + op)
    sa, sb = shapes(op, M, N, K)
    A = torch.randn(sa, generator=gen).to(dtype).cuda()
    Bm = torch.randn(sb, generator=gen).to(dtype).cuda()
    C = torch.full((M, N), float("nan"), dtype=out, device="cuda")
    B.gemm(op, A, Bm, C, engine=1)
    ref = ref_product(op, A, Bm)
    err = (C.double().cpu() - ref).norm() / ref.norm()
    assert err < (4e-3 if out == torch.bfloat16 else 2e-6)
    if out == torch.float32:
        B.gemm(op, A, Bm, C, accumulate=True, engine=1)
        err2 = (C.double().cpu() - 2 * ref).norm() / ref.norm()
        assert err2 < 4e-6


@pytest.mark.parametrize("op", [B.OP_NT, B.OP_NN, B.OP_TN])
@pytest.mark.parametrize("M,N,K", [
    (128, 256, 64),       # exactly one tile, one K slice
    (128, 256, 512),      # pipeline wraps around its stages
    (256, 512, 192),      # several tiles per CTA row/column
    (200, 264, 136),      # ragged in all three dimensions (multiples of 8 for the 16-byte pitch)
    (1000, 688, 256),     # the tiny configuration's d_ff
    (2048, 3584, 1024),   # more tiles than SMs: persistent loop, both accumulator buffers reused
    (384, 512, 448),      # CTA pairs: the odd CTA of the last row tile has no rows; 7 K slices over 6 stages
])
@pytest.mark.parametrize("out", [torch.float32, torch.bfloat16])
def test_tensor_core_product(op, M, N, K, out):
    gen = torch.Generator(device="cpu").manual_seed(M + 3 * N + 7 * K + op)
    sa, sb = shapes(op, M, N, K)
    A = torch.randn(sa, generator=gen).to(torch.bfloat16).cuda()
    Bm = torch.randn(sb, generator=gen).to(torch.bfloat16).cuda()
    C = torch.full((M, N), float("nan"), dtype=out, device="cuda")
    B.gemm(op, A, Bm, C, engine=2)
    torch.cuda.synchronize()
    ref = ref_product(op, A, Bm)
    got = C.double().cpu()
    assert torch.isfinite(got).all()
    err = (got - ref).norm() / ref.norm()
    assert err < (4e-3 if out == torch.bfloat16 else 1e-5), err
    # element-wise too: a misplaced tile or a wrong swizzle shows up as O(1) errors on single entries
    tol = 0.05 * K ** 0.5 if out == torch.bfloat16 else 2e-3 * K ** 0.5
    assert (got - ref).abs().max() < tol
    if out == torch.float32:
        B.gemm(op, A, Bm, C, accumulate=True, engine=2)
        err2 = (C.double().cpu() - 2 * ref).norm() / ref.norm()
        assert err2 < 2e-5, err2


def test_tensor_core_product_strided_views():
    # leading dimensions larger than the logical width (sub-matrices of wider buffers)
    gen = torch.Generator(device="cpu").manual_seed(5)
    Abuf = torch.randn(300, 512, generator=gen).to(torch.bfloat16).cuda()
    Bbuf = torch.randn(400, 512, generator=gen).to(torch.bfloat16).cuda()
    Cbuf = torch.zeros(300, 640, device="cuda")
    A, Bm, C = Abuf[:, 64:64 + 320], Bbuf[:, 128:128 + 320], Cbuf[:, 8:8 + 400]
    B.gemm(B.OP_NT, A, Bm, C, engine=2)
    ref = A.double().cpu() @ Bm.double().cpu().T
    assert ((C.double().cpu() - ref).norm() / ref.norm()) < 1e-5
    assert torch.count_nonzero(Cbuf[:, :8]) == 0 and torch.count_nonzero(Cbuf[:, 408:]) == 0


def _operands(op, M, N, K, gen):
    sa, sb = shapes(op, M, N, K)
    return (torch.randn(sa, generator=gen).bfloat16().cuda(), torch.randn(sb, generator=gen).bfloat16().cuda())


@pytest.mark.parametrize("dynamic", [False, True])
def test_grouped_products_mixed_layouts(dynamic):
    """Four problems of different layouts, output types and tile lengths in one launch: two weight-gradient
    shaped accumulations, one input gradient summed over three K segments, one bf16 forward product; every
    size ragged against the 128 x 256 x 64 tile.  Each output equals the fp64 product of the same bf16
    operands, with either tile schedule, and the scheduler's counters are left at zero."""
    gen = torch.Generator(device="cpu").manual_seed(11)
    n = 328
    a1, b1 = _operands(B.OP_TN, 520, 264, n, gen)
    a2, b2 = _operands(B.OP_TN, 136, 264, n, gen)
    segs = [_operands(B.OP_NN, n, 264, K, gen) for K in (520, 136, 72)]
    a4, b4 = _operands(B.OP_NT, n, 1000, 264, gen)
    base1 = torch.randn(520, 264, generator=gen).cuda()
    C1, C2 = base1.clone(), torch.full((136, 264), float("nan"), device="cuda")
    C3 = torch.full((n, 264), float("nan"), device="cuda")
    C4 = torch.full((n, 1000), float("nan"), device="cuda", dtype=torch.bfloat16)
    sched = torch.zeros(2, dtype=torch.int32, device="cuda") if dynamic else None
    B.gemm_grouped([(B.OP_TN, [(a1, b1)], C1, True), (B.OP_TN, [(a2, b2)], C2, False),
                    (B.OP_NN, segs, C3, False), (B.OP_NT, [(a4, b4)], C4, False)], sched)
    torch.cuda.synchronize()
    r1 = ref_product(B.OP_TN, a1, b1) + base1.double().cpu()
    r2 = ref_product(B.OP_TN, a2, b2)
    r3 = sum(ref_product(B.OP_NN, a, b) for a, b in segs)
    r4 = ref_product(B.OP_NT, a4, b4)
    for got, ref, tol in ((C1, r1, 2e-6), (C2, r2, 2e-6), (C3, r3, 2e-6), (C4, r4, 4e-3)):
        assert torch.isfinite(got).all()
        assert (got.double().cpu() - ref).norm() / ref.norm() < tol
    if dynamic:
        assert sched.tolist() == [0, 0]


def test_grouped_products_schedule_invariance():
    """More tiles than CTAs, long and short tiles mixed: the dynamic schedule gives bit-identical results to
    the static one and to one launch per problem, twice in a row with the same counters."""
    gen = torch.Generator(device="cpu").manual_seed(12)
    n = 1024
    dg, h2 = _operands(B.OP_TN, 4096, 1024, n, gen)          # dWg += dg^T h2
    du = torch.randn(n, 4096, generator=gen).bfloat16().cuda()
    wg = torch.randn(4096, 1024, generator=gen).bfloat16().cuda()
    wu = torch.randn(4096, 1024, generator=gen).bfloat16().cuda()
    sched = torch.zeros(2, dtype=torch.int32, device="cuda")
    outs = []
    for mode in ("static", "dynamic", "dynamic", "single"):
        dWg = torch.ones(4096, 1024, device="cuda")
        dWu = torch.ones(4096, 1024, device="cuda")
        dh2 = torch.full((n, 1024), float("nan"), device="cuda")
        if mode == "single":
            B.gemm(B.OP_TN, dg, h2, dWg, accumulate=True, engine=2)
            B.gemm(B.OP_TN, du, h2, dWu, accumulate=True, engine=2)
            B.gemm_grouped([(B.OP_NN, [(dg, wg), (du, wu)], dh2, False)])
        else:
            B.gemm_grouped([(B.OP_TN, [(dg, h2)], dWg, True), (B.OP_TN, [(du, h2)], dWu, True),
                            (B.OP_NN, [(dg, wg), (du, wu)], dh2, False)], sched if mode == "dynamic" else None)
        torch.cuda.synchronize()
        outs.append((dWg, dWu, dh2))
    assert sched.tolist() == [0, 0]
    ref = ref_product(B.OP_NN, dg, wg) + ref_product(B.OP_NN, du, wu)
    assert (outs[0][2].double().cpu() - ref).norm() / ref.norm() < 1e-5     # fp32 sum over K = 8192
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)


def test_grouped_products_rejects_bad_arguments():
    a = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    c16 = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    c32 = torch.zeros(64, 64, device="cuda")
    assert B.gemm_grouped([(B.OP_NT, [(a, a)], c16, True)], check=False) == B.E_DTYPE       # bf16 C cannot accumulate
    assert B.gemm_grouped([(B.OP_NT, [(a, a)], c32, False)] * 5, check=False) == B.E_SHAPE   # more than 4 problems
    odd = torch.zeros(64, 68, dtype=torch.bfloat16, device="cuda")[:, :64]                   # pitch 68: not 16-byte rows
    assert B.gemm_grouped([(B.OP_NT, [(odd, a)], c32, False)], check=False) == B.E_SHAPE


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("M,N,K", [(256, 128, 64), (1000, 1376, 512), (300, 200, 136), (2048, 2816, 1024)])
def test_swiglu_product(M, N, K, dtype):
    """g = A Wg^T, u = A Wu^T, m = silu(g) * u in one call (one launch on CTA pairs in bf16): ragged rows and columns,
    several tiles per pair, the odd CTA of the last row tile without rows."""
    gen = torch.Generator(device="cpu").manual_seed(M + N + K)
    A = (torch.randn(M, K, generator=gen) * 0.5).to(dtype).cuda()
    Wg = (torch.randn(N, K, generator=gen) * 0.1).to(dtype).cuda()
    Wu = (torch.randn(N, K, generator=gen) * 0.1).to(dtype).cuda()
    g, u, m = (torch.full((M, N), float("nan"), dtype=dtype, device="cuda") for _ in range(3))
    B.gemm_swiglu(A, Wg, Wu, g, u, m)
    torch.cuda.synchronize()
    a = A.double().cpu()
    g_ref, u_ref = a @ Wg.double().cpu().T, a @ Wu.double().cpu().T
    tol = 4e-3 if dtype == torch.bfloat16 else 1e-5
    for got, ref in ((g, g_ref), (u, u_ref)):
        assert torch.isfinite(got).all()
        assert (got.double().cpu() - ref).norm() / ref.norm() < tol
    # m is a function of the STORED g and u: exact up to the last rounding and the fast exponential
    gs, us = g.double().cpu(), u.double().cpu()
    m_ref = gs * torch.sigmoid(gs) * us
    assert (m.double().cpu() - m_ref).norm() / m_ref.norm() < (3e-3 if dtype == torch.bfloat16 else 1e-6)


def test_product_kernel_query():
    """bf16 products run on a tcgen05 kernel: on CTA pairs wherever a two-CTA cluster with the full shared-memory
    carve-out can be scheduled (any B200), else on the single-CTA kernel."""
    assert B.product_kernel() in ("cta_pair", "single_cta")


def test_single_cta_fallback_kernel():
    """The single-CTA product kernel (used where a two-CTA cluster cannot be scheduled) is selected by an environment
    variable read when the library first runs a product: exercised in a fresh interpreter, all three layouts."""
    import os
    import subprocess
    import sys
    code = r"""
import torch
from paper_2506_03077_b200 import binding as B
gen = torch.Generator(device="cpu").manual_seed(3)
for op in (B.OP_NT, B.OP_NN, B.OP_TN):
    M, N, K = 392, 520, 456
    sa, sb = {B.OP_NT: ((M, K), (N, K)), B.OP_NN: ((M, K), (K, N)), B.OP_TN: ((K, M), (K, N))}[op]
    A = torch.randn(sa, generator=gen).bfloat16().cuda(); Bm = torch.randn(sb, generator=gen).bfloat16().cuda()
    a, b = A.double().cpu(), Bm.double().cpu()
    ref = a @ b.T if op == B.OP_NT else (a @ b if op == B.OP_NN else a.T @ b)
    C = torch.full((M, N), float("nan"), device="cuda")
    B.gemm(op, A, Bm, C, engine=2); B.gemm(op, A, Bm, C, accumulate=True, engine=2)
    torch.cuda.synchronize()
    assert ((C.double().cpu() - 2 * ref).norm() / ref.norm()) < 2e-5
A = torch.randn(300, 136, generator=gen).bfloat16().cuda(); Wg = torch.randn(200, 136, generator=gen).bfloat16().cuda()
Wu = torch.randn(200, 136, generator=gen).bfloat16().cuda()
g, u, m = (torch.empty(300, 200, dtype=torch.bfloat16, device="cuda") for _ in range(3))
B.gemm_swiglu(A, Wg, Wu, g, u, m); torch.cuda.synchronize()
ref = A.double().cpu() @ Wg.double().cpu().T
assert ((g.double().cpu() - ref).norm() / ref.norm()) < 4e-3
gs, us = g.double().cpu(), u.double().cpu()
assert ((m.double().cpu() - gs * torch.sigmoid(gs) * us).norm() / (gs * torch.sigmoid(gs) * us).norm()) < 3e-3
print("fallback ok")
"""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, STREAMBP_GEMM_SINGLE_CTA="1", STREAMBP_VERBOSE="1", PYTHONPATH=root)
    out = subprocess.run([sys.executable, "-c", code], env=env, cwd=root, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "fallback ok" in out.stdout and "single CTA" in out.stderr


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    """The tensor-core kernels wait on mbarriers with a time limit; when it runs out the CTA raises a flag, every
    role leaves its loop, tensor memory is freed, the kernel returns and the host reads E_DEVICE_TIMEOUT.  The test
    kernel runs that same wait on a barrier nothing arrives at, with a 1 ms limit: nothing hangs, the status is
    reported once, and a product launched afterwards is correct."""
    ws = B.alloc_workspace(4096)
    ws.zero_()
    assert B.last_device_status(ws) == B.OK
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    assert B.test_expire_wait(1_000_000) == B.OK
    t1.record()
    assert B.last_device_status(ws) == B.E_DEVICE_TIMEOUT
    assert 0.9 < t0.elapsed_time(t1) < 50.0                  # gave up after the limit, not after the 2 s default
    assert B.last_device_status(ws) == B.OK                  # reading the status clears the flag
    assert B.lib().streambp_test_expire_wait(10, None) == B.E_SHAPE     # limits outside 1 us .. 100 ms are refused
    M, N, K = 384, 512, 256
    A = torch.randn(M, K, device="cuda").to(torch.bfloat16)
    Bm = torch.randn(N, K, device="cuda").to(torch.bfloat16)
    Cm = torch.empty(M, N, device="cuda")
    B.gemm(B.OP_NT, A, Bm, Cm, engine=2)
    torch.cuda.synchronize()
    ref = A.double() @ Bm.double().T
    assert float((Cm.double() - ref).norm() / ref.norm()) < 1e-5
    assert B.last_device_status(ws) == B.OK


def test_workspace_guards_catch_an_overrun():
    """Debug mode STREAMBP_WS_GUARD puts a guard after every workspace sub-buffer, filled before and checked after each
    call.  The hook runs that mechanism on three small sub-buffers: untouched guards -> OK; a kernel that writes one
    float (or more) past the end of the second sub-buffer -> E_WORKSPACE_GUARD."""
    ws = B.alloc_workspace(8192)
    L = B.lib()
    for overrun, want in ((0, B.OK), (1, B.E_WORKSPACE_GUARD), (40, B.E_WORKSPACE_GUARD), (0, B.OK)):
        assert L.streambp_test_workspace_guard(ws.data_ptr(), ws.numel(), overrun, None) == B.OK
        assert B.last_device_status(ws) == want, overrun
    assert L.streambp_test_workspace_guard(ws.data_ptr(), 1024, 0, None) == B.E_WORKSPACE
    assert L.streambp_test_workspace_guard(ws.data_ptr() + 4, ws.numel(), 0, None) == B.E_ALIGN


def test_whole_path_is_clean_under_workspace_guards():
    """Layer, packed, grouped, head (SFT / GRPO / DPO) and model calls in a fresh process with STREAMBP_WS_GUARD set:
    every call's guards must be intact (device status OK) and the results must still match the oracle."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, STREAMBP_WS_GUARD="1")
    sel = ["tests/test_gpu_layer.py::test_layer_bf16_matches_oracle", "tests/test_gpu_layer.py::test_layer_fp32_shapes",
           "tests/test_gpu_layer.py::test_weight_gradients_summed_over_groups_of_chunks",
           "tests/test_gpu_layer.py::test_grouped_packed_batch_matches_packed",
           "tests/test_gpu_layer.py::test_bias_column_sums_with_many_row_splits",
           "tests/test_gpu_lmhead.py", "tests/test_gpu_rl_heads.py",
           "tests/test_gpu_model.py::test_tiny_configuration_end_to_end_fp32", "tests/test_gpu_model.py::test_small_model_with_embedding"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + sel, cwd=root,
                       env=env, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
