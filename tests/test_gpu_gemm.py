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
