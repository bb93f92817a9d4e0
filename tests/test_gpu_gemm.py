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
