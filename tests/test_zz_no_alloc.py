"""The allocation-free attention backward (for callers that cannot allocate device memory when they
call) must give what the ordinary entry point gives, twice in a row, alone or after other tests."""
import ctypes as C

import pytest
import torch

from paper_2506_03077_b200 import binding as B

pytestmark = pytest.mark.gpu


def _inputs(n, q0, Hq, Hkv, dh, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g).to(dtype).cuda()
    q, do = mk(n, Hq, dh), mk(n, Hq, dh)
    k, v = mk(q0 + n, Hkv, dh), mk(q0 + n, Hkv, dh)
    o = torch.empty_like(q)
    lse = torch.empty(Hq, n, device="cuda")
    B.attention_forward(q, k, v, q0, o, lse)
    return q, k, v, o, do, lse


@pytest.mark.parametrize("dtype,dh,engine", [(torch.bfloat16, 128, 0), (torch.float32, 64, 1)])
def test_static_scratch_variant_matches_ordinary_entry_point(dtype, dh, engine):
    n, q0, Hq, Hkv = 200, 136, 4, 2
    for call in range(2):                       # the shared array keeps the previous call's contents
        q, k, v, o, do, lse = _inputs(n, q0, Hq, Hkv, dh, dtype, 100 + call)
        ref = [torch.empty(n, Hq, dh, device="cuda"), torch.zeros(q0 + n, Hkv, dh, device="cuda"),
               torch.zeros(q0 + n, Hkv, dh, device="cuda")]
        got = [torch.full_like(ref[0], float("nan")), torch.zeros_like(ref[1]), torch.zeros_like(ref[2])]
        B.attention_backward(q, k, v, o, do, lse, q0, *ref, engine=engine)
        before = torch.cuda.memory_allocated()
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        B.attention_backward_static(q, k, v, o, do, lse, q0, *got, engine=engine)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # the driver's own count of free device memory sees an allocation made behind PyTorch's back; the first
        # call may still load kernels and look up the array's address, so the second call is the one that must
        # leave it unchanged
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before
        for name, a, b in zip(("dq", "dk", "dv"), got, ref):
            err = (a.double() - b.double()).norm() / b.double().norm()
            assert err <= (2e-2 if dtype == torch.bfloat16 else 1e-4), (call, name, float(err))


def test_static_scratch_variant_rejects_oversize():
    n, Hq = B.STATIC_DELTA_MAX_FLOATS // 8 + 1, 8          # one row too many for the fixed array
    st = B.lib().streambp_attention_backward_static(4096, 4096, 4096, 4096, 4096, 4096, n, 0, Hq, 8, 128, 1, 4096,
                                                    4096, 4096, 0, None)
    assert st == B.E_WORKSPACE
    assert "workspace" in B.status_string(st)
