"""The C-ABI library loads, exports what include/streambp.h declares, and rejects bad
arguments on the host (no GPU needed: validation precedes every CUDA call)."""
import ctypes as C
import os
import re

import pytest

from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(B.LIB_PATH):
        build_mod.build()
    return B.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "streambp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(streambp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"streambp_layer_backward", "streambp_lmhead_ce_backward", "streambp_model_backward",
            "streambp_layer_workspace_bytes", "streambp_last_device_status"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)


def test_status_strings(lib):
    assert B.status_string(0) == "ok"
    seen = {B.status_string(s) for s in range(-10, 1)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert B.status_string(-77) == "unknown status"


def cfg(**kw):
    base = dict(d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ff=688, qkv_bias=False, rope_theta=1e4)
    base.update(kw)
    import torch
    return B.LayerConfig(dtype=torch.float32, **base)


def test_workspace_query_rejects_bad_shapes(lib):
    assert B.layer_workspace_bytes(cfg(), 512, 128) > 0
    assert B.layer_workspace_bytes(cfg(head_dim=96), 512, 128) == 0
    assert B.layer_workspace_bytes(cfg(n_kv_heads=3), 512, 128) == 0
    assert B.layer_workspace_bytes(cfg(d_model=250), 512, 128) == 0
    assert B.layer_workspace_bytes(cfg(), 0, 128) == 0
    assert B.layer_workspace_bytes(cfg(), 512, 0) == 0
    # chunk >= T is the un-partitioned mode and needs the most memory
    small, full = B.layer_workspace_bytes(cfg(), 512, 128), B.layer_workspace_bytes(cfg(), 512, 512)
    assert full > small and B.layer_workspace_bytes(cfg(), 512, 4096) == full


def test_workspace_matches_memory_model(lib):
    """Per-chunk activations scale with the chunk, the K/V set with T (Sec. 3.2.2, memory efficiency)."""
    import torch
    c = B.LayerConfig(4096, 32, 8, 128, 14336, False, 5e5, dtype=torch.bfloat16)
    T = 32768
    kv_set = T * 1024 * (2 + 2 + 4 + 4) + T * 128 * 4     # K, V bf16; dK, dV fp32; rope table
    w1, w2 = B.layer_workspace_bytes(c, T, 1024), B.layer_workspace_bytes(c, T, 2048)
    per_row = (w2 - w1) / 1024
    assert abs((w1 - 1024 * per_row) - kv_set) < (1 << 21)
    # one chunk row: 3 [I] + h1,h2,dr_s [d] + Q,O,dO [dq] + dk,dv [dkv] in bf16; fa, r, dr fp32; small vectors
    expect = 2 * (3 * 14336 + 3 * 4096 + 3 * 4096 + 2 * 1024) + 4 * (3 * 4096) + 4 * (2 + 2 * 32)
    assert abs(per_row - expect) < 64


def test_host_side_errors(lib):
    import torch
    c = cfg().c()
    w = B.LayerPtrsC(**{f: 4096 for f in B.WEIGHT_FIELDS})
    g = B.LayerPtrsC(**{f: 4096 for f in B.WEIGHT_FIELDS})
    call = lambda **kw: lib.streambp_layer_backward(
        C.byref(kw.get("c", c)), C.byref(kw.get("w", w)), kw.get("X", 4096), kw.get("dY", 8192), kw.get("T", 512),
        kw.get("chunk", 128), 0, 0, C.byref(kw.get("g", g)), kw.get("dX", 12288), kw.get("ws", 1 << 20),
        kw.get("wsb", 16), None)
    assert call() == B.E_WORKSPACE
    assert call(X=None) == B.E_NULL
    assert call(X=4100) == B.E_ALIGN
    assert call(ws=(1 << 20) + 16) == B.E_ALIGN
    assert call(T=0) == B.E_SHAPE
    assert call(dX=4096) == B.E_SHAPE            # dX aliases X
    bad = cfg().c()
    bad.dtype = 7
    assert call(c=bad) == B.E_DTYPE
    wnull = B.LayerPtrsC(**{f: (None if f == "wo" else 4096) for f in B.WEIGHT_FIELDS})
    assert call(w=wnull) == B.E_NULL
    # biases are required only when the configuration says so
    wnob = B.LayerPtrsC(**{f: (None if f in ("bq", "bk", "bv") else 4096) for f in B.WEIGHT_FIELDS})
    assert call(w=wnob, g=wnob) == B.E_WORKSPACE
    cb = cfg(qkv_bias=True).c()
    assert call(c=cb, w=wnob) == B.E_NULL
    h = B.HeadConfig(256, 4096, dtype=torch.float32).c()
    st = lib.streambp_lmhead_ce_backward(C.byref(h), 4096, 4096, 4096, 4096, 512, 128, 0, 4096, 4096, 4096, 4096,
                                         4096, 1 << 20, 16, None)
    assert st == B.E_WORKSPACE
    st = lib.streambp_lmhead_ce_backward(C.byref(h), 4096, 4096, 4096, None, 512, 128, 0, 4096, 4096, 4096, 4096,
                                         4096, 1 << 20, 1 << 30, None)
    assert st == B.E_NULL
    assert lib.streambp_gemm(5, 8, 8, 8, 4096, 8, 4096, 8, 4096, 8, 1, 0, 0, 0, None) == B.E_SHAPE
    assert lib.streambp_last_device_status(None, None) == B.E_NULL


def test_attention_entry_points_refuse_misaligned_pointers(lib):
    """A tensor that is only 4-byte aligned (an offset view) would fault on the device, where the kernels use 16-byte
    vector accesses and TMA tiles; the three attention entry points return E_ALIGN before anything is enqueued."""
    a = 4096                                  # never dereferenced: validation precedes every CUDA call
    fwd = lambda **kw: lib.streambp_attention_forward(kw.get("q", a), kw.get("k", a), kw.get("v", a), 128, 0, 4, 2, 128,
                                                      1, kw.get("o", a), kw.get("lse", a), 0, None)
    for name in ("q", "k", "v", "o"):
        assert fwd(**{name: a + 4}) == B.E_ALIGN, name
    assert fwd(lse=a + 2) == B.E_ALIGN
    names = ("q", "k", "v", "o", "d_o", "lse", "delta", "dq", "dk", "dv")

    def bwd(static, **kw):
        p = {n: kw.get(n, a) for n in names}
        if static:
            return lib.streambp_attention_backward_static(p["q"], p["k"], p["v"], p["o"], p["d_o"], p["lse"], 128, 0, 4,
                                                          2, 128, 1, p["dq"], p["dk"], p["dv"], 0, None)
        return lib.streambp_attention_backward(p["q"], p["k"], p["v"], p["o"], p["d_o"], p["lse"], 128, 0, 4, 2, 128, 1,
                                               p["delta"], p["dq"], p["dk"], p["dv"], 0, None)
    for static in (False, True):
        for name in ("q", "k", "v", "o", "d_o", "dq", "dk", "dv"):
            assert bwd(static, **{name: a + 4}) == B.E_ALIGN, (static, name)
        assert bwd(static, lse=a + 2) == B.E_ALIGN
    assert bwd(False, delta=a + 2) == B.E_ALIGN


def test_grouped_entry_point_validates_on_the_host(lib):
    import torch
    c = cfg().c()
    w = B.LayerPtrsC(**{f: 4096 for f in B.WEIGHT_FIELDS})
    call = lambda group, wsb=16, cu=None, n=0: lib.streambp_layer_backward_grouped(
        C.byref(c), C.byref(w), 4096, 8192, 512, 128, group, cu, n, 0, 0, C.byref(w), 12288, 1 << 20, wsb, None)
    assert call(0) == B.E_SHAPE and call(-3) == B.E_SHAPE
    assert call(2) == B.E_WORKSPACE                      # 16 bytes of workspace are never enough
    # the size query grows with the group and saturates at the number of chunks (512 / 128 = 4)
    sizes = [lib.streambp_layer_workspace_bytes_grouped(C.byref(c), 512, 128, g) for g in (1, 2, 4, 9)]
    assert sizes[0] == B.layer_workspace_bytes(cfg(), 512, 128) and sizes[0] < sizes[1] < sizes[2] == sizes[3]
    assert lib.streambp_layer_workspace_bytes_grouped(C.byref(c), 512, 128, 0) == 0
    # malformed sequence boundaries are refused before anything else happens
    bad = (C.c_int64 * 3)(0, 300, 400)
    assert call(2, wsb=1 << 30, cu=bad, n=2) == B.E_SHAPE


def test_grouped_head_entry_points_validate_on_the_host(lib):
    import torch
    hc = B.HeadConfig(256, 4096, 1e-6, -100, torch.bfloat16)
    c = hc.c()
    rl = B.RlCfgC(B.OBJ_GRPO, 0.04, 0.2)
    ce = lambda group, wsb=16: lib.streambp_lmhead_ce_backward_grouped(
        C.byref(c), 4096, 8192, 12288, 16384, 512, 128, group, 0, 4096, 4096, 4096, 4096, 4096, 1 << 20, wsb, None)
    rlc = lambda group, wsb=16: lib.streambp_lmhead_rl_backward_grouped(
        C.byref(c), C.byref(rl), 4096, 8192, 12288, 16384, 4096, 4096, 4096, 4096, 512, 128, group, 0, 4096, None,
        None, 4096, 4096, 4096, 1 << 20, wsb, None)
    for call in (ce, rlc):
        assert call(0) == B.E_SHAPE and call(-1) == B.E_SHAPE
        assert call(2) == B.E_WORKSPACE
    # one more chunk of normalised rows and dlogits per slot; saturates at the number of chunks (512 / 128 = 4)
    sizes = [lib.streambp_lmhead_workspace_bytes_grouped(C.byref(c), 512, 128, g) for g in (1, 2, 4, 9)]
    assert sizes[0] == B.lmhead_workspace_bytes(hc, 512, 128) and sizes[0] < sizes[1] < sizes[2] == sizes[3]
    per_slot = 128 * (256 + 4096) * 2
    assert per_slot <= sizes[1] - sizes[0] <= per_slot + 2048
    assert lib.streambp_lmhead_workspace_bytes_grouped(C.byref(c), 512, 128, 0) == 0
    # a workspace sized for the plain call is too small for a grouped one
    assert ce(2, wsb=sizes[0]) == B.E_WORKSPACE


def test_per_device_facts_are_keyed_by_device_ordinal(lib):
    """SM count, shared-memory opt-in and product-kernel choice are cached per device: a second device must not get
    the first one's answer.  The hook runs that cache with a stand-in ordinal."""
    f = lib.streambp_test_per_device_value
    assert f(0, 5) == 5 and f(0, 7) == 5          # first use on ordinal 0 decides; later calls see the cached value
    assert f(1, 7) == 7 and f(1, 9) == 7          # ordinal 1 has its own entry
    assert f(0, 11) == 5
    assert f(63, 3) == 3 and f(64, 4) == 4 and f(64, 6) == 6      # beyond the table: computed every time, never cached
    assert f(-1, 1) == B.E_SHAPE


def test_suggested_chunk_is_the_largest_that_fits(lib):
    """Sec. 4.3: partition size is the memory / time knob.  The suggestion is the largest multiple of 128 (or T)
    whose exact workspace fits the budget, checked against a scan of the planner."""
    import torch
    c = B.LayerConfig(4096, 32, 8, 128, 14336, False, 5e5, dtype=torch.bfloat16)
    T = 32768
    assert B.layer_suggest_chunk(c, T, 1 << 62) == T
    assert B.layer_suggest_chunk(c, T, B.layer_workspace_bytes(c, T, 128) - 1) == 0
    for budget in (int(0.81e9), int(1.5e9), B.layer_workspace_bytes(c, T, 2048), B.layer_workspace_bytes(c, T, 2048) - 1):
        got = B.layer_suggest_chunk(c, T, budget)
        assert got % 128 == 0 and 0 < got < T
        assert B.layer_workspace_bytes(c, T, got) <= budget < B.layer_workspace_bytes(c, T, got + 128)
    assert B.layer_suggest_chunk(c, T, B.layer_workspace_bytes(c, T, 2048)) == 2048
    assert B.layer_suggest_chunk(c, 100, B.layer_workspace_bytes(c, 100, 100)) == 100      # T itself when it fits
    h = B.HeadConfig(3584, 152064, dtype=torch.bfloat16)
    got = B.lmhead_suggest_chunk(h, 32768, int(1e9))
    assert got % 128 == 0 and B.lmhead_workspace_bytes(h, 32768, got) <= 1e9 < B.lmhead_workspace_bytes(h, 32768, got + 128)
    assert B.lmhead_suggest_chunk(h, 0, int(1e9)) == 0
