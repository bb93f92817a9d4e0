"""ctypes binding of libstreambp.so: the same entry points as include/streambp.h.

Only argument marshalling happens here (torch tensors -> device pointers, Python
dataclasses -> C structs); every step of the computation runs in the CUDA library.
There is no fallback: if the library is missing or cannot be loaded, importing
`lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstreambp.so")

STREAMBP_F32, STREAMBP_BF16 = 0, 1
OK = 0
E_NULL, E_SHAPE, E_ALIGN, E_WORKSPACE, E_DTYPE, E_CUDA, E_BAD_LABEL, E_NO_VALID_LABELS, E_DEVICE_TIMEOUT, \
    E_WORKSPACE_GUARD = range(-1, -11, -1)
OP_NT, OP_NN, OP_TN = 0, 1, 2

WEIGHT_FIELDS = ("g1", "wq", "bq", "wk", "bk", "wv", "bv", "wo", "g2", "w_gate", "w_up", "w_down")

EXPORTS = (
    "streambp_layer_workspace_bytes", "streambp_layer_backward",
    "streambp_lmhead_workspace_bytes", "streambp_lmhead_ce_backward",
    "streambp_model_workspace_bytes", "streambp_model_backward",
    "streambp_last_device_status", "streambp_status_string",
    "streambp_last_cuda_error", "streambp_last_launch_count", "streambp_gemm", "streambp_gemm_grouped", "streambp_gemm_swiglu",
    "streambp_layer_suggest_chunk", "streambp_lmhead_suggest_chunk",
    "streambp_profile_enable", "streambp_profile_read", "streambp_product_kernel",
    "streambp_attention_forward", "streambp_attention_backward", "streambp_attention_backward_static",
    "streambp_lmhead_rl_backward", "streambp_layer_backward_packed",
    "streambp_test_expire_wait", "streambp_test_per_device_value",
    "streambp_layer_workspace_bytes_grouped", "streambp_layer_backward_grouped", "streambp_test_workspace_guard",
    "streambp_lmhead_workspace_bytes_grouped", "streambp_lmhead_ce_backward_grouped",
    "streambp_lmhead_rl_backward_grouped",
)


class LayerCfgC(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("qkv_bias", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("dtype", C.c_int32)]


class LayerPtrsC(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in WEIGHT_FIELDS]


class HeadCfgC(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("vocab", C.c_int64), ("rms_eps", C.c_float),
                ("ignore_index", C.c_int64), ("dtype", C.c_int32)]


class RlCfgC(C.Structure):
    _fields_ = [("objective", C.c_int32), ("beta", C.c_float), ("clip_eps", C.c_float)]


class GemmProblemC(C.Structure):
    _fields_ = [("op", C.c_int32), ("n_segments", C.c_int32), ("M", C.c_int64), ("N", C.c_int64),
                ("A", C.c_void_p * 3), ("lda", C.c_int64 * 3), ("B", C.c_void_p * 3), ("ldb", C.c_int64 * 3),
                ("K", C.c_int64 * 3), ("C", C.c_void_p), ("ldc", C.c_int64), ("out_dtype", C.c_int32),
                ("accumulate", C.c_int32)]


class ModelCfgC(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("layer", LayerCfgC), ("head", HeadCfgC)]


class StreamBPError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


_lib = None


def lib() -> C.CDLL:
    """Load libstreambp.so (built by paper_2506_03077_b200.build). Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: build it with `python -m paper_2506_03077_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, sz, i32 = C.c_void_p, C.c_int64, C.c_size_t, C.c_int32
    L.streambp_layer_workspace_bytes.restype = sz
    L.streambp_layer_workspace_bytes.argtypes = [C.POINTER(LayerCfgC), i64, i64]
    L.streambp_layer_backward.restype = C.c_int
    L.streambp_layer_backward.argtypes = [C.POINTER(LayerCfgC), C.POINTER(LayerPtrsC), vp, vp, i64, i64, i64, C.c_int,
                                          C.POINTER(LayerPtrsC), vp, vp, sz, vp]
    L.streambp_layer_backward_packed.restype = C.c_int
    L.streambp_layer_backward_packed.argtypes = [C.POINTER(LayerCfgC), C.POINTER(LayerPtrsC), vp, vp, i64, i64,
                                                 C.POINTER(i64), i32, i64, C.c_int, C.POINTER(LayerPtrsC), vp, vp, sz, vp]
    L.streambp_layer_workspace_bytes_grouped.restype = sz
    L.streambp_layer_workspace_bytes_grouped.argtypes = [C.POINTER(LayerCfgC), i64, i64, i32]
    L.streambp_layer_backward_grouped.restype = C.c_int
    L.streambp_layer_backward_grouped.argtypes = [C.POINTER(LayerCfgC), C.POINTER(LayerPtrsC), vp, vp, i64, i64, i32,
                                                  C.POINTER(i64), i32, i64, C.c_int, C.POINTER(LayerPtrsC), vp, vp, sz, vp]
    L.streambp_lmhead_workspace_bytes.restype = sz
    L.streambp_lmhead_workspace_bytes.argtypes = [C.POINTER(HeadCfgC), i64, i64]
    L.streambp_lmhead_ce_backward.restype = C.c_int
    L.streambp_lmhead_ce_backward.argtypes = [C.POINTER(HeadCfgC), vp, vp, vp, vp, i64, i64, C.c_int, vp, vp, vp, vp,
                                              vp, vp, sz, vp]
    L.streambp_lmhead_rl_backward.restype = C.c_int
    L.streambp_lmhead_rl_backward.argtypes = [C.POINTER(HeadCfgC), C.POINTER(RlCfgC), vp, vp, vp, vp, vp, vp, vp, vp,
                                              i64, i64, C.c_int, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.streambp_lmhead_workspace_bytes_grouped.restype = sz
    L.streambp_lmhead_workspace_bytes_grouped.argtypes = [C.POINTER(HeadCfgC), i64, i64, i32]
    L.streambp_lmhead_ce_backward_grouped.restype = C.c_int
    L.streambp_lmhead_ce_backward_grouped.argtypes = [C.POINTER(HeadCfgC), vp, vp, vp, vp, i64, i64, i32, C.c_int, vp,
                                                      vp, vp, vp, vp, vp, sz, vp]
    L.streambp_lmhead_rl_backward_grouped.restype = C.c_int
    L.streambp_lmhead_rl_backward_grouped.argtypes = [C.POINTER(HeadCfgC), C.POINTER(RlCfgC), vp, vp, vp, vp, vp, vp,
                                                      vp, vp, i64, i64, i32, C.c_int, vp, vp, vp, vp, vp, vp, vp, sz,
                                                      vp]
    L.streambp_model_workspace_bytes.restype = sz
    L.streambp_model_workspace_bytes.argtypes = [C.POINTER(ModelCfgC), i64, i64, i64]
    L.streambp_model_backward.restype = C.c_int
    L.streambp_model_backward.argtypes = [C.POINTER(ModelCfgC), vp, C.POINTER(LayerPtrsC), vp, vp, vp, vp, vp, i64,
                                          i64, i64, C.c_int, vp, vp, C.POINTER(LayerPtrsC), vp, vp, vp, vp, sz, vp]
    L.streambp_last_device_status.restype = C.c_int
    L.streambp_last_device_status.argtypes = [vp, vp]
    L.streambp_status_string.restype = C.c_char_p
    L.streambp_status_string.argtypes = [C.c_int]
    L.streambp_last_cuda_error.restype = C.c_int
    L.streambp_last_cuda_error.argtypes = []
    L.streambp_last_launch_count.restype = i64
    L.streambp_last_launch_count.argtypes = []
    L.streambp_layer_suggest_chunk.restype = i64
    L.streambp_layer_suggest_chunk.argtypes = [C.POINTER(LayerCfgC), i64, sz]
    L.streambp_lmhead_suggest_chunk.restype = i64
    L.streambp_lmhead_suggest_chunk.argtypes = [C.POINTER(HeadCfgC), i64, sz]
    L.streambp_gemm_grouped.restype = C.c_int
    L.streambp_gemm_grouped.argtypes = [C.POINTER(GemmProblemC), i32, vp, vp]
    L.streambp_gemm_swiglu.restype = C.c_int
    L.streambp_gemm_swiglu.argtypes = [vp, i64, vp, vp, i64, i64, i64, i64, vp, vp, vp, i32, vp]
    L.streambp_gemm.restype = C.c_int
    L.streambp_gemm.argtypes = [C.c_int, i64, i64, i64, vp, i64, vp, i64, vp, i64, i32, i32, C.c_int, C.c_int, vp]
    L.streambp_attention_forward.restype = C.c_int
    L.streambp_attention_forward.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, i32, vp, vp, C.c_int, vp]
    L.streambp_attention_backward.restype = C.c_int
    L.streambp_attention_backward.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp,
                                              C.c_int, vp]
    L.streambp_attention_backward_static.restype = C.c_int
    L.streambp_attention_backward_static.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i32, i32, i32, i32, vp, vp, vp,
                                                     C.c_int, vp]
    L.streambp_product_kernel.restype = C.c_int
    L.streambp_product_kernel.argtypes = []
    L.streambp_profile_enable.restype = None
    L.streambp_profile_enable.argtypes = [C.c_int]
    L.streambp_profile_read.restype = C.c_int
    L.streambp_profile_read.argtypes = [C.c_int, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(C.c_double)]
    L.streambp_test_expire_wait.restype = C.c_int
    L.streambp_test_expire_wait.argtypes = [C.c_uint64, vp]
    L.streambp_test_workspace_guard.restype = C.c_int
    L.streambp_test_workspace_guard.argtypes = [vp, sz, i32, vp]
    L.streambp_test_per_device_value.restype = C.c_int
    L.streambp_test_per_device_value.argtypes = [C.c_int, C.c_int]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().streambp_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != OK:
        extra = ""
        if status == E_CUDA:
            extra = f" [cuda error {lib().streambp_last_cuda_error()}]"
        raise StreamBPError(status, what + extra)


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return STREAMBP_F32
    if dt == torch.bfloat16:
        return STREAMBP_BF16
    raise TypeError(f"unsupported storage dtype {dt}")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


@dataclass
class LayerConfig:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    qkv_bias: bool
    rope_theta: float
    rms_eps: float = 1e-6
    dtype: torch.dtype = torch.bfloat16

    def c(self) -> LayerCfgC:
        return LayerCfgC(self.d_model, self.n_q_heads, self.n_kv_heads, self.head_dim, self.d_ff,
                         1 if self.qkv_bias else 0, self.rope_theta, self.rms_eps, _dtype_code(self.dtype))


@dataclass
class HeadConfig:
    d_model: int
    vocab: int
    rms_eps: float = 1e-6
    ignore_index: int = -100
    dtype: torch.dtype = torch.bfloat16

    def c(self) -> HeadCfgC:
        return HeadCfgC(self.d_model, self.vocab, self.rms_eps, self.ignore_index, _dtype_code(self.dtype))


def _ptr_struct(tensors: Dict[str, torch.Tensor]) -> LayerPtrsC:
    return LayerPtrsC(**{f: _ptr(tensors.get(f)) for f in WEIGHT_FIELDS})


def layer_grad_shapes(cfg: LayerConfig) -> Dict[str, tuple]:
    dq, dkv, d, I = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim, cfg.d_model, cfg.d_ff
    shp = {"g1": (d,), "wq": (dq, d), "wk": (dkv, d), "wv": (dkv, d), "wo": (d, dq), "g2": (d,),
           "w_gate": (I, d), "w_up": (I, d), "w_down": (d, I)}
    if cfg.qkv_bias:
        shp.update({"bq": (dq,), "bk": (dkv,), "bv": (dkv,)})
    return shp


def alloc_layer_grads(cfg: LayerConfig, device="cuda") -> Dict[str, torch.Tensor]:
    return {k: torch.zeros(s, dtype=torch.float32, device=device) for k, s in layer_grad_shapes(cfg).items()}


def layer_workspace_bytes(cfg: LayerConfig, T: int, chunk: int, wgrad_group: int = 1) -> int:
    c = cfg.c()
    if wgrad_group != 1:
        return int(lib().streambp_layer_workspace_bytes_grouped(C.byref(c), T, chunk, wgrad_group))
    return int(lib().streambp_layer_workspace_bytes(C.byref(c), T, chunk))


def layer_suggest_chunk(cfg: LayerConfig, T: int, budget_bytes: int) -> int:
    """Largest chunk (multiple of 128 rows, or T) whose layer workspace fits budget_bytes; 0 if none does."""
    c = cfg.c()
    return int(lib().streambp_layer_suggest_chunk(C.byref(c), T, budget_bytes))


def lmhead_suggest_chunk(cfg: HeadConfig, T: int, budget_bytes: int) -> int:
    c = cfg.c()
    return int(lib().streambp_lmhead_suggest_chunk(C.byref(c), T, budget_bytes))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def layer_backward(cfg: LayerConfig, weights: Dict[str, torch.Tensor], X: torch.Tensor, dY: torch.Tensor,
                   chunk: int, grads: Dict[str, torch.Tensor], dX: torch.Tensor, workspace: torch.Tensor,
                   pos0: int = 0, accumulate: bool = False, stream=None, check: bool = True, wgrad_group: int = 1,
                   cu_seqlens: Optional[Sequence[int]] = None) -> int:
    """streambp_layer_backward (or streambp_layer_backward_grouped when wgrad_group != 1); returns the status
    (raises on error when check=True)."""
    c = cfg.c()
    w, g = _ptr_struct(weights), _ptr_struct(grads)
    if wgrad_group != 1:
        cu = (C.c_int64 * len(cu_seqlens))(*cu_seqlens) if cu_seqlens is not None else None
        st = lib().streambp_layer_backward_grouped(C.byref(c), C.byref(w), _ptr(X), _ptr(dY), X.shape[0], chunk,
                                                   wgrad_group, cu, len(cu_seqlens) - 1 if cu_seqlens is not None else 0,
                                                   pos0, 1 if accumulate else 0, C.byref(g), _ptr(dX), _ptr(workspace),
                                                   workspace.numel(), _stream_ptr(stream))
        if check:
            _check(st, "streambp_layer_backward_grouped")
        return st
    st = lib().streambp_layer_backward(C.byref(c), C.byref(w), _ptr(X), _ptr(dY), X.shape[0], chunk, pos0,
                                       1 if accumulate else 0, C.byref(g), _ptr(dX), _ptr(workspace),
                                       workspace.numel(), _stream_ptr(stream))
    if check:
        _check(st, "streambp_layer_backward")
    return st


class HostFedLayerBackward:
    """streambp_layer_backward for activations that live in pinned host memory (plumbing only: streams, events and
    copies; every step of the path still runs in the library's kernels).  Two sets of device buffers alternate:
    while the kernels of step k run on the compute stream, a copy stream brings in the X, dY of step k+1 and
    takes out the dX of step k-1, so a sequence's 3 T d storage-dtype values cross PCIe behind the compute of
    its neighbours instead of in front of its own."""

    def __init__(self, cfg: LayerConfig, weights, grads, T: int, chunk: int, workspace: torch.Tensor,
                 wgrad_group: int = 1):
        self.wgrad_group = wgrad_group
        self.cfg, self.weights, self.grads, self.chunk, self.ws = cfg, weights, grads, chunk, workspace
        dev = workspace.device
        mk = lambda: torch.empty(T, cfg.d_model, dtype=cfg.dtype, device=dev)
        self.X, self.dY, self.dX = [mk(), mk()], [mk(), mk()], [mk(), mk()]
        self.copy_stream = torch.cuda.Stream(device=dev)
        self.loaded = [torch.cuda.Event(), torch.cuda.Event()]      # inputs of buffer i are on the device
        self.computed = [torch.cuda.Event(), torch.cuda.Event()]    # the call on buffer i has finished
        self.n_prefetched = 0       # prefetch() calls so far; call k fills buffer pair k % 2
        self.n_run = 0              # step() calls so far; call k consumes buffer pair k % 2

    def prefetch(self, X_host: torch.Tensor, dY_host: torch.Tensor) -> None:
        """Starts the host-to-device copy of the inputs of the next step that has none yet (at most two ahead)."""
        assert self.n_prefetched - self.n_run < 2, "both buffer pairs hold inputs that have not been consumed"
        i = self.n_prefetched & 1
        cs = self.copy_stream
        if self.n_prefetched >= 2:
            cs.wait_event(self.computed[i])     # the previous user of these buffers is done with them
        with torch.cuda.stream(cs):
            self.X[i].copy_(X_host, non_blocking=True)
            self.dY[i].copy_(dY_host, non_blocking=True)
            self.loaded[i].record(cs)
        self.n_prefetched += 1

    def step(self, dX_host: torch.Tensor, accumulate: bool = False, stream=None) -> None:
        """Runs the backward on the oldest prefetched inputs and starts the copy of its dX to dX_host.  The copy
        stream is in order, so that copy also precedes the next prefetch into the same buffer pair."""
        assert self.n_run < self.n_prefetched, "prefetch() the inputs first"
        i = self.n_run & 1
        st = stream if stream is not None else torch.cuda.current_stream()
        st.wait_event(self.loaded[i])
        layer_backward(self.cfg, self.weights, self.X[i], self.dY[i], self.chunk, self.grads, self.dX[i], self.ws,
                       accumulate=accumulate, stream=st, wgrad_group=self.wgrad_group)
        self.computed[i].record(st)
        cs = self.copy_stream
        cs.wait_event(self.computed[i])
        with torch.cuda.stream(cs):
            dX_host.copy_(self.dX[i], non_blocking=True)
        self.n_run += 1

    def drain(self, stream=None) -> None:
        """Makes `stream` wait for the copies that are still in flight."""
        st = stream if stream is not None else torch.cuda.current_stream()
        st.wait_stream(self.copy_stream)


def layer_backward_packed(cfg: LayerConfig, weights, X, dY, chunk: int, cu_seqlens: Sequence[int], grads, dX, workspace,
                          pos0: int = 0, accumulate: bool = False, stream=None, check: bool = True) -> int:
    """streambp_layer_backward_packed: X, dY hold the sequences back to back; cu_seqlens = [0, ..., T] on the host."""
    c = cfg.c()
    w, g = _ptr_struct(weights), _ptr_struct(grads)
    n = len(cu_seqlens) - 1
    cu = (C.c_int64 * (n + 1))(*[int(v) for v in cu_seqlens])
    st = lib().streambp_layer_backward_packed(C.byref(c), C.byref(w), _ptr(X), _ptr(dY), X.shape[0], chunk, cu, n, pos0,
                                              1 if accumulate else 0, C.byref(g), _ptr(dX), _ptr(workspace),
                                              workspace.numel(), _stream_ptr(stream))
    if check:
        _check(st, "streambp_layer_backward_packed")
    return st


def lmhead_workspace_bytes(cfg: HeadConfig, T: int, chunk: int, wgrad_group: int = 1) -> int:
    c = cfg.c()
    if wgrad_group == 1:
        return int(lib().streambp_lmhead_workspace_bytes(C.byref(c), T, chunk))
    return int(lib().streambp_lmhead_workspace_bytes_grouped(C.byref(c), T, chunk, wgrad_group))


def lmhead_ce_backward(cfg: HeadConfig, g_final, w_vocab, H, labels, chunk: int, loss, n_valid, dH, d_w_vocab,
                       d_g_final, workspace, accumulate: bool = False, stream=None, check: bool = True,
                       wgrad_group: int = 1) -> int:
    """streambp_lmhead_ce_backward; wgrad_group != 1 goes through streambp_lmhead_ce_backward_grouped."""
    c = cfg.c()
    head = (C.byref(c), _ptr(g_final), _ptr(w_vocab), _ptr(H), _ptr(labels), H.shape[0], chunk)
    tail = (1 if accumulate else 0, _ptr(loss), _ptr(n_valid), _ptr(dH), _ptr(d_w_vocab), _ptr(d_g_final),
            _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if wgrad_group == 1:
        name, st = "streambp_lmhead_ce_backward", lib().streambp_lmhead_ce_backward(*head, *tail)
    else:
        name = "streambp_lmhead_ce_backward_grouped"
        st = lib().streambp_lmhead_ce_backward_grouped(*head, wgrad_group, *tail)
    if check:
        _check(st, name)
    return st


def _model_cfg(n_layers: int, layer: LayerConfig, head: HeadConfig) -> ModelCfgC:
    return ModelCfgC(n_layers, layer.c(), head.c())


def model_workspace_bytes(n_layers: int, layer: LayerConfig, head: HeadConfig, T: int, chunk_layer: int,
                          chunk_head: int) -> int:
    c = _model_cfg(n_layers, layer, head)
    return int(lib().streambp_model_workspace_bytes(C.byref(c), T, chunk_layer, chunk_head))


def model_backward(layer: LayerConfig, head: HeadConfig, layers: Sequence[Dict[str, torch.Tensor]], g_final, w_vocab,
                   labels, chunk_layer: int, chunk_head: int, loss, layer_grads: Sequence[Dict[str, torch.Tensor]],
                   d_g_final, d_w_vocab, workspace, embed=None, ids=None, X0=None, d_embed=None, dX0=None,
                   accumulate: bool = False, stream=None, check: bool = True) -> int:
    L = len(layers)
    c = _model_cfg(L, layer, head)
    W = (LayerPtrsC * L)(*[_ptr_struct(w) for w in layers])
    G = (LayerPtrsC * L)(*[_ptr_struct(g) for g in layer_grads])
    T = labels.shape[0]
    st = lib().streambp_model_backward(C.byref(c), _ptr(embed), W, _ptr(g_final), _ptr(w_vocab), _ptr(ids), _ptr(X0),
                                       _ptr(labels), T, chunk_layer, chunk_head, 1 if accumulate else 0, _ptr(loss),
                                       _ptr(d_embed), G, _ptr(d_g_final), _ptr(d_w_vocab), _ptr(dX0), _ptr(workspace),
                                       workspace.numel(), _stream_ptr(stream))
    if check:
        _check(st, "streambp_model_backward")
    return st


def last_device_status(workspace: torch.Tensor, stream=None) -> int:
    return int(lib().streambp_last_device_status(_ptr(workspace), _stream_ptr(stream)))


def last_launch_count() -> int:
    return int(lib().streambp_last_launch_count())


def gemm(op: int, A: torch.Tensor, B: torch.Tensor, C_out: torch.Tensor, accumulate: bool = False, engine: int = 0,
         stream=None, check: bool = True) -> int:
    """streambp_gemm on 2-D row-major tensors (leading dimension = stride(0))."""
    if op == OP_NT:
        M, K = A.shape
        N = B.shape[0]
    elif op == OP_NN:
        M, K = A.shape
        N = B.shape[1]
    else:
        K, M = A.shape
        N = B.shape[1]
    assert A.stride(1) == 1 and B.stride(1) == 1 and C_out.stride(1) == 1
    st = lib().streambp_gemm(op, M, N, K, A.data_ptr(), A.stride(0), B.data_ptr(), B.stride(0), C_out.data_ptr(),
                             C_out.stride(0), _dtype_code(A.dtype), _dtype_code(C_out.dtype), 1 if accumulate else 0,
                             engine, _stream_ptr(stream))
    if check:
        _check(st, "streambp_gemm")
    return st


def gemm_grouped(problems, sched: Optional[torch.Tensor] = None, stream=None, check: bool = True) -> int:
    """streambp_gemm_grouped.  problems: list of (op, [(A, B), ...], C_out, accumulate) with 2-D row-major bf16
    operands; each problem sums its (A, B) segments.  sched: None or an int32 CUDA tensor of two zeros."""
    arr = (GemmProblemC * len(problems))()
    for i, (op, segs, C_out, acc) in enumerate(problems):
        g = arr[i]
        g.op, g.n_segments = op, len(segs)
        for s, (A, B) in enumerate(segs):
            assert A.stride(1) == 1 and B.stride(1) == 1
            if op == OP_NT:
                M, K, N = A.shape[0], A.shape[1], B.shape[0]
            elif op == OP_NN:
                M, K, N = A.shape[0], A.shape[1], B.shape[1]
            else:
                K, M, N = A.shape[0], A.shape[1], B.shape[1]
            g.A[s], g.lda[s], g.B[s], g.ldb[s], g.K[s] = A.data_ptr(), A.stride(0), B.data_ptr(), B.stride(0), K
        g.M, g.N = M, N
        assert C_out.stride(1) == 1 and tuple(C_out.shape) == (M, N)
        g.C, g.ldc, g.out_dtype, g.accumulate = C_out.data_ptr(), C_out.stride(0), _dtype_code(C_out.dtype), 1 if acc else 0
    st = lib().streambp_gemm_grouped(arr, len(problems), _ptr(sched), _stream_ptr(stream))
    if check:
        _check(st, "streambp_gemm_grouped")
    return st


def gemm_swiglu(A, w_gate, w_up, g, u, m, stream=None, check: bool = True) -> int:
    """streambp_gemm_swiglu: g = A w_gate^T, u = A w_up^T, m = silu(g) * u; A [M, K], weights [N, K], outputs [M, N] dense."""
    M, K = A.shape
    N = w_gate.shape[0]
    assert A.stride(1) == 1 and w_gate.stride(1) == 1 and w_up.stride(1) == 1 and w_gate.stride(0) == w_up.stride(0)
    for t in (g, u, m):
        assert t.is_contiguous() and tuple(t.shape) == (M, N)
    st = lib().streambp_gemm_swiglu(_ptr(A), A.stride(0), _ptr(w_gate), _ptr(w_up), w_gate.stride(0), M, N, K, _ptr(g),
                                    _ptr(u), _ptr(m), _dtype_code(A.dtype), _stream_ptr(stream))
    if check:
        _check(st, "streambp_gemm_swiglu")
    return st


KERNEL_CLASSES = {"gemm": 0, "attention_fwd": 1, "attention_bwd": 2}


def test_expire_wait(limit_ns: int, stream=None) -> int:
    """Test hook: one tiny kernel whose bounded wait runs out after `limit_ns` (see streambp.h)."""
    return lib().streambp_test_expire_wait(int(limit_ns), _stream_ptr(stream))


test_expire_wait.__test__ = False     # a library call, not a pytest test


def product_kernel() -> str:
    """Which tcgen05 product kernel runs bf16 products on the current device."""
    return {2: "cta_pair", 1: "single_cta", 0: "none"}[lib().streambp_product_kernel()]


def profile_enable(on: bool) -> None:
    lib().streambp_profile_enable(1 if on else 0)


def profile_read(kernel_class: str):
    """(milliseconds, launches, algorithmic FLOPs) recorded for one kernel class."""
    ms, n, fl = C.c_double(), C.c_int64(), C.c_double()
    _check(lib().streambp_profile_read(KERNEL_CLASSES[kernel_class], C.byref(ms), C.byref(n), C.byref(fl)),
           "streambp_profile_read")
    return ms.value, n.value, fl.value


def attention_forward(q, k, v, q0: int, o, lse, engine: int = 0, stream=None, check: bool = True) -> int:
    """streambp_attention_forward; q, o: [n, Hq, dh], k, v: [q0+n, Hkv, dh], lse: [Hq, n] fp32."""
    n, Hq, dh = q.shape
    st = lib().streambp_attention_forward(_ptr(q), _ptr(k), _ptr(v), n, q0, Hq, k.shape[1], dh, _dtype_code(q.dtype),
                                          _ptr(o), _ptr(lse), engine, _stream_ptr(stream))
    if check:
        _check(st, "streambp_attention_forward")
    return st


def attention_backward(q, k, v, o, d_o, lse, q0: int, dq, dk, dv, engine: int = 0, stream=None,
                       check: bool = True) -> int:
    """streambp_attention_backward; dq fp32 overwritten, dk / dv fp32 accumulated."""
    n, Hq, dh = q.shape
    delta = torch.empty(Hq, n, dtype=torch.float32, device=q.device)
    st = lib().streambp_attention_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), n, q0, Hq,
                                           k.shape[1], dh, _dtype_code(q.dtype), _ptr(delta), _ptr(dq), _ptr(dk),
                                           _ptr(dv), engine, _stream_ptr(stream))
    if check:
        _check(st, "streambp_attention_backward")
    return st


STATIC_DELTA_MAX_FLOATS = 1 << 20


def attention_backward_static(q, k, v, o, d_o, lse, q0: int, dq, dk, dv, engine: int = 0, stream=None,
                              check: bool = True) -> int:
    """streambp_attention_backward_static: like attention_backward, but the row-sum scratch is the
    library's fixed 4 MiB array, so neither this wrapper nor the library allocates device memory.
    For callers that cannot allocate at call time.  Requires n * Hq <= STATIC_DELTA_MAX_FLOATS;
    calls that overlap on the GPU race on the shared array."""
    n, Hq, dh = q.shape
    st = lib().streambp_attention_backward_static(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), n, q0, Hq,
                                                  k.shape[1], dh, _dtype_code(q.dtype), _ptr(dq), _ptr(dk), _ptr(dv),
                                                  engine, _stream_ptr(stream))
    if check:
        _check(st, "streambp_attention_backward_static")
    return st


OBJ_GRPO, OBJ_DPO = 1, 2


def lmhead_rl_backward(cfg: HeadConfig, objective: int, beta: float, clip_eps: float, g_final, w_vocab, H, tokens,
                       logp_old, logp_ref, advantage, weight, chunk: int, loss, dH, d_w_vocab, d_g_final, workspace,
                       logp=None, ell=None, accumulate: bool = False, stream=None, check: bool = True,
                       wgrad_group: int = 1) -> int:
    """streambp_lmhead_rl_backward (GRPO / DPO objectives of the streamed LM head); wgrad_group != 1 goes through
    streambp_lmhead_rl_backward_grouped."""
    c = cfg.c()
    rl = RlCfgC(objective, beta, clip_eps)
    head = (C.byref(c), C.byref(rl), _ptr(g_final), _ptr(w_vocab), _ptr(H), _ptr(tokens), _ptr(logp_old),
            _ptr(logp_ref), _ptr(advantage), _ptr(weight), H.shape[0], chunk)
    tail = (1 if accumulate else 0, _ptr(loss), _ptr(logp), _ptr(ell), _ptr(dH), _ptr(d_w_vocab), _ptr(d_g_final),
            _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if wgrad_group == 1:
        name, st = "streambp_lmhead_rl_backward", lib().streambp_lmhead_rl_backward(*head, *tail)
    else:
        name = "streambp_lmhead_rl_backward_grouped"
        st = lib().streambp_lmhead_rl_backward_grouped(*head, wgrad_group, *tail)
    if check:
        _check(st, name)
    return st
