"""Seeded synthetic inputs shaped like long-sequence SFT workloads.

This module is shared by the tests, the CPU oracle's callers and the benchmark.
It holds no arithmetic of the streamed backward itself: only a counter-based
random generator (splitmix64 -> Box-Muller), bf16 rounding of the generated
values, and the tensor recipes of the benchmark configurations.

Every tensor is a pure function of (seed, tensor name, shape): value k of a
tensor depends only on its flat row-major index k, so any slice can be
regenerated without drawing the rest.
"""
from __future__ import annotations

import os
import zlib
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)
_BLOCK = 1 << 20


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """One splitmix64 output per 64-bit counter (vectorised, wrap-around)."""
    with np.errstate(over="ignore"):
        z = x + _GOLDEN
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        return z ^ (z >> _U64(31))


def _stream_key(seed: int, name: str) -> np.uint64:
    tag = zlib.crc32(name.encode("utf-8")) & 0xFFFFFFFF
    k = np.array([(int(seed) & 0xFFFFFFFF) << 32 | tag], dtype=_U64)
    return _splitmix64(_splitmix64(k))[0]


def random_bits(seed: int, name: str, n: int, offset: int = 0) -> np.ndarray:
    """n 64-bit words of stream (seed, name), starting at counter `offset`."""
    key = _stream_key(seed, name)
    out = np.empty(n, dtype=_U64)
    for s in range(0, n, _BLOCK):
        e = min(n, s + _BLOCK)
        ctr = np.arange(offset + s, offset + e, dtype=_U64)
        with np.errstate(over="ignore"):
            out[s:e] = _splitmix64(key + ctr * _GOLDEN)
    return out


def _normal_block(key, s, e, mean, std, out):
    inv53 = 1.0 / float(1 << 53)
    ctr = np.arange(2 * s, 2 * e, dtype=_U64)
    with np.errstate(over="ignore"):
        bits = _splitmix64(key + ctr * _GOLDEN)
    u = (bits >> _U64(11)).astype(np.float64)
    u1 = (u[0::2] + 1.0) * inv53          # (0, 1]
    u2 = u[1::2] * inv53                  # [0, 1)
    rad = np.sqrt(-2.0 * np.log(u1))
    ang = (2.0 * np.pi) * u2
    out[2 * s:2 * e:2] = (mean + std * rad * np.cos(ang)).astype(np.float32)
    out[2 * s + 1:2 * e:2] = (mean + std * rad * np.sin(ang)).astype(np.float32)


def normal(seed: int, name: str, shape, mean: float = 0.0, std: float = 1.0) -> np.ndarray:
    """float32 N(mean, std) tensor; elements 2k and 2k+1 share one Box-Muller pair."""
    n = int(np.prod(shape))
    npair = (n + 1) // 2
    out = np.empty(2 * npair, dtype=np.float32)
    key = _stream_key(seed, name)
    blocks = [(s, min(npair, s + _BLOCK)) for s in range(0, npair, _BLOCK)]
    if len(blocks) <= 1:
        for s, e in blocks:
            _normal_block(key, s, e, mean, std, out)
    else:
        with ThreadPoolExecutor(max_workers=min(len(blocks), os.cpu_count() or 1)) as ex:
            list(ex.map(lambda se: _normal_block(key, se[0], se[1], mean, std, out), blocks))
    return out[:n].reshape(shape)


def integers(seed: int, name: str, shape, high: int) -> np.ndarray:
    """int64 tensor, uniform in [0, high)."""
    n = int(np.prod(shape))
    bits = random_bits(seed, name, n)
    return (bits % _U64(high)).astype(np.int64).reshape(shape)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    with np.errstate(over="ignore"):
        r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


# --------------------------------------------------------------------------
# configurations
# --------------------------------------------------------------------------

IGNORE_INDEX = -100


@dataclass(frozen=True)
class LayerShape:
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    qkv_bias: bool
    rope_theta: float
    rms_eps: float = 1e-6

    @property
    def dq(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def dkv(self) -> int:
        return self.n_kv_heads * self.head_dim


@dataclass(frozen=True)
class HeadShape:
    d_model: int
    vocab: int
    rms_eps: float = 1e-6
    ignore_index: int = IGNORE_INDEX


TINY_LAYER = LayerShape(256, 4, 2, 64, 688, False, 1e4)
QWEN7B_LAYER = LayerShape(3584, 28, 4, 128, 18944, True, 1e6)
LLAMA8B_LAYER = LayerShape(4096, 32, 8, 128, 14336, False, 5e5)
TINY_HEAD = HeadShape(256, 4096)
QWEN7B_HEAD = HeadShape(3584, 152064)

LAYER_WEIGHT_NAMES = ("g1", "wq", "bq", "wk", "bk", "wv", "bv", "wo", "g2", "w_gate", "w_up", "w_down")


def layer_weight_shapes(s: LayerShape) -> Dict[str, tuple]:
    """Shapes of one decoder layer's parameters, matrices stored [out, in]."""
    shp = {
        "g1": (s.d_model,), "wq": (s.dq, s.d_model), "wk": (s.dkv, s.d_model), "wv": (s.dkv, s.d_model),
        "wo": (s.d_model, s.dq), "g2": (s.d_model,), "w_gate": (s.d_ff, s.d_model),
        "w_up": (s.d_ff, s.d_model), "w_down": (s.d_model, s.d_ff),
    }
    if s.qkv_bias:
        shp.update({"bq": (s.dq,), "bk": (s.dkv,), "bv": (s.dkv,)})
    return shp


def make_layer_weights(s: LayerShape, seed: int, bf16: bool, prefix: str = "layer0") -> Dict[str, np.ndarray]:
    """Matrices and biases ~ N(0, 0.02); RMSNorm gains ~ N(1, 0.02)."""
    out = {}
    for name, shp in layer_weight_shapes(s).items():
        mean = 1.0 if name in ("g1", "g2") else 0.0
        w = normal(seed, f"{prefix}.{name}", shp, mean, 0.02)
        out[name] = round_bf16(w) if bf16 else w
    return out


def make_layer_io(s: LayerShape, seed: int, T: int, bf16: bool, dy_std: float = 1e-3):
    """Layer input X ~ N(0,1) and upstream gradient dY ~ N(0, dy_std), both [T, d]."""
    X = normal(seed, "X", (T, s.d_model), 0.0, 1.0)
    dY = normal(seed, "dY", (T, s.d_model), 0.0, dy_std)
    if bf16:
        X, dY = round_bf16(X), round_bf16(dY)
    return X, dY


def make_head_inputs(h: HeadShape, seed: int, T: int, bf16: bool, masked_prefix: int):
    """Final-norm gain ~ N(1,0.02), W_vocab ~ N(0,0.02), H ~ N(0,1), labels uniform
    with the first `masked_prefix` rows set to the ignore index (prompt tokens)."""
    g = normal(seed, "g_final", (h.d_model,), 1.0, 0.02)
    W = normal(seed, "w_vocab", (h.vocab, h.d_model), 0.0, 0.02)
    H = normal(seed, "H", (T, h.d_model), 0.0, 1.0)
    if bf16:
        g, W, H = round_bf16(g), round_bf16(W), round_bf16(H)
    labels = integers(seed, "labels", (T,), h.vocab)
    labels[:masked_prefix] = h.ignore_index
    return g, W, H, labels


def make_model_tokens(vocab: int, seed: int, T: int, prompt_frac: float, ignore_index: int = IGNORE_INDEX):
    """Token ids uniform in the vocabulary; labels are the ids shifted by one with the
    last row and the prompt prefix (rows t with t+1 < floor(frac*T)) ignored."""
    ids = integers(seed, "ids", (T,), vocab)
    labels = np.full((T,), ignore_index, dtype=np.int64)
    labels[:-1] = ids[1:]
    n_prompt = int(prompt_frac * T)
    if n_prompt > 1:
        labels[: n_prompt - 1] = ignore_index
    return ids, labels


@dataclass
class BenchConfig:
    name: str
    seed: int
    bf16: bool
    T: int
    chunk: int
    layer: Optional[LayerShape] = None
    head: Optional[HeadShape] = None
    n_layers: int = 0
    masked_prefix: int = 0
    prompt_frac: float = 0.0
    chunk_head: int = 0
    notes: str = ""


CONFIGS = {
    "tiny": BenchConfig("tiny", 0, False, 512, 128, TINY_LAYER, TINY_HEAD, 1, masked_prefix=64, chunk_head=128),
    "qwen7b_layer": BenchConfig("qwen7b_layer", 1, True, 8192, 1024, QWEN7B_LAYER),
    "llama8b_layer": BenchConfig("llama8b_layer", 2, True, 32768, 2048, LLAMA8B_LAYER),
    "qwen7b_head": BenchConfig("qwen7b_head", 3, True, 32768, 1024, None, QWEN7B_HEAD, masked_prefix=8192),
    "qwen7b_model": BenchConfig("qwen7b_model", 4, True, 65536, 2048, QWEN7B_LAYER, QWEN7B_HEAD, 28,
                                prompt_frac=0.1, chunk_head=2048),
}
