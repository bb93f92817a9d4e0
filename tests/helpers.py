"""Shared test helpers: synthetic tensors -> device tensors, oracle comparison."""
import numpy as np
import torch

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import binding as B
from paper_2506_03077_b200 import synth

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}   # max relative Frobenius error per gradient tensor


def to_dev(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device="cuda", dtype=dtype).contiguous()


def layer_case(shape: synth.LayerShape, seed: int, T: int, dtype: torch.dtype, dy_std=1e-3, wstd=0.02):
    """Returns (oracle cfg, binding cfg, numpy weights, X, dY) with values already rounded to `dtype`."""
    bf = dtype == torch.bfloat16
    W = {}
    for name, shp in synth.layer_weight_shapes(shape).items():
        w = synth.normal(seed, f"layer0.{name}", shp, 1.0 if name in ("g1", "g2") else 0.0, wstd)
        W[name] = synth.round_bf16(w) if bf else w
    X, dY = synth.make_layer_io(shape, seed, T, bf, dy_std)
    ocfg = O.LayerCfg(shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff, shape.qkv_bias,
                      shape.rope_theta, shape.rms_eps)
    bcfg = B.LayerConfig(shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff,
                         shape.qkv_bias, shape.rope_theta, shape.rms_eps, dtype)
    return ocfg, bcfg, W, X, dY


def run_layer(bcfg, W, X, dY, chunk, pos0=0, accumulate=False, grads=None, wgrad_group=1, cu_seqlens=None):
    dt = bcfg.dtype
    Wd = {k: to_dev(v, dt) for k, v in W.items()}
    Xd, dYd = to_dev(X, dt), to_dev(dY, dt)
    if grads is None:
        grads = B.alloc_layer_grads(bcfg)
        if not accumulate:
            for g in grads.values():
                g.fill_(float("nan"))     # the call must overwrite, not add
    dX = torch.full_like(Xd, float("nan"))
    ws = B.alloc_workspace(B.layer_workspace_bytes(bcfg, X.shape[0], chunk, wgrad_group))
    B.layer_backward(bcfg, Wd, Xd, dYd, chunk, grads, dX, ws, pos0=pos0, accumulate=accumulate, wgrad_group=wgrad_group,
                     cu_seqlens=cu_seqlens)
    assert B.last_device_status(ws) == B.OK
    return dX, grads


# A relative Frobenius norm over a whole tensor cannot see a fault confined to a few rows: at 2e-2 three wrong rows
# of an [8192, d] tensor, or one mis-addressed 128-row tile of a 32k-row one, still pass.  So every comparison also
# bounds the error of each block of BLOCK_ROWS rows (and, for [rows, heads, head_dim] tensors, of each head's
# columns) by BLOCK_FACTOR x the tensor's tolerance, relative to that block's own reference norm -- or to a
# quarter of the mean block norm where the block itself is small (masked rows, keys few queries attend to).
BLOCK_ROWS = 128
BLOCK_FACTOR = 4.0


def block_errors(g: np.ndarray, ref: np.ndarray, heads: int = 1) -> np.ndarray:
    """[row blocks, heads] relative errors as described above; g, ref: float64, same shape, >= 1 dimension."""
    rows = ref.shape[0]
    g2 = g.reshape(rows, heads, -1)
    r2 = ref.reshape(rows, heads, -1)
    edges = list(range(0, rows, BLOCK_ROWS))
    num = np.add.reduceat(((g2 - r2) ** 2).sum(-1), edges, axis=0)
    den = np.add.reduceat((r2 ** 2).sum(-1), edges, axis=0)
    floor = den.mean() / 16.0
    return np.sqrt(num / np.maximum(np.maximum(den, floor), 1e-300))


def assert_close(name, got: torch.Tensor, ref: np.ndarray, tol: float, heads: int = 1):
    g = got.detach().float().cpu().numpy().astype(np.float64)
    assert np.isfinite(g).all(), f"{name}: non-finite values"
    ref = np.asarray(ref, dtype=np.float64)
    assert g.shape == ref.shape, f"{name}: shape {g.shape} vs {ref.shape}"
    err = O.rel_frobenius(g, ref)
    assert err <= tol, f"{name}: relative Frobenius error {err:.3e} > {tol:.1e}"
    if ref.ndim >= 1 and ref.size and np.linalg.norm(ref) > 0.0:
        be = block_errors(g, ref, heads)
        worst = np.unravel_index(np.argmax(be), be.shape)
        assert be[worst] <= BLOCK_FACTOR * tol, \
            f"{name}: rows {worst[0] * BLOCK_ROWS}.., head {worst[1]}: block error {be[worst]:.3e} > {BLOCK_FACTOR * tol:.1e}"
    return err


def compare_layer(ocfg, W, X, dY, dX, grads, tol, pos0=0):
    dX_ref, G_ref = O.layer_backward(ocfg, W, X, dY, pos0=pos0)
    errs = {"dX": assert_close("dX", dX, dX_ref, tol)}
    assert set(grads) == set(G_ref)
    for k in G_ref:
        errs[k] = assert_close(k, grads[k], G_ref[k], tol)
    return errs
