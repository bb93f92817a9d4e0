"""Pins for the CPU oracle: finite differences, closed forms and invariants.

None of these re-type the oracle's formulas: they compare its gradients with
difference quotients of its own forward value, with values fixed by the
mathematics (uniform softmax, single-key attention, orthogonality), or with an
independent PyTorch-autograd statement of the same layer (test_oracle_autograd).
"""
import os

import numpy as np
import pytest

from oracle import streambp_oracle as O
from paper_2506_03077_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_layer(bias, Hq=4, Hkv=2, dh=8, d=24, I=40, theta=1e4):
    return O.LayerCfg(d, Hq, Hkv, dh, I, bias, theta, 1e-6)


def rand_layer(cfg, seed, T, wstd=0.3):
    s = synth.LayerShape(cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ff,
                         cfg.qkv_bias, cfg.rope_theta, cfg.rms_eps)
    W = {k: synth.normal(seed, "w." + k, shp, 1.0 if k in ("g1", "g2") else 0.0, wstd).astype(np.float64)
         for k, shp in synth.layer_weight_shapes(s).items()}
    X = synth.normal(seed, "X", (T, cfg.d_model)).astype(np.float64)
    dY = synth.normal(seed, "dY", (T, cfg.d_model)).astype(np.float64)
    return W, X, dY


def directional_fd(f, theta, u, h):
    return (f(theta + h * u) - f(theta - h * u)) / (2 * h)


@pytest.mark.parametrize("bias", [False, True])
@pytest.mark.parametrize("pos0", [0, 37])
def test_layer_backward_matches_finite_differences(bias, pos0):
    cfg = small_layer(bias)
    T = 16
    W, X, dY = rand_layer(cfg, 5, T)
    dX, G = O.layer_backward(cfg, W, X, dY, pos0=pos0, row_block=5)

    def loss_with(name, val):
        if name == "X":
            return float(np.sum(dY * O.layer_forward(cfg, W, val, pos0, row_block=7)))
        W2 = dict(W)
        W2[name] = val
        return float(np.sum(dY * O.layer_forward(cfg, W2, X, pos0, row_block=7)))

    targets = {"X": (X, dX)}
    targets.update({k: (W[k], G[k]) for k in W})
    assert set(G) == set(W)
    for name, (val, grad) in targets.items():
        u = synth.normal(11, "dir." + name, val.shape).astype(np.float64)
        fd = directional_fd(lambda v: loss_with(name, v), val, u, 1e-5)
        an = float(np.sum(grad * u))
        assert abs(fd - an) <= 1e-6 * max(abs(fd), abs(an)) + 1e-9, (name, fd, an)
        # a few single entries
        flat = np.arange(val.size)
        for k in synth.integers(3, "pick." + name, (3,), val.size):
            e = np.zeros(val.size)
            e[k] = 1.0
            e = e.reshape(val.shape)
            fd1 = directional_fd(lambda v: loss_with(name, v), val, e, 1e-5)
            an1 = float(grad.reshape(-1)[k])
            assert abs(fd1 - an1) <= 2e-6 * max(abs(fd1), abs(an1)) + 1e-8, (name, int(k), fd1, an1)


def rand_head(seed, T, d, V, masked):
    cfg = O.HeadCfg(d, V, 1e-6, -100)
    g = synth.normal(seed, "g", (d,), 1.0, 0.1).astype(np.float64)
    Wv = synth.normal(seed, "wv", (V, d), 0.0, 0.3).astype(np.float64)
    H = synth.normal(seed, "H", (T, d)).astype(np.float64)
    labels = synth.integers(seed, "labels", (T,), V)
    labels[:masked] = -100
    return cfg, g, Wv, H, labels


def test_lmhead_backward_matches_finite_differences():
    cfg, g, Wv, H, labels = rand_head(2, 19, 12, 31, 4)
    labels[9] = -100
    loss, N, dH, dW, dg = O.lmhead_ce_backward(cfg, g, Wv, H, labels, row_block=4)
    assert N == 14
    loss_f, N_f = O.lmhead_ce_forward(cfg, g, Wv, H, labels, row_block=6)
    assert N_f == N and abs(loss - loss_f) < 1e-13
    cases = {
        "H": (H, dH, lambda v: O.lmhead_ce_forward(cfg, g, Wv, v, labels)[0]),
        "W": (Wv, dW, lambda v: O.lmhead_ce_forward(cfg, g, v, H, labels)[0]),
        "g": (g, dg, lambda v: O.lmhead_ce_forward(cfg, v, Wv, H, labels)[0]),
    }
    for name, (val, grad, f) in cases.items():
        u = synth.normal(4, "dir." + name, val.shape).astype(np.float64)
        fd = directional_fd(f, val, u, 1e-5)
        an = float(np.sum(grad * u))
        assert abs(fd - an) <= 1e-6 * max(abs(fd), abs(an)) + 1e-10, (name, fd, an)
    # masked rows receive exactly zero gradient
    assert np.all(dH[:4] == 0.0) and np.all(dH[9] == 0.0)
    # rows of softmax-minus-onehot sum to zero, hence the vocabulary sum of dW vanishes
    assert np.abs(dW.sum(axis=0)).max() < 1e-14


def test_model_backward_matches_finite_differences():
    lc = small_layer(True, Hq=2, Hkv=1, dh=4, d=8, I=12)
    hc = O.HeadCfg(8, 17, 1e-6, -100)
    T, L = 9, 2
    layers = [rand_layer(lc, 20 + l, T)[0] for l in range(L)]
    E = synth.normal(9, "E", (17, 8)).astype(np.float64)
    g = synth.normal(9, "g", (8,), 1.0, 0.1).astype(np.float64)
    Wv = synth.normal(9, "wv", (17, 8), 0.0, 0.3).astype(np.float64)
    ids = synth.integers(9, "ids", (T,), 17)
    ids[3] = ids[5]  # a repeated token exercises the scatter-add
    labels = np.full(T, -100, dtype=np.int64)
    labels[2:-1] = ids[3:]
    res = O.model_backward(lc, hc, layers, g, Wv, labels, embed=E, ids=ids, row_block=4)

    def f_E(v):
        return O.model_forward_loss(lc, hc, layers, g, Wv, labels, embed=v, ids=ids)

    def f_layer(l, name):
        def f(v):
            ls = [dict(w) for w in layers]
            ls[l][name] = v
            return O.model_forward_loss(lc, hc, ls, g, Wv, labels, embed=E, ids=ids)
        return f

    checks = [("E", E, res["d_embed"], f_E),
              ("g_final", g, res["g_final"], lambda v: O.model_forward_loss(lc, hc, layers, v, Wv, labels, embed=E, ids=ids)),
              ("w_vocab", Wv, res["w_vocab"], lambda v: O.model_forward_loss(lc, hc, layers, g, v, labels, embed=E, ids=ids))]
    for l in range(L):
        for name in ("wq", "bk", "w_down", "g1", "wv"):
            checks.append((f"l{l}.{name}", layers[l][name], res["layers"][l][name], f_layer(l, name)))
    for name, val, grad, f in checks:
        u = synth.normal(6, "dir." + name, val.shape).astype(np.float64)
        fd = directional_fd(f, val, u, 1e-5)
        an = float(np.sum(grad * u))
        assert abs(fd - an) <= 1e-6 * max(abs(fd), abs(an)) + 1e-10, (name, fd, an)
    # X0 path gives the same gradients as the embedding path
    res2 = O.model_backward(lc, hc, layers, g, Wv, labels, X0=E[ids])
    assert np.allclose(res2["dX0"], res["dX0"], rtol=0, atol=1e-15)
    assert res2["d_embed"] is None


def test_lmhead_zero_weight_closed_form():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "lmhead_zero_weight.txt")) if not l.startswith("#")]
    table = {int(v): float(x) for v, x in rows}
    V, d, T = 4096, 16, 12
    cfg = O.HeadCfg(d, V, 1e-6, -100)
    g = synth.normal(1, "g", (d,), 1.0, 0.02).astype(np.float64)
    H = synth.normal(1, "H", (T, d)).astype(np.float64)
    labels = synth.integers(1, "labels", (T,), V)
    labels[:3] = -100
    loss, N, dH, dW, dg = O.lmhead_ce_backward(cfg, g, np.zeros((V, d)), H, labels)
    assert N == 9
    assert abs(loss - table[V]) < 1e-12
    assert np.all(dH == 0.0) and np.all(dg == 0.0)
    # dW[v] = (1/N) sum_t (1/V - [v == y_t]) hn_t over unmasked rows
    hn = H / np.sqrt((H * H).mean(-1, keepdims=True) + 1e-6) * g
    expect = np.tile(hn[3:].sum(0) / (V * N), (V, 1))
    for t in range(3, T):
        expect[labels[t]] -= hn[t] / N
    assert np.abs(dW - expect).max() < 1e-15
    assert abs(np.log(152064.0) - table[152064]) < 1e-12


def test_single_token_attention_is_identity_on_v():
    # one key: softmax == 1, so o = v and no gradient reaches q, k (hence Wq, Wk, bq, bk)
    cfg = small_layer(True)
    W, X, dY = rand_layer(cfg, 8, 1)
    dX, G = O.layer_backward(cfg, W, X, dY, pos0=5)
    for k in ("wq", "wk", "bq", "bk"):
        assert np.all(G[k] == 0.0), k
    assert np.abs(G["wv"]).max() > 0


def test_causality_zero_upstream_tail_gives_zero_input_gradient_tail():
    cfg = small_layer(False)
    T, t0 = 12, 7
    W, X, dY = rand_layer(cfg, 3, T)
    dY[t0:] = 0.0
    dX, _ = O.layer_backward(cfg, W, X, dY)
    assert np.all(dX[t0:] == 0.0)
    assert np.abs(dX[:t0]).min() > 0
    # and the prefix gradient does not depend on the rows after it
    dX_short, _ = O.layer_backward(cfg, W, X[:t0], dY[:t0])
    assert np.allclose(dX[:t0], dX_short, rtol=1e-12, atol=1e-15)


def test_rope_is_an_isometry_and_relative():
    T, H, dh = 10, 3, 16
    u = synth.normal(2, "u", (T, H, dh)).astype(np.float64)
    w = synth.normal(2, "w", (T, H, dh)).astype(np.float64)
    cos, sin = O.rope_tables(100 + np.arange(T), dh, 5e5)
    ur = O.rope_apply(u, cos, sin)
    assert np.allclose(np.linalg.norm(ur, axis=-1), np.linalg.norm(u, axis=-1), rtol=1e-13)
    # transpose == inverse
    assert np.allclose(O.rope_apply_transpose(ur, cos, sin), u, atol=1e-13)
    # <rope(u), w> == <u, rope^T(w)>
    assert abs(np.sum(ur * w) - np.sum(u * O.rope_apply_transpose(w, cos, sin))) < 1e-11
    # position 0 is the identity; frequency 0 at position p rotates by p radians
    c0, s0 = O.rope_tables(np.array([0, 3]), dh, 1e4)
    assert np.all(c0[0] == 1.0) and np.all(s0[0] == 0.0)
    assert abs(c0[1, 0] - np.cos(3.0)) < 1e-15 and abs(s0[1, 0] - np.sin(3.0)) < 1e-15
    assert abs(c0[1, 1] - np.cos(3.0 * 1e4 ** (-2.0 / dh))) < 1e-15
    # pairing is (j, j + dh/2): rotating e_0 by position 3 lands in coordinates 0 and dh/2
    e = np.zeros((1, 1, dh)); e[0, 0, 0] = 1.0
    r = O.rope_apply(e, c0[1:2], s0[1:2])[0, 0]
    assert abs(r[0] - np.cos(3.0)) < 1e-15 and abs(r[dh // 2] - np.sin(3.0)) < 1e-15
    assert np.count_nonzero(r) == 2


def test_layer_gradients_do_not_depend_on_position_offset():
    cfg = small_layer(True)
    W, X, dY = rand_layer(cfg, 4, 14)
    dX0, G0 = O.layer_backward(cfg, W, X, dY, pos0=0)
    dX1, G1 = O.layer_backward(cfg, W, X, dY, pos0=12345)
    assert O.rel_frobenius(dX1, dX0) < 1e-10
    for k in G0:
        assert O.rel_frobenius(G1[k], G0[k]) < 1e-9, k


def test_rmsnorm_backward_closed_forms():
    T, d, eps = 6, 10, 1e-3
    x = synth.normal(1, "x", (T, d)).astype(np.float64)
    gain = synth.normal(1, "g", (d,), 1.0, 0.3).astype(np.float64)
    dh = synth.normal(1, "dh", (T, d)).astype(np.float64)
    h, xhat, rms = O.rmsnorm_forward(x, gain, eps)
    dx, dgain = O.rmsnorm_backward(dh, xhat, rms, gain)
    # <x_t, dx_t> = <x_t, w_t> eps / rms_t^3, so the gradient is orthogonal to x as eps -> 0
    w = dh * gain
    lhs = np.sum(x * dx, axis=-1)
    rhs = np.sum(x * w, axis=-1) * eps / rms[:, 0] ** 3
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-15)
    # unit gain, eps = 0: output rows have mean square 1
    h1, _, _ = O.rmsnorm_forward(x, np.ones(d), 0.0)
    assert np.allclose((h1 * h1).mean(-1), 1.0, rtol=1e-13)
    # scaling the input leaves the output unchanged when eps = 0
    h2, _, _ = O.rmsnorm_forward(3.0 * x, np.ones(d), 0.0)
    assert np.allclose(h1, h2, rtol=1e-13)


def test_attention_uniform_when_keys_are_equal():
    # identical keys => every causal row is a uniform average of the values seen so far
    T, Hq, Hkv, dh = 7, 4, 2, 8
    q = synth.normal(1, "q", (T, Hq, dh)).astype(np.float64)
    k = np.tile(synth.normal(1, "k", (1, Hkv, dh)).astype(np.float64), (T, 1, 1))
    v = synth.normal(1, "v", (T, Hkv, dh)).astype(np.float64)
    o = O.attention_forward(q, k, v, row_block=3)
    for h in range(Hq):
        expect = np.cumsum(v[:, h // 2, :], axis=0) / np.arange(1, T + 1)[:, None]
        assert np.allclose(o[:, h, :], expect, rtol=1e-13, atol=1e-15)


def test_attention_query_window_selects_rows_only():
    # evaluating the rows q_start.. alone gives those rows of the full result; their dk / dv contribution is what
    # the full backward gives when the upstream gradient of the other rows is zero (linearity in do)
    T, Hq, Hkv, dh, q0 = 19, 4, 2, 8, 11
    q = synth.normal(2, "q", (T, Hq, dh)).astype(np.float64)
    k = synth.normal(2, "k", (T, Hkv, dh)).astype(np.float64)
    v = synth.normal(2, "v", (T, Hkv, dh)).astype(np.float64)
    do = synth.normal(2, "do", (T, Hq, dh)).astype(np.float64)
    o = O.attention_forward(q, k, v, row_block=5)
    ow = O.attention_forward(q[q0:], k, v, row_block=3, q_start=q0)
    assert np.allclose(ow, o[q0:], rtol=1e-13, atol=1e-15)
    do0 = do.copy()
    do0[:q0] = 0.0
    dq, dk, dv = O.attention_backward(q, k, v, do0, row_block=5)
    dqw, dkw, dvw = O.attention_backward(q[q0:], k, v, do[q0:], row_block=4, q_start=q0)
    assert np.allclose(dqw, dq[q0:], rtol=1e-12, atol=1e-15)
    assert np.allclose(dkw, dk, rtol=1e-12, atol=1e-15) and np.allclose(dvw, dv, rtol=1e-12, atol=1e-15)
    assert np.abs(dq[:q0]).max() == 0.0


def test_row_block_is_only_a_memory_knob():
    cfg = small_layer(True)
    W, X, dY = rand_layer(cfg, 6, 21)
    a = O.layer_backward(cfg, W, X, dY, row_block=21)
    b = O.layer_backward(cfg, W, X, dY, row_block=4)
    assert O.rel_frobenius(b[0], a[0]) < 1e-13
    for k in a[1]:
        assert O.rel_frobenius(b[1][k], a[1][k]) < 1e-12, k


def test_two_linear_layers_streamed_sum_equals_one_shot():
    # App. A.1: Y = X W1, Z = Y W2, L = sum(Z) => dZ = 1, dY = dZ W2^T,
    # dW1 = sum_i X_i^T dY_i, dW2 = sum_i Y_i^T dZ_i for any row partition.
    D, m, n, k = 12, 5, 4, 3
    X = synth.normal(1, "X", (D, m)).astype(np.float64)
    W1 = synth.normal(1, "W1", (m, n)).astype(np.float64)
    W2 = synth.normal(1, "W2", (n, k)).astype(np.float64)
    dZ = np.ones((D, k))
    dW1 = X.T @ (dZ @ W2.T)
    dW2 = (X @ W1).T @ dZ
    s1, s2 = np.zeros_like(dW1), np.zeros_like(dW2)
    for rows in (slice(0, 5), slice(5, 6), slice(6, 12)):
        Yi = X[rows] @ W1
        dYi = dZ[rows] @ W2.T
        s1 += X[rows].T @ dYi
        s2 += Yi.T @ dZ[rows]
    assert np.allclose(s1, dW1, rtol=1e-13) and np.allclose(s2, dW2, rtol=1e-13)
    # closed form for this loss: dW2 = column sums of Y broadcast over k
    assert np.allclose(dW2, np.tile((X @ W1).sum(0)[:, None], (1, k)), rtol=1e-13)


def test_error_metrics():
    a = np.array([1.0, 2.0, 2.0])
    assert abs(O.rel_frobenius(a * 1.01, a) - 0.01) < 1e-12
    ea, er = O.paper_errors(a + 0.5, a)
    assert abs(ea - 0.5) < 1e-12 and abs(er - (0.5 + 0.25 + 0.25) / 3) < 1e-9


def test_packed_batch_is_a_set_of_independent_sequences():
    cfg = small_layer(True)
    W, X, dY = rand_layer(cfg, 9, 20)
    one = O.layer_backward(cfg, W, X, dY)
    packed_one = O.layer_backward_packed(cfg, W, X, dY, [0, 20])
    assert np.array_equal(one[0], packed_one[0]) and all(np.array_equal(one[1][k], packed_one[1][k]) for k in one[1])
    dXp, Gp = O.layer_backward_packed(cfg, W, X, dY, [0, 7, 20])
    X2 = X.copy()
    X2[7:] += 1.0                                       # changing the second sequence leaves the first one's dX alone
    dXq, _ = O.layer_backward_packed(cfg, W, X2, dY, [0, 7, 20])
    assert np.array_equal(dXp[:7], dXq[:7]) and not np.allclose(dXp[7:], dXq[7:])
    # and differs from treating the rows as one sequence
    assert O.rel_frobenius(dXp, one[0]) > 1e-3
