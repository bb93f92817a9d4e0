import numpy as np
import torch

from paper_2506_03077_b200 import synth


def test_normal_is_reproducible_and_sliceable():
    a = synth.normal(3, "t", (1000, 33))
    b = synth.normal(3, "t", (1000 * 33,))
    assert np.array_equal(a.ravel(), b)
    assert np.array_equal(synth.normal(3, "t", (50,)), b[:50])
    assert not np.array_equal(a, synth.normal(4, "t", (1000, 33)))
    assert not np.array_equal(a, synth.normal(3, "u", (1000, 33)))
    big = synth.normal(1, "big", (3 << 20,), 1.0, 0.02)
    assert abs(big.mean() - 1.0) < 1e-4 and abs(big.std() - 0.02) < 1e-4


def test_round_bf16_matches_torch():
    a = synth.normal(0, "r", (4096,), 0.0, 3.0)
    a[:4] = [0.0, -0.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8]   # ties
    ref = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert np.array_equal(synth.round_bf16(a), ref)


def test_integers_and_labels():
    x = synth.integers(5, "l", (100000,), 4096)
    assert x.min() >= 0 and x.max() < 4096 and x.dtype == np.int64
    assert len(np.unique(x)) > 4000
    g, W, H, labels = synth.make_head_inputs(synth.TINY_HEAD, 0, 512, False, 64)
    assert (labels[:64] == -100).all() and (labels[64:] >= 0).all()
    assert abs(float(g.mean()) - 1.0) < 0.01 and abs(float(W.std()) - 0.02) < 1e-3


def test_config_table_matches_declared_shapes():
    c = synth.CONFIGS
    assert c["tiny"].layer.dq == 256 and c["tiny"].layer.dkv == 128 and c["tiny"].layer.d_ff == 688
    assert c["qwen7b_layer"].layer.dq == 3584 and c["qwen7b_layer"].layer.dkv == 512
    assert c["llama8b_layer"].layer.dkv == 1024 and c["llama8b_layer"].T == 32768
    assert c["qwen7b_head"].head.vocab == 152064 and c["qwen7b_head"].masked_prefix == 8192
    assert c["qwen7b_model"].n_layers == 28
    w = synth.make_layer_weights(synth.TINY_LAYER, 0, True)
    assert "bq" not in w and w["w_down"].shape == (256, 688)
    assert np.array_equal(synth.round_bf16(w["wq"]), w["wq"])
