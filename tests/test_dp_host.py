"""Data-parallel plumbing on CPU: the flat gradient bucket and, with two gloo ranks, the one-exchange-per-layer
rule of the paper's distributed design (Sec. 3.3 / App. A.3): every rank sums its own sequence's gradient
first; the reduce-scatter of the finished sums gives each rank its shard of the batch gradient."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from oracle import streambp_oracle as O  # noqa: E402
from paper_2506_03077_b200 import dp, synth  # noqa: E402

SHAPES = {"g1": (40,), "wq": (48, 40), "bq": (48,), "wk": (16, 40), "w_down": (40, 100)}


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_bucket_layout(world):
    table, total = dp.bucket_layout(SHAPES, world)
    assert total % (world * dp.ALIGN_ELEMS) == 0
    end = 0
    for name, shp in SHAPES.items():
        off, n = table[name]
        assert off % dp.ALIGN_ELEMS == 0 and off >= end and n == int(np.prod(shp))
        end = off + n
    assert end <= total < end + world * dp.ALIGN_ELEMS + dp.ALIGN_ELEMS
    b = dp.GradBucket(SHAPES, world, device="cpu")
    # views alias the flat buffer; the shards tile it; every element of every tensor has exactly one owner
    b.views["wk"].fill_(3.0)
    o, n = b.table["wk"]
    assert float(b.flat[o:o + n].sum()) == 3.0 * n and float(b.flat.sum()) == 3.0 * n
    owned = {k: 0 for k in SHAPES}
    for r in range(world):
        lo, hi = b.shard_range(r)
        assert hi - lo == b.shard_elems
        for k, (a, e) in b.owner_slices(r).items():
            owned[k] += e - a
    assert owned == {k: int(np.prod(s)) for k, s in SHAPES.items()}


def _rank_main(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shape = synth.LayerShape(32, 2, 1, 16, 48, True, 1e4)
    T = 24
    W = synth.make_layer_weights(shape, 9, False)
    ocfg = O.LayerCfg(shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.d_ff, shape.qkv_bias,
                      shape.rope_theta, shape.rms_eps)
    ios = [synth.make_layer_io(shape, 90 + r, T, False) for r in range(world)]
    # this rank's finished sum over its own sequence (the oracle stands in for the library on CPU)
    _, G = O.layer_backward(ocfg, W, ios[rank][0], ios[rank][1])
    shapes = {k: v.shape for k, v in G.items()}
    bucket = dp.GradBucket(shapes, world, device="cpu")
    for k, v in G.items():
        bucket.views[k].copy_(torch.from_numpy(np.ascontiguousarray(v)).float())
    shard = torch.zeros(bucket.shard_elems)
    dp.reduce_scatter_sum(bucket.flat, shard)
    full = dp.gather_full_gradients(bucket, shard)
    # the batch gradient: both sequences as one packed batch
    X = np.concatenate([io[0] for io in ios]); dY = np.concatenate([io[1] for io in ios])
    _, Gb = O.layer_backward_packed(ocfg, W, X, dY, [T * i for i in range(world + 1)])
    worst = max(O.rel_frobenius(full[k].double().numpy(), Gb[k]) for k in Gb)
    # this rank's shard is its slice of the reassembled flat sum
    lo, hi = bucket.shard_range(rank)
    flat_sum = torch.zeros(bucket.total)
    for k, (o, n) in bucket.table.items():
        flat_sum[o:o + n] = full[k].flatten()
    own_ok = bool(torch.equal(shard, flat_sum[lo:hi]))
    q.put((rank, worst, hi - lo, own_ok))
    dist.barrier()
    dist.destroy_process_group()


def test_reduce_scatter_after_local_accumulation_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29600 + os.getpid() % 300
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=300) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(g[0] for g in got) == [0, 1]
    for _, worst, n, own_ok in got:
        assert worst < 1e-6          # fp32 bucket against the fp64 batch gradient
        assert n > 0 and own_ok
