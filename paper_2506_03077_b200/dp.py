"""Data-parallel streamed backward: one process per GPU, each on its own sequences, and ONE exchange per layer.

The paper's distributed setting (Sec. 3.3 and App. A.3, "Distributed StreamBP", gradient communication
design) keeps the sequence-partitioned accumulation local to a rank: g_W is summed over the partitions D of that rank's sequences first, and only the
finished per-layer sum crosses the interconnect -- one gradient reduce-scatter (or all-reduce) per layer after
its chunk loop, instead of one per partition.  This module is the plumbing for that:

  * GradBucket  -- every fp32 weight-gradient tensor of a layer is a view into one flat buffer, each view
                   256-byte aligned (the C ABI wants 16), the total padded so that it splits evenly over the
                   ranks.  The library accumulates into the views; the exchange sees one contiguous tensor.
  * reduce_scatter_sum / all_reduce_sum -- torch.distributed on whatever backend the group has (NCCL over
                   NVLink / NVSwitch on GPUs; gloo on CPU, where reduce-scatter is an all-reduce plus a slice).
  * DataParallelLayerBackward -- layer backward on the compute stream, then the bucket's reduce-scatter on a
                   communication stream, so that the exchange of layer l overlaps the chunk loop of layer l-1.

Nothing here computes a gradient: the arithmetic is the library's (streambp_layer_backward) and NCCL's sum.
No kernel of the library reads another GPU's memory, and no TMA multicast is used anywhere.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import torch
import torch.distributed as dist

ALIGN_ELEMS = 64          # 256 bytes of fp32


def bucket_layout(shapes: Dict[str, Tuple[int, ...]], world: int) -> Tuple[Dict[str, Tuple[int, int]], int]:
    """Offsets (in fp32 elements) of every tensor inside the flat bucket and the padded total.

    Tensors are laid out in the order of `shapes`, each starting on a 256-byte boundary; the total is rounded
    up to a multiple of world * ALIGN_ELEMS so that every rank's shard has the same size and alignment."""
    if world < 1:
        raise ValueError("world must be >= 1")
    off, table = 0, {}
    for name, shp in shapes.items():
        n = 1
        for s in shp:
            n *= int(s)
        off = (off + ALIGN_ELEMS - 1) // ALIGN_ELEMS * ALIGN_ELEMS
        table[name] = (off, n)
        off += n
    unit = world * ALIGN_ELEMS
    total = (off + unit - 1) // unit * unit
    return table, total


class GradBucket:
    """Flat fp32 gradient storage of one layer with named views."""

    def __init__(self, shapes: Dict[str, Tuple[int, ...]], world: int, device="cuda"):
        self.shapes, self.world = dict(shapes), world
        self.table, self.total = bucket_layout(shapes, world)
        self.flat = torch.zeros(self.total, dtype=torch.float32, device=device)
        self.views = {k: self.flat[o:o + n].view(self.shapes[k]) for k, (o, n) in self.table.items()}
        self.shard_elems = self.total // world

    def shard_range(self, rank: int) -> Tuple[int, int]:
        return rank * self.shard_elems, (rank + 1) * self.shard_elems

    def owner_slices(self, rank: int) -> Dict[str, Tuple[int, int]]:
        """For each tensor, the [begin, end) range of its flattened elements that rank's shard holds."""
        lo, hi = self.shard_range(rank)
        out = {}
        for k, (o, n) in self.table.items():
            a, b = max(lo, o), min(hi, o + n)
            if a < b:
                out[k] = (a - o, b - o)
        return out


def reduce_scatter_sum(flat: torch.Tensor, shard: torch.Tensor, group=None) -> None:
    """shard <- this rank's slice of the element-wise sum of `flat` over the group."""
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    n = flat.numel() // world
    assert flat.numel() == n * world and shard.numel() == n
    if dist.get_backend(group) == "nccl":
        dist.reduce_scatter_tensor(shard, flat, op=dist.ReduceOp.SUM, group=group)
    else:   # gloo has no reduce-scatter: same result through an all-reduce
        tmp = flat.clone()
        dist.all_reduce(tmp, op=dist.ReduceOp.SUM, group=group)
        shard.copy_(tmp[rank * n:(rank + 1) * n])


def all_reduce_sum(flat: torch.Tensor, group=None) -> None:
    dist.all_reduce(flat, op=dist.ReduceOp.SUM, group=group)


class DataParallelLayerBackward:
    """streambp_layer_backward on this rank's sequence, then one reduce-scatter of the layer's gradient bucket.

    step() enqueues the backward on the compute stream and the exchange on a communication stream that waits
    for it; the caller goes on to the next layer (or the next micro-batch with accumulate=True, in which case
    it passes exchange=False until the last one) and calls wait() before reading `shard`."""

    def __init__(self, cfg, weights, T: int, chunk: int, group=None, device="cuda"):
        from . import binding as B
        self.B, self.cfg, self.weights, self.chunk, self.group = B, cfg, weights, chunk, group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.bucket = GradBucket(B.layer_grad_shapes(cfg), self.world, device)
        self.shard = torch.zeros(self.bucket.shard_elems, dtype=torch.float32, device=device)
        self.ws = B.alloc_workspace(B.layer_workspace_bytes(cfg, T, chunk), device)
        self.comm_stream = torch.cuda.Stream(device=device)
        self.computed = torch.cuda.Event()
        self.exchanged = torch.cuda.Event()

    def step(self, X, dY, dX, accumulate: bool = False, exchange: bool = True, stream=None) -> None:
        st = stream if stream is not None else torch.cuda.current_stream()
        st.wait_event(self.exchanged)      # a previous exchange may still be reading the bucket (no-op before the first)
        self.B.layer_backward(self.cfg, self.weights, X, dY, self.chunk, self.bucket.views, dX, self.ws,
                              accumulate=accumulate, stream=st)
        if not exchange:
            return
        self.computed.record(st)
        self.comm_stream.wait_event(self.computed)
        with torch.cuda.stream(self.comm_stream):
            if self.world > 1:
                reduce_scatter_sum(self.bucket.flat, self.shard, self.group)
            else:
                self.shard.copy_(self.bucket.flat)
            self.exchanged.record(self.comm_stream)

    def wait(self, stream=None) -> None:
        st = stream if stream is not None else torch.cuda.current_stream()
        st.wait_event(self.exchanged)


def gather_full_gradients(bucket: GradBucket, shard: torch.Tensor, group=None) -> Dict[str, torch.Tensor]:
    """All ranks' shards reassembled into named tensors (for tests and for optimizers that want full tensors)."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world > 1:
        parts: List[torch.Tensor] = [torch.empty_like(shard) for _ in range(world)]
        dist.all_gather(parts, shard, group=group)
        flat = torch.cat(parts)
    else:
        flat = shard
    return {k: flat[o:o + n].view(bucket.shapes[k]).clone() for k, (o, n) in bucket.table.items()}
