"""Data-parallel Moonwalk step: the batch is cut into equal shards, one per rank; parameters are
replicated; every step of the method is per sample except the weight vjp's sum over the batch
(Eq. "g_i"), so the only exchange is an all-reduce(sum) of each layer's gradient.  Algorithm 1
produces the gradients front to back: a bucket of the first layers can be reduced while the
sweep still works on the later ones (mw_sweep_bucket_events).

The partitioning, the loss scaling and the bucketed reduction below hold none of the method's
arithmetic; `torch.distributed` does the exchange (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import Callable, List, Sequence


def shard_bounds(batch: int, rank: int, world: int):
    """Rows [lo, hi) of the global batch that `rank` owns (equal shards)."""
    if batch % world != 0:
        raise ValueError(f"batch {batch} is not a multiple of the world size {world}")
    per = batch // world
    return rank * per, (rank + 1) * per


def gradient_scale(loss: str, world: int) -> float:
    """Factor that turns the SUM over ranks of per-shard gradients into the gradient of the global
    loss: mean losses are means over the shard on every rank (1 / world); the half sum of squares
    is a plain sum (1)."""
    return 1.0 if loss == "half_sse" else 1.0 / world


def buckets(n_layers: int, layers_per_bucket: int) -> List[range]:
    k = max(1, int(layers_per_bucket))
    return [range(b, min(b + k, n_layers)) for b in range(0, n_layers, k)]


def allreduce_gradients(grads: Sequence, loss: str, world: int, layers_per_bucket: int = 8, group=None,
                        wait_for: Callable[[int], None] = None) -> None:
    """In place: grads[l] <- scale * sum over ranks of grads[l], bucket by bucket in layer order.
    `wait_for(b)` (optional) is called before bucket b is touched: on GPUs it makes the reducing
    stream wait for the sweep's event of that bucket."""
    import torch.distributed as dist
    scale = gradient_scale(loss, world)
    for b, layers in enumerate(buckets(len(grads), layers_per_bucket)):
        if wait_for is not None:
            wait_for(b)
        for l in layers:
            if grads[l] is None:
                continue
            if world > 1:
                dist.all_reduce(grads[l], op=dist.ReduceOp.SUM, group=group)
            if scale != 1.0:
                grads[l].mul_(scale)


class DataParallelStep:
    """One rank of a data-parallel Moonwalk gradient step on a GPU.  The net is built for the
    SHARD's batch; `step` runs Phases I-II and the forward sweep on this rank's rows and reduces
    the gradients on a side stream, bucket by bucket, while the sweep is still running."""

    def __init__(self, net, loss: str, world: int, layers_per_bucket: int = 8, group=None, device="cuda"):
        import torch
        self.torch, self.net, self.loss, self.world, self.group = torch, net, loss, world, group
        self.k = max(1, int(layers_per_bucket))
        nb = len(buckets(len(net.layers), self.k))
        self.events = [torch.cuda.Event() for _ in range(nb)]
        for e in self.events:                      # a first record creates the event's handle
            e.record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        net.set_bucket_events(self.k, self.events)
        self.comm = torch.cuda.Stream(device=device)

    def step(self, params, x_shard, target_shard, workspace, g0, dW, loss_out=None):
        torch = self.torch
        main = torch.cuda.current_stream()
        self.net.input_cotangent(params, x_shard, target_shard, workspace, g0_out=g0, loss_out=loss_out)
        self.net.forward_sweep(params, x_shard, g0, workspace, dW_out=dW)
        with torch.cuda.stream(self.comm):
            allreduce_gradients(dW, self.loss, self.world, self.k, self.group,
                                wait_for=lambda b: self.comm.wait_event(self.events[b]))
        main.wait_stream(self.comm)
        return dW
