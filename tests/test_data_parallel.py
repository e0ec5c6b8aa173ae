"""Data-parallel partitioning of the Moonwalk step, with two gloo ranks on CPU: every rank takes its
shard of the batch through the oracle's Algorithm 1 and the bucketed all-reduce must reproduce the
gradient of the whole batch (the single-rank oracle), for a mean loss and for a sum loss."""
import os
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, loss, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from oracle import moonwalk_oracle as O
    from paper_2402_14212_b200 import data_parallel as dp
    from paper_2402_14212_b200 import synth as S
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    p = S.tiny_mlp(seed=3, depth=5, n=32, batch=24, reseed_every=2)
    lo, hi = dp.shard_bounds(p.batch, rank, world)
    mine = O.moonwalk(p.layers, p.params, p.x[lo:hi], p.target[lo:hi], loss, reseed_every=p.reseed_every)
    grads = [torch.from_numpy(np.array(g)) for g in mine["dW"]]
    seen = []
    dp.allreduce_gradients(grads, loss, world, layers_per_bucket=2, wait_for=seen.append)
    full = O.backprop(p.layers, p.params, p.x, p.target, loss)["dW"]
    err = max(float(np.abs(g.numpy() - f).max() / np.abs(f).max()) for g, f in zip(grads, full))
    out.put((rank, err, seen))
    dist.destroy_process_group()


@pytest.mark.parametrize("loss", ["mse_mean", "half_sse"])
def test_two_ranks_reproduce_the_full_batch_gradient(loss):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000 + (7 if loss == "half_sse" else 0)
    procs = [ctx.Process(target=_rank, args=(r, 2, port, loss, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, err, seen in got:
        assert err <= 1e-12, (rank, err)
        assert seen == [0, 1, 2]              # 5 layers in buckets of 2, signalled in layer order


def test_partition_helpers():
    sys.path.insert(0, ROOT)
    from paper_2402_14212_b200 import data_parallel as dp
    assert [dp.shard_bounds(24, r, 4) for r in range(4)] == [(0, 6), (6, 12), (12, 18), (18, 24)]
    with pytest.raises(ValueError):
        dp.shard_bounds(10, 0, 4)
    assert dp.gradient_scale("mse_mean", 4) == 0.25 and dp.gradient_scale("xent_mean", 2) == 0.5
    assert dp.gradient_scale("half_sse", 8) == 1.0
    assert [list(b) for b in dp.buckets(5, 2)] == [[0, 1], [2, 3], [4]]
