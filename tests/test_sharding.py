"""Two CPU processes over gloo: the batch shards over ranks with no exchange on the data path, and the all-reduced
gradient of M equals the single-process gradient over the concatenated batch; times reduce to the slowest rank's."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ref
from paper_2603_04127_b200 import inputs, sharding

WL = inputs.small(name="shard", wid=40, B=2, H=2, N=48, d=8, m=16, causal=True, dtype="f32", backward=True)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_tensors(rank):
    """Rank `rank`'s batch; the parameters M and W are rank 0's (replicated, as in data-parallel training)."""
    t = inputs.generate(sharding.rank_workload(WL, rank))
    t0 = inputs.generate(sharding.rank_workload(WL, 0))
    t.M, t.W = t0.M, t0.W
    return t


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert sharding.env_rank_world() == (rank, world, rank)
        t = _rank_tensors(rank)
        dQ, dK, dV, dM, _ = ref.backward(t.Q, t.K, t.V, t.M, t.W, t.dO, causal=True)
        dM = sharding.all_reduce_dm(torch.from_numpy(np.ascontiguousarray(dM)))
        slowest = sharding.max_over_ranks(10.0 + rank)            # rank r "took" 10 + r ms
        out[rank] = (dM.numpy().copy(), dQ, slowest)
    finally:
        dist.destroy_process_group()


def test_batch_sharding_over_two_gloo_ranks():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = {r: out[r] for r in range(world)}
    # single process, both ranks' batches concatenated
    ts = [_rank_tensors(r) for r in range(world)]
    cat = lambda name: np.concatenate([getattr(t, name) for t in ts], axis=0)
    dQ, dK, dV, dM, _ = ref.backward(cat("Q"), cat("K"), cat("V"), ts[0].M, ts[0].W, cat("dO"), causal=True)
    for r in range(world):
        np.testing.assert_allclose(res[r][0], dM, rtol=1e-10, atol=1e-12)            # every rank holds the full-batch dM
        np.testing.assert_allclose(res[r][1], dQ[r * WL.B:(r + 1) * WL.B], rtol=1e-12, atol=1e-14)   # data path: no exchange
        assert res[r][2] == 11.0                                                      # the slowest rank's time
    assert not np.allclose(ts[0].Q, ts[1].Q)                                          # the ranks' batches differ
    assert sharding.job_throughput(100.0, 2, 0.5) == 400.0


def test_single_process_helpers_are_no_ops():
    x = torch.ones(3)
    assert sharding.all_reduce_dm(x) is x and float(x.sum()) == 3.0
    assert sharding.max_over_ranks(2.5) == 2.5
    assert sharding.rank_workload(WL, 0) == WL and sharding.rank_workload(WL, 3).wid == WL.wid + 300
