"""The multi-rank host path on CPU: two gloo ranks split one grid by event count, each
evaluates its shard (the CPU oracle stands in for the GPU estimator here: the test is
about sharding and gathering, not arithmetic), the slices are gathered and must equal
the unsharded result; scalar reductions give max and sum over ranks."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    import oracle
    from paper_2404_10933_b200 import grids, multi
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert multi.env_rank_world() == (rank, world, rank)
        cfgs = np.concatenate([grids.g1_small(), grids.g2_shape_grid(11, 1)[::5]])
        whole = oracle.estimate(cfgs, level=2)
        counts = oracle.estimate(cfgs[:0], level=1)["count"]  # empty call works
        assert counts.size == 0
        weights = np.array([oracle.event_count(cfgs[i:i + 1], formula=True)[1] for i in range(len(cfgs))])
        lo, hi = multi.shard_of(len(cfgs), weights, rank, world)
        mine = oracle.estimate(cfgs[lo:hi], level=2)
        peaks = multi.gather_slices(torch.from_numpy(mine["peak"]), len(cfgs), lo)
        assert np.array_equal(peaks.numpy(), whole["peak"])
        two_d = torch.from_numpy(np.stack([mine["peak"], mine["status"].astype(np.int64)], axis=1))
        both = multi.gather_slices(two_d, len(cfgs), lo)
        assert np.array_equal(both[:, 1].numpy(), whole["status"].astype(np.int64))
        # shards are contiguous, disjoint, cover everything and are balanced by weight
        los = multi.gather_slices(torch.tensor([[lo, hi]]), world, rank)
        assert los[0, 0] == 0 and los[-1, 1] == len(cfgs) and (los[1:, 0] == los[:-1, 1]).all()
        share = weights[lo:hi].sum() / weights.sum()
        assert abs(share - 1.0 / world) < 0.2
        assert multi.reduce_scalar(rank + 1.5, "max") == world + 0.5
        assert multi.reduce_scalar(float(hi - lo), "sum") == len(cfgs)
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_rank_sharding_and_gather(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_process_helpers_are_identity():
    from paper_2404_10933_b200 import multi
    assert multi.reduce_scalar(3.25, "max") == 3.25
    t = torch.arange(5)
    assert multi.gather_slices(t, 5, 0) is t
    assert multi.shard_of(10, None, 1, 2) == (5, 10)
