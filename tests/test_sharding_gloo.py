"""N > 1 host logic on CPU (gloo, world size 2): coordinate ranges, and the fact that ranks
working on their own shards with no data-path collective reproduce the unsharded step."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_1810_05291_b200 import inputs, sharding


@pytest.mark.parametrize("d", [0, 1, 31, 32, 33, 64, 1000, 25_557_032])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_shard_ranges_partition_the_coordinates(d, world):
    prev = 0
    sizes = []
    for r in range(world):
        a, b = sharding.shard_range(d, r, world)
        assert a == prev and a <= b <= d
        assert a % 32 == 0 or a == d
        prev = b
        sizes.append((b - a + 31) // 32)
    assert prev == d
    assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, d, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        case = inputs.cfg3(d)
        case.M = 5
        grads = inputs.gradients(case, "cpu", 0)
        x = inputs.initial_params(case, "cpu")
        a, b = sharding.shard_range(d, rank, world)
        g_np = [g[a:b].numpy().copy() for g in grads]
        moms = [np.zeros(b - a, dtype=np.float32) for _ in range(case.M)]
        x_np = x[a:b].numpy().copy()
        vote = oracle.fused_step(g_np, moms, x_np, case.beta, case.lr)
        # the step itself used no collective; gather only to check the result
        gathered = [None] * world
        dist.all_gather_object(gathered, (a, b, vote, x_np))
        t = sharding.max_over_ranks(1.0 + rank)
        if rank == 0:
            np.save(os.path.join(out_dir, "vote.npy"), np.concatenate([v for (_, _, v, _) in gathered]))
            np.save(os.path.join(out_dir, "x.npy"), np.concatenate([xx for (_, _, _, xx) in gathered]))
            np.save(os.path.join(out_dir, "t.npy"), np.array([t]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step(tmp_path):
    d, world = 32 * 301 + 8, 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, d, str(tmp_path)), nprocs=world, join=True)
    case = inputs.cfg3(d)
    case.M = 5
    grads = [g.numpy().copy() for g in inputs.gradients(case, "cpu", 0)]
    x = inputs.initial_params(case, "cpu").numpy().copy()
    moms = [np.zeros(d, dtype=np.float32) for _ in range(case.M)]
    vote = oracle.fused_step(grads, moms, x, case.beta, case.lr)
    assert np.array_equal(np.load(tmp_path / "vote.npy"), vote)
    assert np.array_equal(np.load(tmp_path / "x.npy"), x)
    assert float(np.load(tmp_path / "t.npy")[0]) == 2.0     # max over ranks of (1, 2)
