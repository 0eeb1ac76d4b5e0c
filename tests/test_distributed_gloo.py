"""The one-worker-per-process form of Algorithm 1 on CPU (gloo, world sizes 2 and 3).

The kernels need a GPU, so here the CPU oracle stands in for them and what is under test is the
host side of ``paper_1810_05291_b200.distributed``: buffer sizes, slice arithmetic, padding and
the collectives. Every rank rebuilds all M gradients from the seed, plays its own worker through
``PackedExchange``, and must end with the parameters and the packed vote that the oracle's
M-worker step gives, in both exchange layouts.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_1810_05291_b200.distributed import PackedExchange, packed_words


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _as_i32(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(a.view(np.int32).copy())


def _as_u32(t: torch.Tensor) -> np.ndarray:
    return t.numpy().view(np.uint32).copy()


def _rank_main(rank, world, port, d, mode, flip):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        beta, lr, wd = 0.9, 1e-3, 0.01
        rng = np.random.default_rng(1234 + d)
        x0 = rng.standard_normal(d).astype(np.float32)
        ex = PackedExchange(d, world, rank, "cpu", mode)
        x = x0.copy()                                   # this worker's copy of the parameters
        v = np.zeros(d, dtype=np.float32)               # this worker's momentum
        ref_x = x0.copy()
        ref_v = [np.zeros(d, dtype=np.float32) for _ in range(world)]
        for step in range(3):
            grads = [rng.standard_normal(d).astype(np.float32) for _ in range(world)]
            want = oracle.fused_step(grads, ref_v, ref_x, beta, lr, wd, flip)
            # worker side (kernel stand-in: the oracle), written where the kernel would write
            ex.local_words().copy_(_as_i32(oracle.signum_update(grads[rank], v, beta)))
            if mode == "allgather":
                ex.gather()
                rows = [_as_u32(r) for r in ex.worker_rows()]
                vote = oracle.majority_vote(rows, d, flip)
            else:
                ex.scatter_slices()
                n = ex.slice_coordinates()
                assert len(ex.slice_rows()) == world
                if n > 0:
                    rows = [_as_u32(r) for r in ex.slice_rows()]
                    ex.slice_vote().copy_(_as_i32(oracle.majority_vote(rows, n, flip)))
                ex.gather_vote()
                vote = _as_u32(ex.vote_words())
            oracle.apply_vote(x, vote, lr, wd)
            assert np.array_equal(vote, want), "rank %d step %d: vote differs" % (rank, step)
            assert np.array_equal(x.view(np.uint32), ref_x.view(np.uint32)), "rank %d: x differs" % rank
            assert np.array_equal(v.view(np.uint32), ref_v[rank].view(np.uint32))
        # all workers hold the same parameters (Algorithm 1 keeps one copy of x per worker)
        digest = torch.from_numpy(x.copy())
        other = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(other, digest)
        for o in other:
            assert torch.equal(o, digest)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("mode,world,d,flip", [
    ("allgather", 2, 100_003, 0b01), ("allgather", 3, 70, 0),
    ("sharded", 2, 1000, 0), ("sharded", 3, 1000, 0b100), ("sharded", 3, 33, 0b010),
    ("sharded", 2, 100_003, 0b01)])
def test_workers_over_gloo_reproduce_the_m_worker_step(world, d, flip, mode):
    mp.spawn(_rank_main, args=(world, _free_port(), d, mode, flip), nprocs=world, join=True)


@pytest.mark.parametrize("d,world", [(1, 1), (1, 4), (31, 2), (32, 2), (33, 2), (1000, 3), (1024, 4),
                                     (25_557_032, 15), (61_100_840, 7)])
def test_slices_partition_the_words(d, world):
    W = packed_words(d)
    covered = 0
    for r in range(world):
        ex = PackedExchange(d, world, r, "meta", "sharded")
        assert ex.W == W and ex.W_pad == ex.slice_words * world >= W
        assert ex.W_pad - W < 4 * world                  # fewer than four padding words per worker
        assert ex.slice_words % 4 == 0                   # rows and slices start on 16-byte boundaries
        n = ex.slice_coordinates()
        assert 0 <= n <= 32 * ex.slice_words
        assert (n % 32 == 0) or (32 * r * ex.slice_words + n == d)   # only the slice holding the end is ragged
        covered += n
    assert covered == d


def test_bytes_per_step_follow_the_papers_count():
    # Appendix B: 2 M d bits per iteration over the whole system. All-gather moves (M-1) d/8 bytes
    # into every worker; the sharded server about 2 (M-1)/M d/8.
    d, M = 25_557_032, 15
    W = packed_words(d)
    ag = PackedExchange(d, M, 0, "meta", "allgather").bytes_received_per_step()
    sh = PackedExchange(d, M, 0, "meta", "sharded").bytes_received_per_step()
    assert abs(ag - (M - 1) * 4 * W) <= (M - 1) * 4 * 4 * M
    assert abs(sh - 2 * (M - 1) * 4 * W / M) <= 2 * (M - 1) * 4 * 4
    assert sh * 7 < ag
