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
from paper_1810_05291_b200.distributed import (MajorityVoteWorker, PackedExchange, collective_barrier,
                                               packed_words)


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


class OracleKernels:
    """Stand-in for the CUDA binding on CPU ranks: the same ``ss_*`` names and in-place behaviour,
    served by the CPU oracle on views of the torch tensors. Only the tests use it; it lets
    ``MajorityVoteWorker.step`` run unchanged, so that what is exercised is the order of kernels
    and collectives and the buffers they are handed."""

    def __init__(self):
        self.calls = []

    @staticmethod
    def _f32(t):
        return t.numpy()

    @staticmethod
    def _u32(t):
        return t.numpy().view(np.uint32)

    def ss_sign_pack(self, grad, out_words, stream=None):
        self.calls.append("ss_sign_pack")
        self._u32(out_words)[:] = oracle.sign_pack(self._f32(grad))

    def ss_signum_update(self, grad, momentum, beta, out_words, stream=None):
        self.calls.append("ss_signum_update")
        self._u32(out_words)[:] = oracle.signum_update(self._f32(grad), self._f32(momentum), beta)

    def ss_signum_update_push(self, grad, momentum, beta, dests, stream=None):
        self.calls.append("ss_signum_update_push")
        words = oracle.signum_update(self._f32(grad), self._f32(momentum), beta)
        for dst in dests:
            self._u32(dst)[:] = words

    def ss_majority_vote(self, packed, d, flip_mask, vote_words, stream=None):
        self.calls.append("ss_majority_vote")
        self._u32(vote_words)[:] = oracle.majority_vote([self._u32(p).copy() for p in packed], d, flip_mask)

    def ss_apply_vote(self, param, vote_words, lr, weight_decay=0.0, stream=None):
        self.calls.append("ss_apply_vote")
        oracle.apply_vote(self._f32(param), self._u32(vote_words).copy(), lr, weight_decay)

    def ss_vote_apply(self, packed, param, lr, weight_decay=0.0, flip_mask=0, vote_words_out=None, stream=None):
        self.calls.append("ss_vote_apply")
        vote = oracle.majority_vote([self._u32(p).copy() for p in packed], param.numel(), flip_mask)
        oracle.apply_vote(self._f32(param), vote, lr, weight_decay)
        if vote_words_out is not None:
            self._u32(vote_words_out)[:] = vote


EXPECTED_ORDER = {
    "allgather": ["start", "kernel:pack", "exchange:all_gather", "kernel:vote_apply"],
    "sharded": ["start", "kernel:pack", "exchange:all_to_all", "kernel:vote", "exchange:all_gather",
                "kernel:apply"],
    "push": ["start", "kernel:pack", "exchange:barrier", "kernel:vote_apply", "exchange:barrier"],
}


def _worker_main(rank, world, port, d, mode, flip, beta, shared):
    """One rank = one MajorityVoteWorker driven through step(); the oracle serves as its kernels."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lr, wd = 1e-3, 0.01
        rng = np.random.default_rng(4321 + d)
        x0 = rng.standard_normal(d).astype(np.float32)
        phases = []
        kernels = OracleKernels()
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()), beta, lr, wd, mode, world=world, rank=rank,
                               kernels=kernels, on_phase=phases.append)
        if mode == "push":
            # the receive buffers live in shared memory: a stand-in for peer-mapped device memory,
            # written by the other ranks' processes and ordered only by the barrier
            w.ex.gathered = shared[rank]
            slot = lambda buf: buf[rank * w.ex.W_pad: rank * w.ex.W_pad + w.ex.W]
            w.set_push_destinations([slot(shared[m]) for m in range(world)],
                                    collective_barrier(None, "cpu"))
        ref_x = x0.copy()
        ref_v = [np.zeros(d, dtype=np.float32) for _ in range(world)] if beta is not None else None
        for step in range(3):
            grads = [rng.standard_normal(d).astype(np.float32) for _ in range(world)]
            want = oracle.fused_step(grads, ref_v, ref_x, beta if beta is not None else 0.0, lr, wd, flip)
            del phases[:]
            vote = w.step(torch.from_numpy(grads[rank].copy()), flip)
            assert phases == EXPECTED_ORDER[mode], phases
            assert np.array_equal(_as_u32(vote), want), "rank %d step %d: vote differs" % (rank, step)
            assert np.array_equal(w.x.numpy().view(np.uint32), ref_x.view(np.uint32)), "rank %d: x differs" % rank
            if beta is not None:
                assert np.array_equal(w.momentum.numpy().view(np.uint32), ref_v[rank].view(np.uint32))
        want_calls = {"allgather": ["ss_signum_update" if beta is not None else "ss_sign_pack", "ss_vote_apply"],
                      "sharded": ["ss_signum_update" if beta is not None else "ss_sign_pack",
                                  "ss_majority_vote", "ss_apply_vote"],
                      "push": ["ss_signum_update_push", "ss_vote_apply"]}[mode]
        if mode == "sharded" and w.ex.slice_coordinates() == 0:
            want_calls = [c for c in want_calls if c != "ss_majority_vote"]
        assert kernels.calls == want_calls * 3, kernels.calls
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("mode,world,d,flip,beta", [
    ("allgather", 2, 100_003, 0b01, 0.9), ("allgather", 3, 70, 0, None),
    ("sharded", 2, 1000, 0, 0.9), ("sharded", 3, 33, 0b010, None), ("sharded", 3, 100_003, 0b100, 0.9),
    ("push", 2, 100_003, 0b10, 0.9), ("push", 3, 1000, 0, 0.9)])
def test_majority_vote_worker_step_over_gloo(mode, world, d, flip, beta):
    shared = None
    if mode == "push":
        W_pad = PackedExchange(d, world, 0, "meta", "push").W_pad
        shared = [torch.zeros(world * W_pad, dtype=torch.int32).share_memory_() for _ in range(world)]
    mp.spawn(_worker_main, args=(world, _free_port(), d, mode, flip, beta, shared), nprocs=world, join=True)


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
