"""The one-worker-per-process form of Algorithm 1 on CPU (gloo, world sizes 2 and 3).

The kernels need a GPU, so here the CPU oracle stands in for them and what is under test is the
host side of ``paper_1810_05291_b200.distributed``: buffer sizes, slice arithmetic, padding and
the collectives. Every rank rebuilds all M gradients from the seed, plays its own worker through
``PackedExchange``, and must end with the parameters and the packed vote that the oracle's
M-worker step gives, in both exchange layouts.
"""
import os
import socket
import time

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


    # ---- a fused vector of several tensors: the "device table" is a dict on the host here
    @staticmethod
    def ss_packed_words(d):
        return (int(d) + 31) // 32

    @staticmethod
    def segment_table(n, device):
        return {}

    def ss_segments_upload(self, begins, lrs, weight_decays, d, segments_dev, stream=None):
        self.calls.append("ss_segments_upload")
        segments_dev.update(begins=list(begins), lrs=list(lrs), wds=list(weight_decays))

    def ss_fused_step_segments(self, grads, momenta, param, beta, segments_dev, n_segments, flip_mask=0,
                               vote_words_out=None, stream=None):
        self.calls.append("ss_fused_step_segments")
        t = segments_dev
        vote = oracle.fused_step_segments([self._f32(g) for g in grads],
                                          None if momenta is None else [self._f32(v) for v in momenta],
                                          self._f32(param), beta, t["begins"], t["lrs"], t["wds"], flip_mask)
        if vote_words_out is not None:
            self._u32(vote_words_out)[:] = vote

    def _apply_segments(self, param, vote, segments_dev):
        # one "worker" whose gradient carries the vote's signs: its lone vote is the vote
        d = param.numel()
        g = np.where(oracle.unpack(vote, d) > 0, 1.0, -1.0).astype(np.float32)
        t = segments_dev
        oracle.fused_step_segments([g], None, self._f32(param), 0.0, t["begins"], t["lrs"], t["wds"], 0)

    def ss_vote_apply_segments(self, packed, param, segments_dev, n_segments, flip_mask=0, vote_words_out=None,
                               stream=None):
        self.calls.append("ss_vote_apply_segments")
        vote = oracle.majority_vote([self._u32(p).copy() for p in packed], param.numel(), flip_mask)
        self._apply_segments(param, vote, segments_dev)
        if vote_words_out is not None:
            self._u32(vote_words_out)[:] = vote

    def ss_apply_vote_segments(self, param, vote_words, segments_dev, n_segments, stream=None):
        self.calls.append("ss_apply_vote_segments")
        self._apply_segments(param, self._u32(vote_words).copy(), segments_dev)

    # ---- flag-ordered exchange: the flags are words of shared memory that other processes write
    SS_MAX_WORKERS = 64

    def ss_flags_signal(self, flags, index, epoch, stream=None):
        self.calls.append("ss_flags_signal")
        for f in flags:
            f[index] = epoch

    def ss_flags_wait(self, flags_local, M, epoch, timeout_ns, status_dev, stream=None):
        self.calls.append("ss_flags_wait")
        deadline = time.monotonic() + timeout_ns * 1e-9
        while True:
            seen = flags_local[:M].clone()
            late = (seen < epoch).nonzero()
            if late.numel() == 0:
                status_dev[0] = 0
                return
            if time.monotonic() > deadline:
                status_dev[0] = int(late[0]) + 1
                return
            time.sleep(0.001)

    def ss_flags_signal_wait(self, flags, index, flags_local, M, epoch, timeout_ns, status_dev, stream=None):
        self.ss_flags_signal(flags, index, epoch)
        self.ss_flags_wait(flags_local, M, epoch, timeout_ns, status_dev)

    def ss_vote_apply_guarded(self, packed, param, lr, weight_decay, flip_mask, vote_words_out,
                              skip_if_nonzero_dev, stream=None):
        self.calls.append("ss_vote_apply_guarded")
        if int(skip_if_nonzero_dev[0]) != 0:
            return
        self.calls.pop()
        self.ss_vote_apply(packed, param, lr, weight_decay, flip_mask, vote_words_out, stream)
        self.calls[-1] = "ss_vote_apply_guarded"

    def ss_vote_apply_guarded_segments(self, packed, param, segments_dev, n_segments, flip_mask, vote_words_out,
                                       skip_if_nonzero_dev, stream=None):
        self.calls.append("ss_vote_apply_guarded_segments")
        if int(skip_if_nonzero_dev[0]) != 0:
            return
        self.calls.pop()
        self.ss_vote_apply_segments(packed, param, segments_dev, n_segments, flip_mask, vote_words_out, stream)
        self.calls[-1] = "ss_vote_apply_guarded_segments"


EXPECTED_ORDER = {
    "allgather": ["start", "kernel:pack", "exchange:all_gather", "kernel:vote_apply"],
    "sharded": ["start", "kernel:pack", "exchange:all_to_all", "kernel:vote", "exchange:all_gather",
                "kernel:apply"],
    "push": ["start", "kernel:pack", "exchange:barrier", "kernel:vote_apply", "exchange:barrier"],
    "push-flags": ["start", "kernel:pack", "exchange:signal", "exchange:wait", "kernel:vote_apply"],
    "push-flags-fused": ["start", "kernel:pack", "exchange:wait", "kernel:vote_apply"],
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
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()), beta, lr, wd, mode.split("-")[0], world=world,
                               rank=rank, kernels=kernels, on_phase=phases.append)
        if mode.startswith("push-flags"):
            # two receive buffers and one flag array per rank, all in shared memory; no barrier, no
            # collective: the ranks are ordered by the flags alone
            n = world * w.ex.W_pad
            slot = lambda buf: buf[rank * w.ex.W_pad: rank * w.ex.W_pad + w.ex.W]
            w.set_flag_exchange([shared[rank][0], shared[rank][1]],
                                [[slot(shared[m][parity]) for m in range(world)] for parity in (0, 1)],
                                [shared[m][2] for m in range(world)], shared[rank][2], timeout_ns=20_000_000_000,
                                signal_with_wait=mode.endswith("fused"))
        elif mode == "push":
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
            if mode.startswith("push-flags") and rank == 1:
                time.sleep(0.05 * step)              # a straggler: the others must wait for its flag
            vote = w.step(torch.from_numpy(grads[rank].copy()), flip)
            w.check()
            assert phases == EXPECTED_ORDER[mode], phases
            assert np.array_equal(_as_u32(vote), want), "rank %d step %d: vote differs" % (rank, step)
            assert np.array_equal(w.x.numpy().view(np.uint32), ref_x.view(np.uint32)), "rank %d: x differs" % rank
            if beta is not None:
                assert np.array_equal(w.momentum.numpy().view(np.uint32), ref_v[rank].view(np.uint32))
        want_calls = {"allgather": ["ss_signum_update" if beta is not None else "ss_sign_pack", "ss_vote_apply"],
                      "sharded": ["ss_signum_update" if beta is not None else "ss_sign_pack",
                                  "ss_majority_vote", "ss_apply_vote"],
                      "push": ["ss_signum_update_push", "ss_vote_apply"],
                      "push-flags": ["ss_signum_update_push", "ss_flags_signal", "ss_flags_wait",
                                     "ss_vote_apply_guarded"]}[mode.replace("-fused", "")]
        if mode == "sharded" and w.ex.slice_coordinates() == 0:
            want_calls = [c for c in want_calls if c != "ss_majority_vote"]
        assert kernels.calls == want_calls * 3, kernels.calls
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("mode,world,d,flip,beta", [
    ("allgather", 2, 100_003, 0b01, 0.9), ("allgather", 3, 70, 0, None),
    ("sharded", 2, 1000, 0, 0.9), ("sharded", 3, 33, 0b010, None), ("sharded", 3, 100_003, 0b100, 0.9),
    ("push", 2, 100_003, 0b10, 0.9), ("push", 3, 1000, 0, 0.9),
    ("push-flags", 2, 100_003, 0b10, 0.9), ("push-flags", 3, 1000, 0, 0.9),
    ("push-flags-fused", 3, 100_003, 0b001, 0.9)])
def test_majority_vote_worker_step_over_gloo(mode, world, d, flip, beta):
    shared = None
    W_pad = PackedExchange(d, world, 0, "meta", "push").W_pad
    if mode == "push":
        shared = [torch.zeros(world * W_pad, dtype=torch.int32).share_memory_() for _ in range(world)]
    if mode.startswith("push-flags"):
        shared = [[torch.zeros(world * W_pad, dtype=torch.int32).share_memory_(),
                   torch.zeros(world * W_pad, dtype=torch.int32).share_memory_(),
                   torch.zeros(64, dtype=torch.int32).share_memory_()] for _ in range(world)]
    mp.spawn(_worker_main, args=(world, _free_port(), d, mode, flip, beta, shared), nprocs=world, join=True)


def _leaver_main(rank, world, port, d, shared, out_dir):
    """Failure made on the host: rank 1 takes part in step 1 and then leaves (between steps, with
    nothing of its own in flight). Rank 0's wait of step 2 must run out of time, name worker 1, and
    leave the parameters of step 1 untouched."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rng = np.random.default_rng(99)
        x0 = rng.standard_normal(d).astype(np.float32)
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()), 0.9, 1e-3, 0.0, "push", world=world, rank=rank,
                               kernels=OracleKernels())
        slot = lambda buf: buf[rank * w.ex.W_pad: rank * w.ex.W_pad + w.ex.W]
        w.set_flag_exchange([shared[rank][0], shared[rank][1]],
                            [[slot(shared[m][parity]) for m in range(world)] for parity in (0, 1)],
                            [shared[m][2] for m in range(world)], shared[rank][2], timeout_ns=300_000_000)
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(world)]
        w.step(torch.from_numpy(grads[rank].copy()))
        w.check()
        if rank == 1:
            return                                    # leaves; never pushes again
        x_after_step_1 = w.x.clone()
        t0 = time.monotonic()
        w.step(torch.from_numpy(grads[rank].copy()))
        waited = time.monotonic() - t0
        try:
            w.check()
            outcome = "no error"
        except RuntimeError as e:
            outcome = str(e)
        with open(os.path.join(out_dir, "outcome.txt"), "w") as f:
            f.write("%s\n%.3f\n%d\n" % (outcome, waited, int(torch.equal(w.x, x_after_step_1))))
    finally:
        dist.destroy_process_group()


def test_a_worker_that_leaves_is_detected_by_the_bounded_wait(tmp_path):
    d, world = 1000, 2
    W_pad = PackedExchange(d, world, 0, "meta", "push").W_pad
    shared = [[torch.zeros(world * W_pad, dtype=torch.int32).share_memory_(),
               torch.zeros(world * W_pad, dtype=torch.int32).share_memory_(),
               torch.zeros(64, dtype=torch.int32).share_memory_()] for _ in range(world)]
    mp.spawn(_leaver_main, args=(world, _free_port(), d, shared, str(tmp_path)), nprocs=world, join=True)
    outcome, waited, unchanged = open(tmp_path / "outcome.txt").read().strip().split("\n")
    assert "worker 1 did not arrive" in outcome and "step 2" in outcome
    assert 0.25 < float(waited) < 5.0                # waited about the time limit, then gave up
    assert unchanged == "1"                          # the update of the failed step was skipped as a whole


def _local_flag_workers(world, d, timeout_ns):
    """`world` workers in this process, wired to one another's buffers and flags, on the stand-in kernels."""
    workers = [MajorityVoteWorker(torch.zeros(d), 0.9, 1e-3, 0.0, "push", world=world, rank=m,
                                  kernels=OracleKernels()) for m in range(world)]
    W_pad = workers[0].ex.W_pad
    bufs = [[torch.zeros(world * W_pad, dtype=torch.int32) for _ in (0, 1)] for _ in range(world)]
    flags = [torch.zeros(64, dtype=torch.int32) for _ in range(world)]
    for m, w in enumerate(workers):
        slot = lambda buf: buf[m * W_pad: m * W_pad + w.ex.W]
        w.set_flag_exchange(bufs[m], [[slot(bufs[p][parity]) for p in range(world)] for parity in (0, 1)],
                            flags, flags[m], timeout_ns)
    return workers


def test_a_timed_out_step_is_reported_by_a_later_check():
    """Host logic of the status ring: worker 1 is late for step 1; worker 0 carries on, step 2 goes
    through, and only then is its status looked at. The check names step 1; worker 1 has no complaint."""
    d = 500
    w0, w1 = _local_flag_workers(2, d, timeout_ns=5_000_000)
    g = torch.from_numpy(np.random.default_rng(3).standard_normal(d).astype(np.float32))
    w0.pack_local(g)
    x_before = w0.x.clone()
    w0.finish(0)                                           # times out: worker 1 has not pushed
    assert torch.equal(w0.x, x_before)
    w1.pack_local(g)
    w1.finish(0)
    for w in (w0, w1):
        w.pack_local(g)
    for w in (w0, w1):
        w.finish(0)
    assert int(w0.step_status()) == 0 and not torch.equal(w0.x, x_before)
    with pytest.raises(RuntimeError, match="step 1: the packed signs of worker 1 did not arrive"):
        w0.check()
    w1.check()
    assert w1.checked_epoch == 2 and w0.checked_epoch == 0


def test_finish_checks_by_itself_before_reusing_a_status_word():
    w = _local_flag_workers(1, 40, timeout_ns=1_000_000)[0]
    g = torch.ones(40)
    for _ in range(w.STATUS_RING + 2):
        w.step(g)
    assert w.checked_epoch >= 1 and w.epoch == w.STATUS_RING + 2
    # a failure that is about to fall out of the ring is raised by finish() itself
    w.flags["status"][(w.checked_epoch + 1) % w.STATUS_RING] = 1
    with pytest.raises(RuntimeError, match="worker 0 did not arrive"):
        for _ in range(w.STATUS_RING):
            w.step(g)


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
