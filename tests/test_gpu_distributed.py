"""MajorityVoteWorker on GPUs.

On one GPU the M workers of Algorithm 1 are M worker objects in one process whose collectives are
served by an in-process stand-in that copies between their buffers (all on one stream, one after
another: no kernel waits on another). The kernels, the buffers and the slice arithmetic are the
ones a multi-GPU run uses; the NCCL transport itself is exercised with a one-rank process group.
Where the machine has two or three GPUs, the last test runs one worker per GPU as separate
processes over NCCL in all three exchange layouts; with fewer GPUs it is reported as skipped (a
skip proves nothing about that path). Every worker must end each step with the parameters, momentum
and packed vote of the oracle's M-worker step.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import oracle
from paper_1810_05291_b200.distributed import MajorityVoteWorker

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class InProcessFabric:
    """Stand-in for torch.distributed inside one process: rank r's call is served at once from
    the other ranks' buffers, which the test has filled in an earlier phase."""

    def __init__(self):
        self.workers = []

    def endpoint(self, rank):
        fabric = self

        class Endpoint:
            def all_gather_into_tensor(self, out, inp, group=None):
                n = inp.numel()
                for m, w in enumerate(fabric.workers):
                    src = w.ex.local if inp is fabric.workers[rank].ex.local else w.ex.vote_slice
                    out[m * n:(m + 1) * n].copy_(src)

            def all_to_all_single(self, out, inp, group=None):
                n = out.numel() // len(fabric.workers)
                for m, w in enumerate(fabric.workers):
                    out[m * n:(m + 1) * n].copy_(w.ex.local[rank * n:(rank + 1) * n])

        return Endpoint()


@pytest.mark.parametrize("mode", ["allgather", "sharded"])
@pytest.mark.parametrize("M,d,beta,flip", [(3, 1000, None, 0), (7, 100_003, 0.9, 0b1000000),
                                           (15, 32 * 3000 + 8, 0.9, 0), (4, 70, 0.9, 0b0011),
                                           (5, 33, None, 0b00001)])
def test_m_workers_in_one_process_match_the_oracle(M, d, beta, flip, mode):
    rng = np.random.default_rng(100 * M + d)
    x0 = rng.standard_normal(d).astype(np.float32)
    fabric = InProcessFabric()
    for m in range(M):
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()).to(DEV), beta, 1e-3, 0.01, mode,
                               world=M, rank=m, collectives=fabric.endpoint(m))
        fabric.workers.append(w)
    ref_x = x0.copy()
    ref_v = [np.zeros(d, dtype=np.float32) for _ in range(M)] if beta is not None else None
    for step in range(3):
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
        want = oracle.fused_step(grads, ref_v, ref_x, beta if beta is not None else 0.0, 1e-3, 0.01, flip)
        for m, w in enumerate(fabric.workers):
            w.pack_local(torch.from_numpy(grads[m]).to(DEV))
        for w in fabric.workers:
            w.serve(flip)
        votes = [w.finish(flip) for w in fabric.workers]
        torch.cuda.synchronize()
        for m, w in enumerate(fabric.workers):
            assert np.array_equal(votes[m].cpu().numpy().view(np.uint32), want), "vote, worker %d" % m
            assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32)), "x, worker %d" % m
            if beta is not None:
                assert np.array_equal(w.momentum.cpu().numpy().view(np.uint32), ref_v[m].view(np.uint32))


@pytest.mark.parametrize("M,d,flip", [(3, 1000, 0), (7, 100_003, 0b0100000), (15, 32 * 3000 + 8, 0)])
def test_push_mode_fills_every_workers_receive_buffer(M, d, flip):
    rng = np.random.default_rng(7 * M + d)
    x0 = rng.standard_normal(d).astype(np.float32)
    workers = [MajorityVoteWorker(torch.from_numpy(x0.copy()).to(DEV), 0.9, 1e-3, 0.0, "push",
                                  world=M, rank=m) for m in range(M)]
    calls = []
    for m, w in enumerate(workers):           # worker m's slot in every worker's receive buffer
        w.set_push_destinations([peer.ex.slot(m) for peer in workers], lambda: calls.append(1))
    ref_x = x0.copy()
    ref_v = [np.zeros(d, dtype=np.float32) for _ in range(M)]
    for step in range(3):
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
        want = oracle.fused_step(grads, ref_v, ref_x, 0.9, 1e-3, 0.0, flip)
        for m, w in enumerate(workers):
            w.pack_local(torch.from_numpy(grads[m]).to(DEV))
        votes = [w.finish(flip) for w in workers]
        torch.cuda.synchronize()
        for m, w in enumerate(workers):
            assert np.array_equal(votes[m].cpu().numpy().view(np.uint32), want)
            assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))
            assert np.array_equal(w.momentum.cpu().numpy().view(np.uint32), ref_v[m].view(np.uint32))
    assert len(calls) == 3 * M * 2


@pytest.mark.parametrize("mode", ["allgather", "sharded"])
def test_one_rank_nccl_group_runs_the_real_collectives(mode):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        d = 32 * 5000 + 8
        rng = np.random.default_rng(9)
        x0 = rng.standard_normal(d).astype(np.float32)
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()).to(DEV), 0.9, 1e-3, 0.0, mode)
        ref_x, ref_v = x0.copy(), [np.zeros(d, dtype=np.float32)]
        for step in range(2):
            g = rng.standard_normal(d).astype(np.float32)
            want = oracle.fused_step([g], ref_v, ref_x, 0.9, 1e-3)
            vote = w.step(torch.from_numpy(g).to(DEV))
            torch.cuda.synchronize()
            assert np.array_equal(vote.cpu().numpy().view(np.uint32), want)
            assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("barrier", ["collective", "signal", "flags"])
def test_push_mode_over_symmetric_memory_with_one_rank(barrier):
    """The symmetric-memory wiring of push mode on a one-rank group: the receive buffer is a
    symmetric allocation, the push goes to the address the rendezvous reports, and the barrier (a
    stream-ordered one-element all-reduce by default, the handle's signal barrier on request)
    orders the steps."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(DEV))
    try:
        d = 32 * 5000 + 8
        rng = np.random.default_rng(19)
        x0 = rng.standard_normal(d).astype(np.float32)
        w = MajorityVoteWorker(torch.from_numpy(x0.copy()).to(DEV), 0.9, 1e-3, 0.0, "push")
        try:
            w.connect_push(barrier=barrier)
        except (RuntimeError, NotImplementedError) as e:
            pytest.skip("symmetric memory is not available here: %s" % str(e)[:200])
        ref_x, ref_v = x0.copy(), [np.zeros(d, dtype=np.float32)]
        for step in range(3):
            g = rng.standard_normal(d).astype(np.float32)
            want = oracle.fused_step([g], ref_v, ref_x, 0.9, 1e-3)
            vote = w.step(torch.from_numpy(g).to(DEV))
            torch.cuda.synchronize()
            w.check()
            assert np.array_equal(vote.cpu().numpy().view(np.uint32), want)
            assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))
    finally:
        dist.destroy_process_group()


def _flag_workers(M, d, x0, timeout_ns):
    """M workers in one process wired for the flag-ordered push: two receive buffers and a flag
    array each, every destination a local tensor."""
    from paper_1810_05291_b200 import binding as B
    workers = [MajorityVoteWorker(torch.from_numpy(x0.copy()).to(DEV), 0.9, 1e-3, 0.0, "push", world=M, rank=m)
               for m in range(M)]
    n = workers[0].ex.world * workers[0].ex.W_pad
    bufs = [[torch.zeros(n, dtype=torch.int32, device=DEV) for _ in (0, 1)] for _ in range(M)]
    flags = [B.flag_array(DEV) for _ in range(M)]
    for m, w in enumerate(workers):
        slot = lambda buf: buf[m * w.ex.W_pad: m * w.ex.W_pad + w.ex.W]
        w.set_flag_exchange(bufs[m], [[slot(bufs[p][parity]) for p in range(M)] for parity in (0, 1)],
                            flags, flags[m], timeout_ns)
    return workers


@pytest.mark.parametrize("M,d,flip", [(3, 1000, 0), (7, 100_003, 0b0100000), (15, 32 * 3000 + 8, 0)])
def test_flag_ordered_push_in_one_process(M, d, flip):
    """Push, signal, bounded wait, guarded vote + update, with no barrier and no collective. On one
    GPU the workers' kernels run one after another on one stream, so every wait finds its flags
    already raised: this checks the flags, epochs, alternating buffers and the guard, not concurrency."""
    rng = np.random.default_rng(11 * M + d)
    x0 = rng.standard_normal(d).astype(np.float32)
    workers = _flag_workers(M, d, x0, timeout_ns=200_000_000)
    ref_x = x0.copy()
    ref_v = [np.zeros(d, dtype=np.float32) for _ in range(M)]
    for step in range(5):                                  # both buffer parities, several epochs
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
        want = oracle.fused_step(grads, ref_v, ref_x, 0.9, 1e-3, 0.0, flip)
        for m, w in enumerate(workers):
            w.pack_local(torch.from_numpy(grads[m]).to(DEV))
        votes = [w.finish(flip) for w in workers]
        for m, w in enumerate(workers):
            w.check()
            assert np.array_equal(votes[m].cpu().numpy().view(np.uint32), want)
            assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))
            assert np.array_equal(w.momentum.cpu().numpy().view(np.uint32), ref_v[m].view(np.uint32))
            assert w.flags["local"][:M].tolist() == [step + 1] * M


def test_wait_runs_out_when_a_worker_never_signals():
    """The failure is made on the host: worker 2 simply does not take part in the step. Worker 0's
    wait must come back after its time limit, name worker 2, leave x and the vote buffer as they
    were, and leave the GPU usable."""
    import time

    from paper_1810_05291_b200 import binding as B
    M, d = 3, 50_000
    rng = np.random.default_rng(5)
    x0 = rng.standard_normal(d).astype(np.float32)
    workers = _flag_workers(M, d, x0, timeout_ns=30_000_000)          # 30 ms
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
    for m in (0, 1):
        workers[m].pack_local(torch.from_numpy(grads[m]).to(DEV))
    w = workers[0]
    w.vote.fill_(-1)
    torch.cuda.synchronize()
    t0 = time.monotonic()
    w.finish(0)
    torch.cuda.synchronize()
    waited = time.monotonic() - t0
    assert 0.025 < waited < 2.0
    assert int(w.step_status().item()) == 3                             # 1 + the missing worker
    with pytest.raises(RuntimeError, match="worker 2 did not arrive"):
        w.check()
    assert np.array_equal(w.x.cpu().numpy().view(np.uint32), x0.view(np.uint32))   # nothing was updated
    assert bool((w.vote == -1).all())
    # the context is intact: an ordinary call still runs and is right
    g = torch.from_numpy(grads[0]).to(DEV)
    words = torch.zeros(B.ss_packed_words(d), dtype=torch.int32, device=DEV)
    B.ss_sign_pack(g, words)
    assert np.array_equal(words.cpu().numpy().view(np.uint32), oracle.sign_pack(grads[0]))
    # the late worker arrives: the same epoch's wait now succeeds and the step goes through
    workers[2].pack_local(torch.from_numpy(grads[2]).to(DEV))
    w.finish(0)
    w.check()
    ref_x, ref_v = x0.copy(), [np.zeros(d, dtype=np.float32) for _ in range(M)]
    want = oracle.fused_step(grads, ref_v, ref_x, 0.9, 1e-3)
    assert np.array_equal(w.vote.cpu().numpy().view(np.uint32), want)
    assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32))


def test_a_step_that_timed_out_stays_on_record_until_it_is_checked():
    """Worker 1 is late for step 1 only (made on the host); worker 0 goes on to step 2, which goes
    through, and looks at its status only afterwards: the check must still name step 1."""
    M, d = 2, 20_000
    rng = np.random.default_rng(6)
    x0 = rng.standard_normal(d).astype(np.float32)
    workers = _flag_workers(M, d, x0, timeout_ns=20_000_000)
    g = [torch.from_numpy(rng.standard_normal(d).astype(np.float32)).to(DEV) for _ in range(M)]
    workers[0].pack_local(g[0])
    workers[0].finish(0)                                   # step 1: worker 1 has not pushed
    workers[1].pack_local(g[1])
    workers[1].finish(0)
    for w in workers:                                      # step 2: everybody takes part
        w.pack_local(g[0])
    for w in workers:
        w.finish(0)
    torch.cuda.synchronize()
    assert int(workers[0].step_status().item()) == 0       # the last step's own word is clean
    with pytest.raises(RuntimeError, match="step 1: the packed signs of worker 1 did not arrive"):
        workers[0].check()
    workers[1].check()                                     # worker 1 missed nothing


def test_the_status_ring_is_checked_before_a_word_is_reused():
    M, d = 1, 64
    w = _flag_workers(M, d, np.zeros(d, dtype=np.float32), timeout_ns=1_000_000)[0]
    g = torch.ones(d, device=DEV)
    for _ in range(w.STATUS_RING + 3):
        w.step(g)
    assert w.epoch == w.STATUS_RING + 3 and w.checked_epoch >= 2    # finish() ran a check by itself
    w.check()
    assert w.checked_epoch == w.epoch


def test_flag_epochs_compare_as_serial_numbers():
    from paper_1810_05291_b200 import binding as B
    flags = B.flag_array(DEV)
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    flags[0], flags[1] = 5, 5
    B.ss_flags_wait(flags, 2, 0xFFFFFFFE, 1_000_000, status)          # 5 is "after" 2^32 - 2
    assert int(status.item()) == 0
    flags[1] = -1                                                      # 2^32 - 1 is "before" 2
    B.ss_flags_wait(flags, 2, 2, 1_000_000, status)
    assert int(status.item()) == 2
    B.ss_flags_signal([flags], 1, 3)
    B.ss_flags_wait(flags, 2, 3, 1_000_000, status)
    assert int(status.item()) == 0 and flags[:3].tolist() == [5, 3, 0]


def test_guarded_vote_apply_skips_everything_or_nothing():
    from paper_1810_05291_b200 import binding as B
    M, d = 7, 64 * 32 * 3 + 45
    gen = torch.Generator(device=DEV).manual_seed(8)
    W = B.ss_packed_words(d)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV, dtype=torch.int64).to(torch.int32)
              for _ in range(M)]
    x0 = torch.randn(d, generator=gen, device=DEV)
    for misalign in (0, 1):                                            # pair kernel and word kernel
        xs = torch.zeros(d + misalign, device=DEV)[misalign:]
        xs.copy_(x0)
        vote = torch.full((W,), -1, dtype=torch.int32, device=DEV)
        guard = torch.full((1,), 4, dtype=torch.int32, device=DEV)
        B.ss_vote_apply_guarded(packed, xs, 1e-3, 0.0, 0b11, vote, guard)
        assert torch.equal(xs, x0) and bool((vote == -1).all())
        guard.zero_()
        B.ss_vote_apply_guarded(packed, xs, 1e-3, 0.0, 0b11, vote, guard)
        xr, vr = x0.clone(), torch.zeros(W, dtype=torch.int32, device=DEV)
        B.ss_vote_apply(packed, xr, 1e-3, 0.0, 0b11, vr)
        assert torch.equal(xs, xr) and torch.equal(vote, vr)


def test_guarded_vote_apply_over_a_table_of_tensors():
    from paper_1810_05291_b200 import binding as B
    from paper_1810_05291_b200.fusion import FlatLayout
    M = 5
    layout = FlatLayout([(37, 11), (5,), (1000,), (3, 3, 7)], [1e-2, 3e-3, 1e-3, 2e-2], [0.0, 0.01, 0.1, 0.0], DEV)
    d = layout.d
    gen = torch.Generator(device=DEV).manual_seed(9)
    W = B.ss_packed_words(d)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV, dtype=torch.int64).to(torch.int32)
              for _ in range(M)]
    x0 = torch.randn(d, generator=gen, device=DEV)
    xs = x0.clone()
    vote = torch.full((W,), -1, dtype=torch.int32, device=DEV)
    guard = torch.full((1,), 2, dtype=torch.int32, device=DEV)
    B.ss_vote_apply_guarded_segments(packed, xs, layout.segments_dev, layout.n_segments, 0b100, vote, guard)
    assert torch.equal(xs, x0) and bool((vote == -1).all())
    guard.zero_()
    B.ss_vote_apply_guarded_segments(packed, xs, layout.segments_dev, layout.n_segments, 0b100, vote, guard)
    xr, vr = x0.clone(), torch.zeros(W, dtype=torch.int32, device=DEV)
    B.ss_vote_apply_segments(packed, xr, layout.segments_dev, layout.n_segments, 0b100, vr)
    assert torch.equal(xs, xr) and torch.equal(vote, vr)
    # against the oracle: the vote, then the per-tensor update (a lone worker whose gradient carries the vote's signs)
    want_vote = oracle.majority_vote([p.cpu().numpy().view(np.uint32) for p in packed], d, 0b100)
    assert np.array_equal(vote.cpu().numpy().view(np.uint32), want_vote)
    ref = x0.cpu().numpy().copy()
    g = np.where(oracle.unpack(want_vote, d) > 0, 1.0, -1.0).astype(np.float32)
    oracle.fused_step_segments([g], None, ref, 0.0, layout.begins, layout.lrs, layout.weight_decays, 0)
    assert np.array_equal(xs.cpu().numpy().view(np.uint32), ref.view(np.uint32))


def _nccl_worker(rank, world, port, mode, d, beta, flip, errors):
    """One process = one worker of Algorithm 1 on GPU `rank`, talking NCCL to the others."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["NCCL_NVLS_ENABLE"] = "0"          # plain peer traffic only
    try:
        torch.cuda.set_device(rank)
        dev = torch.device("cuda", rank)
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
        try:
            rng = np.random.default_rng(5000 + d + world)
            x0 = rng.standard_normal(d).astype(np.float32)
            w = MajorityVoteWorker(torch.from_numpy(x0.copy()).to(dev), beta, 1e-3, 0.01, mode.split("-")[0])
            if mode.startswith("push"):
                w.connect_push(barrier="flags" if mode == "push-flags" else "collective")
            ref_x = x0.copy()
            ref_v = [np.zeros(d, dtype=np.float32) for _ in range(world)] if beta is not None else None
            for step in range(4):
                grads = [rng.standard_normal(d).astype(np.float32) for _ in range(world)]
                want = oracle.fused_step(grads, ref_v, ref_x, beta if beta is not None else 0.0, 1e-3, 0.01, flip)
                vote = w.step(torch.from_numpy(grads[rank]).to(dev), flip)
                torch.cuda.synchronize()
                w.check()
                assert np.array_equal(vote.cpu().numpy().view(np.uint32), want), "vote, step %d" % step
                assert np.array_equal(w.x.cpu().numpy().view(np.uint32), ref_x.view(np.uint32)), "x, step %d" % step
                if beta is not None:
                    assert np.array_equal(w.momentum.cpu().numpy().view(np.uint32), ref_v[rank].view(np.uint32))
        finally:
            dist.destroy_process_group()
    except Exception as e:                          # reported by the parent
        errors.put("rank %d: %r" % (rank, e))
        raise


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("mode,beta", [("allgather", 0.9), ("allgather", None), ("sharded", 0.9), ("push", 0.9),
                                       ("push-flags", 0.9)])
def test_one_worker_per_gpu_over_nccl(world, mode, beta):
    if torch.cuda.device_count() < world:
        pytest.skip("needs %d GPUs, this machine shows %d: the one-worker-per-GPU path over NCCL is "
                    "not exercised here" % (world, torch.cuda.device_count()))
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    errors = ctx.Queue()
    d = 32 * 40_000 + 8
    flip = 0b10
    mp.spawn(_nccl_worker, args=(world, port, mode, d, beta, flip, errors), nprocs=world, join=True)
    assert errors.empty()
