"""Algorithm 1 as a torch optimiser over a model's own tensors (``SignumVote``).

Host logic on CPU, with the oracle standing in for the kernels: flattening and views, the
per-tensor table (parameter groups, a schedule that moves), momentum state through a state_dict
round trip, gradients that are missing or were replaced, and M processes over gloo whose replicas
must stay bit-identical and equal the oracle's M-worker step. On a GPU the same model runs through
the CUDA kernels and is compared with the oracle bit for bit.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_1810_05291_b200.optim import SignumVote
from tests.test_distributed_gloo import OracleKernels


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _model(seed, device="cpu", width=7):
    torch.manual_seed(seed)
    return torch.nn.Sequential(torch.nn.Linear(5, width), torch.nn.Tanh(), torch.nn.Linear(width, 3)).to(device)


def _groups(model, lr_w=1e-2, lr_b=5e-3):
    weights = [p for n, p in model.named_parameters() if n.endswith("weight")]
    biases = [p for n, p in model.named_parameters() if n.endswith("bias")]
    return [dict(params=weights, lr=lr_w, weight_decay=0.01), dict(params=biases, lr=lr_b, weight_decay=0.0)]


def _batch(step, rank=0, device="cpu", n=16):
    g = torch.Generator().manual_seed(1000 * rank + step)
    return torch.randn(n, 5, generator=g).to(device), torch.randn(n, 3, generator=g).to(device)


def _loss(model, step, rank=0, device="cpu"):
    a, b = _batch(step, rank, device)
    return ((model(a) - b) ** 2).mean()


def _reference_step(opt, grads_np, ref_x, ref_v, beta, flip=0):
    """The oracle's per-tensor loop on host copies, with the optimiser's own layout and table."""
    lrs, wds = opt._hyperparameters()
    oracle.fused_step_segments(grads_np, ref_v, ref_x, 0.0 if beta is None else beta, opt.layout.begins, lrs, wds, flip)


def _bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("beta", [0.9, None])
def test_one_process_follows_the_oracle_and_a_moving_schedule(beta):
    model = _model(1)
    opt = SignumVote(_groups(model), momentum=beta, kernels=OracleKernels())
    sched = torch.optim.lr_scheduler.StepLR(opt, step_size=2, gamma=0.1)
    ref_x = opt.flat_param.numpy().copy()
    ref_v = [np.zeros_like(ref_x)] if beta is not None else None
    in_layout_order = [p for group in opt.param_groups for p in group["params"]]
    for p, view in zip(in_layout_order, opt.layout.views(opt.flat_param)):
        assert p.data_ptr() == view.data_ptr() and p.grad.data_ptr() != p.data_ptr()
    for step in range(5):
        opt.zero_grad()
        _loss(model, step).backward()
        g = opt.flat_grad.numpy().copy()
        assert np.abs(g).sum() > 0                      # backward accumulated straight into the flat buffer
        _reference_step(opt, [g], ref_x, ref_v, beta)
        opt.step()
        sched.step()
        assert np.array_equal(_bits(opt.flat_param), ref_x.view(np.uint32)), "step %d" % step
        if beta is not None:
            assert np.array_equal(_bits(opt.flat_momentum), ref_v[0].view(np.uint32))
    # two decays by ten reached the device table (it held 1e-2 at the start)
    assert opt.param_groups[0]["lr"] == pytest.approx(1e-4) and opt.layout.lrs[0] == pytest.approx(1e-4)
    # the model computes with the updated values: its tensors are the flat vector
    flat_again = torch.cat([p.detach().reshape(-1) for p in in_layout_order])
    packed = torch.cat([v.reshape(-1) for v in opt.layout.views(opt.flat_param)])
    assert torch.equal(flat_again, packed)


def test_missing_and_replaced_gradients_are_brought_back_into_the_flat_buffer():
    model = _model(2)
    opt = SignumVote(model.parameters(), lr=1e-2, momentum=None, kernels=OracleKernels())
    params = list(model.parameters())
    opt.zero_grad(set_to_none=True)                        # still zeroes in place
    assert all(p.grad is not None and float(p.grad.abs().sum()) == 0.0 for p in params)
    params[0].grad = None                                  # votes with a zero gradient: +1
    params[1].grad = torch.full_like(params[1], -2.0)      # a tensor of the caller's
    x0 = opt.flat_param.clone()
    opt.step()
    views = opt.layout.views(opt.flat_param)
    before = opt.layout.views(x0)
    assert torch.equal(views[0], before[0] - 1e-2)         # sign(0) = +1 under the one-bit reading
    assert torch.equal(views[1], before[1] + 1e-2)
    assert params[1].grad.data_ptr() == opt.layout.views(opt.flat_grad)[1].data_ptr()


def test_state_dict_round_trip_continues_bit_for_bit():
    def run(steps_before, steps_after, reload):
        model = _model(3)
        opt = SignumVote(_groups(model), momentum=0.8, kernels=OracleKernels())
        for step in range(steps_before):
            opt.zero_grad()
            _loss(model, step).backward()
            opt.step()
        if reload:
            saved_model, saved_opt = model.state_dict(), opt.state_dict()
            saved_model = {k: v.clone() for k, v in saved_model.items()}
            model = _model(99)
            model.load_state_dict(saved_model)
            opt = SignumVote(_groups(model), momentum=0.8, kernels=OracleKernels())
            opt.load_state_dict(saved_opt)
            in_layout_order = [p for group in opt.param_groups for p in group["params"]]
            for p, mv in zip(in_layout_order, opt.layout.views(opt.flat_momentum)):
                assert opt.state[p]["momentum_buffer"].data_ptr() == mv.data_ptr()
        for step in range(steps_before, steps_before + steps_after):
            opt.zero_grad()
            _loss(model, step).backward()
            opt.step()
        # per tensor: the padding coordinates between tensors belong to no tensor and are not saved
        return ([v.clone() for v in opt.layout.views(opt.flat_param)],
                [v.clone() for v in opt.layout.views(opt.flat_momentum)])

    xa, va = run(3, 3, reload=False)
    xb, vb = run(3, 3, reload=True)
    assert all(torch.equal(a, b) for a, b in zip(xa, xb)) and all(torch.equal(a, b) for a, b in zip(va, vb))


def test_the_optimiser_trains_a_small_model():
    """Signum's fixed-size steps bring a student network's loss on a fixed teacher's outputs down
    (Theorem 1's setting with M = 1: x <- x - eta sign(v))."""
    teacher = _model(21)
    student = _model(22)
    opt = SignumVote(student.parameters(), lr=2e-3, momentum=0.9, kernels=OracleKernels())
    g = torch.Generator().manual_seed(5)
    a = torch.randn(256, 5, generator=g)
    with torch.no_grad():
        b = teacher(a)
    losses = []
    for _ in range(300):
        opt.zero_grad()
        loss = ((student(a) - b) ** 2).mean()
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
    assert losses[-1] < 0.2 * losses[0]


def test_bad_arguments_are_refused():
    model = _model(4)
    with pytest.raises(ValueError):
        SignumVote(model.parameters(), lr=-1.0, kernels=OracleKernels())
    with pytest.raises(ValueError):
        SignumVote(model.parameters(), momentum=1.0, kernels=OracleKernels())
    with pytest.raises(ValueError):
        SignumVote([torch.nn.Parameter(torch.zeros(3, dtype=torch.float64))], kernels=OracleKernels())


def _rank_main(rank, world, port, mode, beta, flip):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        model = _model(7)                                   # every replica starts from the same parameters
        opt = SignumVote(_groups(model), momentum=beta, mode=mode, kernels=OracleKernels())
        ref_x = opt.flat_param.numpy().copy()
        ref_v = [np.zeros_like(ref_x) for _ in range(world)] if beta is not None else None
        for step in range(4):
            opt.zero_grad()
            _loss(model, step, rank).backward()             # every worker sees its own mini-batch
            g = opt.flat_grad.clone()
            everyone = [torch.zeros_like(g) for _ in range(world)]
            dist.all_gather(everyone, g)                    # test only: the reference needs all M gradients
            _reference_step(opt, [e.numpy() for e in everyone], ref_x, ref_v, beta, flip)
            opt.step(flip_mask=flip)
            assert np.array_equal(_bits(opt.flat_param), ref_x.view(np.uint32)), "rank %d step %d" % (rank, step)
            if beta is not None:
                assert np.array_equal(_bits(opt.flat_momentum), ref_v[rank].view(np.uint32))
        digest = opt.flat_param.clone()
        others = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(others, digest)
        assert all(torch.equal(o, digest) for o in others)  # the replicas never drifted apart
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("mode,world,beta,flip", [("allgather", 3, 0.9, 0), ("sharded", 2, 0.9, 0b10),
                                                   ("allgather", 2, None, 0), ("sharded", 3, None, 0b001)])
def test_workers_over_gloo_train_identical_replicas(mode, world, beta, flip):
    mp.spawn(_rank_main, args=(world, _free_port(), mode, beta, flip), nprocs=world, join=True)


@pytest.mark.gpu
@pytest.mark.parametrize("beta", [0.9, None])
def test_gpu_one_process_matches_the_oracle(beta):
    dev = torch.device("cuda", 0)
    model = _model(11, dev, width=193)                      # 5*193 + 193 + 193*3 + 3 coordinates: ragged tail
    opt = SignumVote(_groups(model), momentum=beta)
    ref_x = opt.flat_param.cpu().numpy().copy()
    ref_v = [np.zeros_like(ref_x)] if beta is not None else None
    for step in range(4):
        opt.zero_grad()
        _loss(model, step, 0, dev).backward()
        g = opt.flat_grad.cpu().numpy().copy()
        if step == 2:
            opt.param_groups[1]["lr"] = 2.5e-3              # a schedule moves one group
        _reference_step(opt, [g], ref_x, ref_v, beta)
        opt.step()
        assert np.array_equal(_bits(opt.flat_param), ref_x.view(np.uint32)), "step %d" % step
        if beta is not None:
            assert np.array_equal(_bits(opt.flat_momentum), ref_v[0].view(np.uint32))
        words = opt.vote.cpu().numpy().view(np.uint32)
        assert words.shape[0] == oracle.packed_words(opt.layout.d)


@pytest.mark.gpu
@pytest.mark.parametrize("mode", ["allgather", "sharded", "push", "push:signal", "push:flags"])
def test_gpu_worker_path_with_a_table_in_a_group_of_one(mode):
    """The worker-and-exchange path of the optimiser on real kernels and real NCCL collectives with
    nobody to talk to: momentum and packing, the exchange, vote and per-tensor update."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(_free_port())
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    try:
        model = _model(13, dev, width=61)
        layout, _, barrier = mode.partition(":")
        opt = SignumVote(_groups(model), momentum=0.9, mode=layout, exchange=True, push_barrier=barrier or "collective")
        assert opt.worker is not None
        ref_x = opt.flat_param.cpu().numpy().copy()
        ref_v = [np.zeros_like(ref_x)]
        for step in range(3):
            opt.zero_grad()
            _loss(model, step, 0, dev).backward()
            g = opt.flat_grad.cpu().numpy().copy()
            _reference_step(opt, [g], ref_x, ref_v, 0.9)
            opt.step()
            torch.cuda.synchronize()
            opt.worker.check()
            assert np.array_equal(_bits(opt.flat_param), ref_x.view(np.uint32)), "step %d" % step
            assert np.array_equal(_bits(opt.flat_momentum), ref_v[0].view(np.uint32))
    finally:
        dist.destroy_process_group()
