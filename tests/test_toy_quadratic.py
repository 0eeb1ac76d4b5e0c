"""The toy problem of Figure 1: signSGD with majority vote on a 1000-dimensional quadratic with
N(0,1) noise added to every gradient component, 27 workers in the adversarial runs.

f(x) = 1/2 |x|^2, so worker m's stochastic gradient is x + n_m. The figure's plots cannot be
read (and its notebook is not used); what is checked is what Theorem 2 and Definition 1 state:
with fewer than half of the workers adversarial the objective still falls, with more than half
inverting it rises, a worker that multiplies its gradient by -10 is the same as one that
inverts its sign bits, and sign-randomising workers carry no information either way. The CPU
half pins the oracle to those statements; the GPU half runs the same trajectories through the
C ABI and compares every iterate with the oracle, bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle

D, M, LR = 1000, 27, 1e-2


def objective(x) -> float:
    return 0.5 * float((np.asarray(x, dtype=np.float64) ** 2).sum())


def make_run(steps: int, n_adv: int, kind: str, seed: int):
    """Initial point and per-step, per-worker gradient noise of one run (shared by both sides)."""
    rng = np.random.default_rng(seed)
    x0 = rng.standard_normal(D).astype(np.float32)
    noise = rng.standard_normal((steps, M, D)).astype(np.float32)
    signs = rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=(steps, M, D))
    flip = 0
    if kind == "invert":
        for m in range(M - n_adv, M):
            flip |= 1 << m
    return x0, noise, signs, flip


def worker_gradients(x: np.ndarray, noise_t: np.ndarray, signs_t: np.ndarray, n_adv: int, kind: str):
    """g_m = x + n_m; the last n_adv workers apply their blind multiplicative vector (Definition 1)."""
    grads = []
    for m in range(M):
        g = (x + noise_t[m]).astype(np.float32)
        if m >= M - n_adv:
            if kind == "neg10":
                g = (np.float32(-10.0) * g).astype(np.float32)
            elif kind == "rand":
                g = (np.float32(10.0) * g * signs_t[m]).astype(np.float32)
        grads.append(np.ascontiguousarray(g))
    return grads


def oracle_run(steps, n_adv, kind, seed=0, beta=None):
    x0, noise, signs, flip = make_run(steps, n_adv, kind, seed)
    x = x0.copy()
    moms = [np.zeros(D, dtype=np.float32) for _ in range(M)] if beta is not None else None
    for t in range(steps):
        grads = worker_gradients(x, noise[t], signs[t], n_adv, kind)
        oracle.fused_step(grads, moms, x, beta if beta is not None else 0.0, LR, 0.0, flip)
    return x0, x


# ---- CPU: the oracle against what the paper states ------------------------------------------

def test_majority_vote_descends_on_the_noisy_quadratic():
    x0, x = oracle_run(300, 0, "invert")
    assert objective(x) < 0.01 * objective(x0)


@pytest.mark.parametrize("n_adv", [3, 9, 12])
def test_fewer_than_half_inverting_workers_still_descend(n_adv):
    x0, x = oracle_run(300, n_adv, "invert")
    assert objective(x) < 0.2 * objective(x0)


def test_more_adversaries_never_help():
    finals = [objective(oracle_run(300, k, "invert")[1]) for k in (0, 3, 9, 12, 13)]
    assert all(a < b for a, b in zip(finals, finals[1:]))


@pytest.mark.parametrize("n_adv", [14, 18])
def test_more_than_half_inverting_workers_ascend(n_adv):
    x0, x = oracle_run(300, n_adv, "invert")
    assert objective(x) > 2.0 * objective(x0)


@pytest.mark.parametrize("n_adv", [3, 13])
def test_scaling_by_minus_ten_is_the_same_as_inverting_the_sign_bits(n_adv):
    # sign(v * g) = sign(v) * sign(g): identical iterates unless a gradient component is exactly 0
    _, xa = oracle_run(120, n_adv, "invert", seed=5)
    _, xb = oracle_run(120, n_adv, "neg10", seed=5)
    assert np.array_equal(xa.view(np.uint32), xb.view(np.uint32))


def test_sign_randomising_workers_are_harmless_even_in_the_majority():
    for n_adv in (13, 18):
        x0, x = oracle_run(300, n_adv, "rand")
        assert objective(x) < 0.05 * objective(x0)


def test_signum_momentum_descends_too():
    x0, x = oracle_run(300, 9, "invert", beta=0.9)
    assert objective(x) < 0.2 * objective(x0)


# ---- GPU: the same trajectories through the C ABI ------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("n_adv,kind,beta", [(0, "invert", None), (13, "invert", None),
                                             (9, "neg10", None), (13, "rand", None),
                                             (9, "invert", 0.9), (14, "invert", 0.9)])
def test_gpu_trajectory_matches_the_oracle(n_adv, kind, beta):
    from paper_1810_05291_b200 import binding as B
    dev = "cuda:0"
    steps = 60
    x0, noise, signs, flip = make_run(steps, n_adv, kind, seed=11)
    x_cpu = x0.copy()
    m_cpu = [np.zeros(D, dtype=np.float32) for _ in range(M)] if beta is not None else None
    x_gpu = torch.from_numpy(x0.copy()).to(dev)
    m_gpu = [torch.zeros(D, device=dev) for _ in range(M)] if beta is not None else None
    vote = torch.zeros(B.ss_packed_words(D), dtype=torch.int32, device=dev)
    for t in range(steps):
        # both sides build the gradients from their own (identical) iterate
        g_cpu = worker_gradients(x_cpu, noise[t], signs[t], n_adv, kind)
        g_gpu_src = worker_gradients(x_gpu.cpu().numpy(), noise[t], signs[t], n_adv, kind)
        g_gpu = [torch.from_numpy(g).to(dev) for g in g_gpu_src]
        want = oracle.fused_step(g_cpu, m_cpu, x_cpu, beta if beta is not None else 0.0, LR, 0.0, flip)
        B.ss_fused_step(g_gpu, m_gpu, x_gpu, beta if beta is not None else 0.0, LR, 0.0, flip, vote)
        got = vote.cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want), "vote words differ at step %d" % t
        assert np.array_equal(x_gpu.cpu().numpy().view(np.uint32), x_cpu.view(np.uint32)), \
            "iterate differs at step %d" % t
    if beta is not None:
        for a, b in zip(m_gpu, m_cpu):
            assert np.array_equal(a.cpu().numpy().view(np.uint32), b.view(np.uint32))
    f0, fT = objective(x0), objective(x_cpu)
    if kind == "invert" and n_adv > M // 2:
        assert fT > f0
    else:
        assert fT < f0
