"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input generation only -- none of the method's arithmetic (no sign,
no packing, no vote, no momentum, no update). It serves both the CUDA path and the CPU
checks: a case is generated once, on one device, and the checker receives a copy of
the very same bytes, so no second random number generator has to agree with the first.

Value model: each worker's mini-batch gradient is a shared "true gradient" signal plus
independent per-worker noise, g_m = s + sigma * n_m (Lemma 1's setting: an unbiased
estimate with unimodal symmetric noise; Section 3.1 observes near-Gaussian noise). The
sizes are the parameter counts of ResNet-50 (25,557,032) and AlexNet (61,100,840) and
the worker counts of Section 4 (7 to 15 machines). They stand in for ImageNet
gradients, which are not available here.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

RESNET50_PARAMS = 25_557_032
ALEXNET_PARAMS = 61_100_840
BASE_SEED = 181005291


def seed_for(cfg: int, step: int = 0) -> int:
    return BASE_SEED + 1000 * int(cfg) + int(step)


@dataclass
class Case:
    """One workload: M gradient buffers plus the optimiser settings of Algorithm 1."""
    name: str
    M: int
    d: int
    dtype: torch.dtype
    beta: Optional[float]          # None: signSGD (no momentum buffers)
    lr: float
    weight_decay: float = 0.0
    flip_mask: int = 0             # bit m set: worker m inverts its sign bits
    sigma: float = 1.0
    noise: str = "gauss"           # "gauss" | "student3"
    has_signal: bool = True        # False: g_m is pure noise (i.i.d. across workers)
    zero_frac: float = 0.0         # per-element probability of an exact zero
    zero_prefix: int = 0           # coordinates [0, zero_prefix) are zero in all workers
    dup_last_from: Optional[int] = None  # worker M-1 is a copy of this worker (tie probe)
    cfg: int = 0
    extra: dict = field(default_factory=dict)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def signal(case: Case, device, step: int = 0) -> Optional[torch.Tensor]:
    """The shared signal s ~ N(0,1) of a step (None for pure-noise cases)."""
    if not case.has_signal:
        return None
    gen = _gen(device, seed_for(case.cfg, step) * 7919 + 1)
    return torch.randn(case.d, generator=gen, device=device, dtype=torch.float32)


def worker_gradient(case: Case, m: int, device, step: int = 0,
                    s: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Gradient buffer of worker m at a step, in the case's dtype."""
    src = m
    if case.dup_last_from is not None and m == case.M - 1:
        src = case.dup_last_from
    gen = _gen(device, (seed_for(case.cfg, step) * 7919 + 2) * 131 + src)
    d = case.d
    if case.noise == "gauss":
        g = torch.randn(d, generator=gen, device=device, dtype=torch.float32)
    elif case.noise == "student3":
        z = torch.randn(d, generator=gen, device=device, dtype=torch.float32)
        chi = torch.zeros(d, device=device, dtype=torch.float32)
        for _ in range(3):
            w = torch.randn(d, generator=gen, device=device, dtype=torch.float32)
            chi.addcmul_(w, w)
            del w
        g = z / torch.sqrt(chi / 3.0)
        del z, chi
    else:
        raise ValueError(case.noise)
    if case.sigma != 1.0:
        g.mul_(case.sigma)
    if s is None and case.has_signal:
        s = signal(case, device, step)
    if s is not None:
        g.add_(s)
    if case.zero_frac > 0.0:
        u = torch.rand(d, generator=gen, device=device, dtype=torch.float32)
        g.masked_fill_(u < case.zero_frac, 0.0)
        del u
    if case.zero_prefix > 0:
        g[: min(case.zero_prefix, d)] = 0.0
    return g.to(case.dtype).contiguous()


def gradients(case: Case, device, step: int = 0) -> List[torch.Tensor]:
    s = signal(case, device, step)
    return [worker_gradient(case, m, device, step, s) for m in range(case.M)]


def initial_params(case: Case, device) -> torch.Tensor:
    gen = _gen(device, seed_for(case.cfg, 0) * 7919 + 3)
    return torch.randn(case.d, generator=gen, device=device, dtype=torch.float32)


def zero_momenta(case: Case, device) -> Optional[List[torch.Tensor]]:
    if case.beta is None:
        return None
    return [torch.zeros(case.d, device=device, dtype=torch.float32) for _ in range(case.M)]


# ---- the five named workloads (d can be overridden to get a scaled-down copy) ------------

def cfg1(d: int = 1 << 20) -> Case:
    return Case("cfg1: M=3 d=2^20 fp32 N(0,1), vote+apply, no momentum", M=3, d=d,
                dtype=torch.float32, beta=None, lr=1e-3, has_signal=False, cfg=1)


def cfg2(d: int = ALEXNET_PARAMS) -> Case:
    return Case("cfg2: M=7 AlexNet-sized fp32, signal+N(0,2^2) noise, 3 inverting workers",
                M=7, d=d, dtype=torch.float32, beta=None, lr=1e-4, sigma=2.0,
                flip_mask=0x70, cfg=2)


def cfg3(d: int = RESNET50_PARAMS) -> Case:
    return Case("cfg3: M=15 ResNet-50-sized fp32, signal+N(0,1) noise, Signum beta=0.9",
                M=15, d=d, dtype=torch.float32, beta=0.9, lr=1e-4, sigma=1.0, cfg=3)


def cfg4(d: int = RESNET50_PARAMS, tie_probe: bool = False) -> Case:
    M = 16 if tie_probe else 15
    return Case("cfg4: M=%d ResNet-50-sized bf16, Student-t(3) noise, 10%% zeros, Signum" % M,
                M=M, d=d, dtype=torch.bfloat16, beta=0.9, lr=1e-4, noise="student3",
                zero_frac=0.10, zero_prefix=4096, dup_last_from=0 if tie_probe else None,
                cfg=4)


def cfg5(d: int, M: int, momentum: bool = False) -> Case:
    return Case("cfg5: sweep d=%d M=%d fp32 N(0,1)" % (d, M), M=M, d=d, dtype=torch.float32,
                beta=0.9 if momentum else None, lr=1e-3, has_signal=False, cfg=5)


SWEEP_D = (1 << 16, 1 << 20, 1 << 24, 1 << 28)
SWEEP_M = (1, 3, 7, 15, 31, 63)


# ---- adversary variants of Definition 1, as input transformations -----------------------

def rescale_adversary(g: torch.Tensor, seed: int) -> torch.Tensor:
    """Definition 1(i): multiply by an arbitrary positive vector chosen blind."""
    gen = _gen(g.device, seed)
    scale = torch.exp(4.0 * torch.randn(g.shape[0], generator=gen, device=g.device))
    return (g.float() * scale).to(g.dtype)


def random_sign_adversary(g: torch.Tensor, seed: int, scale: float = 10.0) -> torch.Tensor:
    """Definition 1(ii) as in the Multi-Krum comparison: times 10, then random signs."""
    gen = _gen(g.device, seed)
    flip = torch.randint(0, 2, (g.shape[0],), generator=gen, device=g.device) * 2 - 1
    return (g.float() * scale * flip).to(g.dtype)
