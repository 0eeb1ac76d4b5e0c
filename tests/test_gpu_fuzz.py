"""Seeded random cases of the fused step against the oracle: worker count, length, gradient type,
momentum, inverters, weight decay and pointer alignment drawn together, so that combinations no
hand-written case names still pass through the dispatcher (unrolled or run-time worker loop, quad,
octet or ballot form, with or without a per-tensor table) and come out bit-identical."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B
from tests.test_gpu_parity import _fused_case
from tests.util import count_bit_mismatch, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw(seed):
    rng = np.random.default_rng(seed)
    M = int(rng.choice([1, 2, 3, 4, 6, 7, 9, 15, 16, 17, 27, 31, 33, 63, 64, int(rng.integers(1, 65))]))
    d = int(rng.choice([int(rng.integers(1, 300)), int(rng.integers(300, 70_000)), 32 * int(rng.integers(1, 3000)),
                        32 * int(rng.integers(1, 3000)) + int(rng.integers(1, 32))]))
    dtype = torch.float32 if rng.random() < 0.5 else torch.bfloat16
    momentum = bool(rng.random() < 0.6)
    flip = int(rng.integers(0, 1 << 62)) & ((1 << M) - 1) if rng.random() < 0.5 else 0
    wd = float(rng.choice([0.0, 0.0, 0.03]))
    misalign = int(rng.choice([0, 0, 0, 1, 2, 4]))
    return M, d, dtype, momentum, flip, wd, misalign


@pytest.mark.parametrize("seed", range(48))
def test_random_fused_step(seed):
    M, d, dtype, momentum, flip, wd, misalign = _draw(7000 + seed)
    _fused_case(M, d, dtype, momentum, flip, wd, misalign, steps=2, seed=9000 + 13 * seed)


@pytest.mark.parametrize("seed", range(12))
def test_random_fused_step_with_a_table_of_tensors(seed):
    """The same through ss_fused_step_segments with a random table, against one oracle step per tensor."""
    M, d, dtype, momentum, flip, _, _ = _draw(8000 + seed)
    rng = np.random.default_rng(8100 + seed)
    n_seg = int(rng.integers(1, 40))
    begins = [0] + sorted(int(c) for c in rng.integers(0, d + 1, size=n_seg - 1))
    lrs = [float(10.0 ** rng.uniform(-4, -2)) for _ in range(n_seg)]
    wds = [0.0 if rng.random() < 0.5 else float(10.0 ** rng.uniform(-3, -1)) for _ in range(n_seg)]
    gen = torch.Generator(device=DEV).manual_seed(8200 + seed)
    grads = [torch.randn(d, generator=gen, device=DEV).to(dtype) for _ in range(M)]
    x = torch.randn(d, generator=gen, device=DEV)
    moms = [0.1 * torch.randn(d, generator=gen, device=DEV) for _ in range(M)] if momentum else None
    g_np = [to_np(g) for g in grads]
    x_np = to_np(x)
    m_np = [to_np(v) for v in moms] if momentum else None
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)
    vote = torch.full((B.ss_packed_words(d),), -1, dtype=torch.int32, device=DEV)
    for step in range(2):
        B.ss_fused_step_segments(grads, moms, x, 0.9, tab, n_seg, flip, vote)
        want = oracle.fused_step_segments(g_np, m_np, x_np, 0.9, begins, lrs, wds, flip)
        assert np.array_equal(to_np(vote), want), "vote, step %d" % step
        assert count_bit_mismatch(x, x_np) == 0
        if momentum:
            for v, v_np in zip(moms, m_np):
                assert count_bit_mismatch(v, v_np) == 0
