"""The ternary comparison codec (Appendix B: 1-bit max-norm QSGD) on the GPU against the oracle:
max-norm, code words and decoded values, bit for bit, with the generator's stream reproduced by
the oracle from the seed alone."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B
from tests.util import to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CANARY = 0x5A5A5A5A


def _grad(d, seed, dtype, misalign=0, specials=False):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    g = torch.randn(d + misalign, generator=gen, device=DEV)
    if specials and d >= 8:
        g[misalign + 1] = 0.0
        g[misalign + 2] = -0.0
        g[misalign + 3] = float("nan")
        g[misalign + 5] = -7.5            # the maximum, negative
    return g.to(dtype)[misalign:]


def _codes_buffer(d):
    W = B.ss_ternary_words(d)
    full = torch.full((W + 16,), CANARY, dtype=torch.int32, device=DEV)
    return full, full[8: 8 + W]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("d", [1, 15, 16, 17, 63, 64, 4097, 100_003, 32 * 4096 * 3 + 8])
def test_absmax_pack_unpack_match_the_oracle(d, misalign, dtype):
    g = _grad(d, 7 * d + 1, dtype, misalign, specials=True)
    g_np = to_np(g)
    gmax = torch.full((1,), -1.0, device=DEV)
    B.ss_absmax(g, gmax)
    want_max = oracle.absmax(g_np)
    assert float(gmax.item()) == want_max
    for seed in (0, 0xDEADBEEF12345678):
        full, codes = _codes_buffer(d)
        B.ss_ternary_pack(g, gmax, seed, codes)
        want = oracle.ternary_pack(g_np, gmax=want_max, seed=seed)
        got = to_np(codes)
        assert np.array_equal(got, want), "codes differ in %d words" % int((got != want).sum())
        f = full.cpu()
        assert bool((f[:8] == CANARY).all()) and bool((f[8 + codes.numel():] == CANARY).all())
        out_full = torch.full((d + 8 + misalign,), 123.0, device=DEV)
        out = out_full[4 + misalign: 4 + misalign + d]
        B.ss_ternary_unpack(codes, gmax, out)
        assert np.array_equal(to_np(out).view(np.uint32),
                              oracle.ternary_unpack(want, d, want_max).view(np.uint32))
        o = out_full.cpu()
        assert bool((o[:4 + misalign] == 123.0).all()) and bool((o[4 + misalign + d:] == 123.0).all())


def test_resnet50_sized_gradient_whole_vector():
    d = 25_557_032
    g = _grad(d, 99, torch.float32)
    gmax = torch.zeros(1, device=DEV)
    B.ss_absmax(g, gmax)
    g_np = to_np(g)
    assert float(gmax.item()) == oracle.absmax(g_np)
    codes = torch.zeros(B.ss_ternary_words(d), dtype=torch.int32, device=DEV)
    B.ss_ternary_pack(g, gmax, 2026, codes)
    want = oracle.ternary_pack(g_np, seed=2026)
    assert np.array_equal(to_np(codes), want)
    # the share of kept coordinates is the mean of |g| / max
    kept = float(((codes.view(-1, 1) >> torch.arange(0, 32, 2, device=DEV, dtype=torch.int32)) & 1).float().mean())
    assert abs(kept - float((g.abs() / gmax).mean())) < 5e-4


def test_sign_vector_and_degenerate_inputs():
    d = 5000
    s = torch.where(torch.rand(d, device=DEV, generator=torch.Generator(device=DEV).manual_seed(3)) < 0.5, -0.25, 0.25)
    gmax = torch.zeros(1, device=DEV)
    B.ss_absmax(s, gmax)
    codes = torch.zeros(B.ss_ternary_words(d), dtype=torch.int32, device=DEV)
    B.ss_ternary_pack(s, gmax, 5, codes)
    back = torch.empty(d, device=DEV)
    B.ss_ternary_unpack(codes, gmax, back)
    assert torch.equal(back, s)                                   # Appendix B: sign vectors are left as they are
    z = torch.zeros(d, device=DEV)
    B.ss_absmax(z, gmax)
    assert float(gmax.item()) == 0.0
    codes.fill_(-1)
    B.ss_ternary_pack(z, gmax, 5, codes)
    assert not bool(codes.any())
    empty = torch.zeros(0, device=DEV)
    gmax.fill_(9.0)
    B.ss_absmax(empty, gmax)
    assert float(gmax.item()) == 0.0
