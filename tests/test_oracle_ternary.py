"""Pins of the oracle's ternary codec (Appendix B: 1-bit max-norm QSGD, the comparison codec).

What fixes it from outside: the published known-answer vectors of the Philox4x32-10 generator;
hand-worked keep/drop decisions at the rounding boundary with the draws given as inputs; the two
special cases Appendix B itself states (a sign vector is left unchanged; a vector with a single
non-zero entry keeps that entry alone); the size 2d bits; and the probabilities
|g_i| / ||g||_inf themselves, checked statistically over many seeds, together with the
unbiasedness E[||g||_inf q] = g that the stochastic rounding is for.
"""
import os
import re

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _records(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [p.strip() for p in line.split("|")]


def _hex_words(s):
    out = []
    for m in re.finditer(r"(\d+)\*\(([^)]*)\)|([0-9a-fA-F]+)", s):
        if m.group(1):
            out.extend(m.group(2).split() * int(m.group(1)))
        else:
            out.append(m.group(3))
    return np.array([int(t, 16) for t in out], dtype=np.uint32)


def test_generator_reproduces_the_published_known_answers():
    n = 0
    for counter, key, want in _records("philox4x32_10_kat.txt"):
        got = oracle.philox4x32_10(_hex_words(counter), _hex_words(key))
        assert np.array_equal(got, _hex_words(want)), (counter, key)
        n += 1
    assert n == 3


def test_draws_are_the_generators_blocks_addressed_by_coordinate():
    seed = 0x0123456789ABCDEF
    r = oracle.ternary_draws(seed, 1003)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for c in (0, 1, 2, 3, 4, 5, 999, 1002):
        block = oracle.philox4x32_10([c // 4, 0, 0, 0], key)
        assert r[c] == block[c % 4]
    assert np.array_equal(r[:500], oracle.ternary_draws(seed, 500))       # a prefix is a prefix
    assert not np.array_equal(r, oracle.ternary_draws(seed + 1, 1003))    # the seed matters
    # roughly uniform: the mean of 1003 draws of 32 bits
    assert abs(r.astype(np.float64).mean() / 2 ** 32 - 0.5) < 0.05


def test_hand_worked_decisions():
    n = 0
    for gmax, values, draws, want in _records("ternary_hand_vectors.txt"):
        g = np.array([float(v) for v in values.split()], dtype=np.float32)
        r = _hex_words(draws)
        codes = oracle.ternary_pack(g, gmax=float(gmax), draws=r)
        assert np.array_equal(codes, _hex_words(want)), values
        assert oracle.absmax(g) == float(gmax)
        n += 1
    assert n == 3


def test_size_is_two_bits_per_coordinate():
    for d, w in ((0, 0), (1, 1), (16, 1), (17, 2), (25_557_032, 1_597_315)):
        assert oracle.ternary_words(d) == w
    assert oracle.ternary_words(1 << 20) * 32 == 2 * (1 << 20)       # 2 d bits (Appendix B)


def test_sign_vectors_come_through_unchanged():
    rng = np.random.default_rng(5)
    d = 1000
    s = np.where(rng.random(d) < 0.5, -1.0, 1.0).astype(np.float32) * np.float32(0.37)
    for seed in (1, 2, 3):
        codes = oracle.ternary_pack(s, seed=seed)
        back = oracle.ternary_unpack(codes, d, oracle.absmax(s))
        assert np.array_equal(back, s)
    # padding bits of the last word are zero
    assert int(codes[-1]) >> (2 * (d % 16)) == 0


def test_a_single_non_zero_entry_is_kept_alone():
    g = np.zeros(777, dtype=np.float32)
    g[123] = -2.5
    for seed in range(5):
        back = oracle.ternary_unpack(oracle.ternary_pack(g, seed=seed), 777, 1.0)
        want = np.zeros(777, dtype=np.float32)
        want[123] = -1.0
        assert np.array_equal(back, want)


def test_special_values():
    g = np.array([np.nan, 0.0, -0.0, 1.0, -np.nan], dtype=np.float32)
    assert oracle.absmax(g) == 1.0                                         # NaN is skipped
    back = oracle.ternary_unpack(oracle.ternary_pack(g, seed=9), 5, 1.0)
    assert np.array_equal(back, np.array([0, 0, 0, 1, 0], dtype=np.float32))
    assert oracle.absmax(np.zeros(4, dtype=np.float32)) == 0.0
    assert not oracle.ternary_pack(np.zeros(40, dtype=np.float32), seed=1).any()
    inf = np.array([np.inf, 1.0, -3.0], dtype=np.float32)                  # an infinite maximum keeps nothing
    assert not oracle.ternary_pack(inf, seed=1).any()
    assert oracle.absmax(np.zeros(0, dtype=np.float32)) == 0.0


def test_bf16_gradients_are_widened_exactly():
    g32 = np.array([1.5, -0.75, 0.0, 3.0, -3.0, 0.125], dtype=np.float32)   # all exact in bf16
    raw = (g32.view(np.uint32) >> 16).astype(np.uint16)
    assert oracle.absmax(raw) == 3.0
    for seed in (4, 5):
        assert np.array_equal(oracle.ternary_pack(raw, seed=seed), oracle.ternary_pack(g32, seed=seed))


def test_keep_rate_and_unbiasedness_over_many_seeds():
    """P[kept] = |g_i| / ||g||_inf and E[||g||_inf q_i] = g_i (the point of stochastic rounding)."""
    rng = np.random.default_rng(11)
    d, n_seeds = 40_000, 96
    g = rng.standard_normal(d).astype(np.float32)
    gmax = oracle.absmax(g)
    assert gmax == float(np.abs(g).max())
    p = np.abs(g.astype(np.float64)) / gmax
    kept = np.zeros(d)
    mean = np.zeros(d)
    for seed in range(n_seeds):
        q = oracle.ternary_unpack(oracle.ternary_pack(g, seed=1000 + seed), d, 1.0).astype(np.float64)
        assert np.all((q == 0) | (np.sign(q) == np.sign(g)))               # a kept sign is the gradient's
        kept += q != 0
        mean += q
    # keep rate per probability bin against the bin's mean probability
    edges = np.linspace(0, 1, 11)
    for lo, hi in zip(edges[:-1], edges[1:]):
        sel = (p >= lo) & (p < hi)
        n = int(sel.sum()) * n_seeds
        if n < 2000:
            continue
        rate, want = kept[sel].sum() / n, p[sel].mean()
        sigma = np.sqrt(max(want * (1 - want), 1e-6) / n)
        assert abs(rate - want) < 5 * sigma, (lo, hi, rate, want)
    # unbiasedness: standardised residuals of the per-coordinate mean have mean 0 and variance 1
    est = mean / n_seeds * gmax
    sd = gmax * np.sqrt(p * (1 - p) / n_seeds)
    ok = sd > 0
    z = (est[ok] - g[ok]) / sd[ok]
    assert abs(z.mean()) < 5 / np.sqrt(ok.sum())
    assert abs((z ** 2).mean() - 1.0) < 0.05
    # the coordinate that attains the maximum is always kept
    assert kept[np.argmax(np.abs(g))] == n_seeds
