"""Pins for the CPU oracle: what Algorithm 1 and plain mathematics fix, checked without a GPU.

Each test is chosen so that a plausible slip in the oracle (a wrong bit order, a sign(0)
or tie rule applied inconsistently, a dropped worker, a fused multiply-add, a padding
leak) fails at least one of them.
"""
import itertools

import numpy as np
import pytest

import oracle
from tests import golden_io

GOLD = golden_io.load()


def _f32(x):
    return np.asarray(x, dtype=np.float32)


# ---- sizes: 32x compression, 2Md bits per iteration (abstract; Appendix B) ---------------

@pytest.mark.parametrize("d,w", [(0, 0), (1, 1), (31, 1), (32, 1), (33, 2), (64, 2), (65, 3),
                                 (1 << 20, 1 << 15), (25_557_032, 798_658),
                                 (61_100_840, 1_909_402), (1 << 28, 1 << 23)])
def test_packed_words(d, w):
    assert oracle.packed_words(d) == w


def test_compression_ratio_and_bits_per_iteration():
    d, M = 1 << 20, 15
    packed_bytes = 4 * oracle.packed_words(d)
    assert 4 * d == 32 * packed_bytes                       # 32x less than fp32
    bits = M * 8 * packed_bytes + M * 8 * packed_bytes      # M up, one vote down to each
    assert bits == 2 * M * d


# ---- hand vectors -------------------------------------------------------------------------

@pytest.mark.parametrize("rec", GOLD["pack"], ids=lambda r: "%s-d%d" % (r[0], len(r[1])))
def test_pack_hand_vectors(rec):
    _, arr, want = rec
    got = oracle.sign_pack(arr)
    assert got.tolist() == want.tolist()


@pytest.mark.parametrize("rec", GOLD["vote"], ids=lambda r: "d%d-M%d-f%x" % (r[0], len(r[2]), r[1]))
def test_vote_hand_vectors(rec):
    d, flip, workers, want = rec
    got = oracle.majority_vote(workers, d, flip)
    assert got.tolist() == want.tolist()


@pytest.mark.parametrize("rec", GOLD["momentum"])
def test_momentum_hand_vectors(rec):
    beta, g, v0, v1, bit = rec
    v = _f32([v0])
    w = oracle.signum_update(_f32([g]), v, beta)
    assert v[0] == np.float32(v1)
    assert int(w[0]) == bit


@pytest.mark.parametrize("rec", GOLD["apply"])
def test_apply_hand_vectors(rec):
    x0, bit, lr, wd, x1 = rec
    x = _f32([x0])
    oracle.apply_vote(x, np.array([bit], dtype=np.uint32), lr, wd)
    assert x[0] == np.float32(x1)


# ---- pack: library routine, round trip, padding -------------------------------------------

@pytest.mark.parametrize("d", [1, 2, 31, 32, 33, 63, 64, 65, 127, 1000, 4097])
def test_pack_equals_numpy_little_endian_packbits(d):
    rng = np.random.default_rng(d)
    g = rng.standard_normal(d).astype(np.float32)
    g[rng.random(d) < 0.1] = 0.0
    g[rng.random(d) < 0.05] = -0.0
    bits = (g >= 0)
    by = np.packbits(bits, bitorder="little")
    by = np.concatenate([by, np.zeros((-len(by)) % 4, dtype=np.uint8)])
    want = by.view("<u4")
    assert oracle.sign_pack(g).tolist() == want.tolist()


def test_pack_unpack_round_trip_and_padding():
    rng = np.random.default_rng(7)
    for d in (1, 5, 32, 40, 999):
        g = rng.standard_normal(d).astype(np.float32)
        w = oracle.sign_pack(g)
        s = oracle.unpack(w, d)
        assert np.array_equal(s, np.where(g >= 0, 1, -1).astype(np.int8))
        if d % 32:
            assert int(w[-1]) >> (d % 32) == 0
        # pack(unpack(w)) == w
        assert oracle.sign_pack(s.astype(np.float32)).tolist() == w.tolist()


def test_bf16_pack_matches_fp32_pack_of_widened_values():
    rng = np.random.default_rng(3)
    h = rng.integers(0, 1 << 16, size=5000, dtype=np.uint16)
    f = (h.astype(np.uint32) << 16).view(np.float32)
    assert oracle.sign_pack(h).tolist() == oracle.sign_pack(f).tolist()


# ---- vote: brute force over every sign pattern --------------------------------------------

@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 6, 7, 8])
def test_vote_brute_force_all_patterns(M):
    # coordinate c carries pattern c: worker m sends +1 iff bit m of c is set.
    d = 1 << M
    signs = np.array([[1 if (c >> m) & 1 else -1 for c in range(d)] for m in range(M)])
    packed = [oracle.sign_pack(signs[m].astype(np.float32)) for m in range(M)]
    vote, tally = oracle.majority_vote(packed, d, 0, return_tally=True)
    V = signs.sum(axis=0)
    assert np.array_equal(tally, V)
    want = np.where(V >= 0, 1, -1)
    assert np.array_equal(oracle.unpack(vote, d), want)
    # and with every possible set of inverting workers
    for flip in range(1 << M):
        f = np.array([-1 if (flip >> m) & 1 else 1 for m in range(M)])[:, None]
        Vf = (signs * f).sum(axis=0)
        got = oracle.unpack(oracle.majority_vote(packed, d, flip), d)
        assert np.array_equal(got, np.where(Vf >= 0, 1, -1)), (M, flip)


def test_vote_m3_is_textbook_majority():
    rng = np.random.default_rng(11)
    d = 32 * 50
    a, b, c = (rng.integers(0, 1 << 32, size=50, dtype=np.uint32) for _ in range(3))
    want = (a & b) | (a & c) | (b & c)
    assert oracle.majority_vote([a, b, c], d).tolist() == want.tolist()


def test_vote_m1_is_identity():
    rng = np.random.default_rng(12)
    a = rng.integers(0, 1 << 32, size=9, dtype=np.uint32)
    assert oracle.majority_vote([a], 288).tolist() == a.tolist()


@pytest.mark.parametrize("M", [1, 2, 3, 7, 15, 16, 31, 63, 64])
def test_vote_identical_inputs_returns_input(M):
    rng = np.random.default_rng(M)
    d = 32 * 17 + 5
    g = rng.standard_normal(d).astype(np.float32)
    w = oracle.sign_pack(g)
    assert oracle.majority_vote([w.copy() for _ in range(M)], d).tolist() == w.tolist()


def test_vote_permutation_invariance_and_monotonicity():
    rng = np.random.default_rng(5)
    M, d = 7, 32 * 8 + 3
    W = oracle.packed_words(d)
    tail = np.uint32((1 << (d % 32)) - 1)
    packed = [rng.integers(0, 1 << 32, size=W, dtype=np.uint32) for _ in range(M)]
    for p in packed:
        p[-1] &= tail
    base = oracle.majority_vote(packed, d)
    perm = [packed[i] for i in rng.permutation(M)]
    assert oracle.majority_vote(perm, d).tolist() == base.tolist()
    # raising one worker's bits from 0 to 1 can only raise vote bits
    up = [p.copy() for p in packed]
    up[3] |= rng.integers(0, 1 << 32, size=W, dtype=np.uint32)
    up[3][-1] &= tail
    raised = oracle.majority_vote(up, d)
    assert np.all((base & ~raised) == 0)


@pytest.mark.parametrize("M", [3, 7, 15])
def test_vote_negation_symmetry_odd_m(M):
    rng = np.random.default_rng(100 + M)
    d = 32 * 6 + 9
    W = oracle.packed_words(d)
    tail = np.uint32((1 << (d % 32)) - 1)
    packed = [rng.integers(0, 1 << 32, size=W, dtype=np.uint32) for _ in range(M)]
    for p in packed:
        p[-1] &= tail
    v = oracle.majority_vote(packed, d)
    vn = oracle.majority_vote(packed, d, (1 << M) - 1)     # every worker inverts
    mask = np.full(W, 0xFFFFFFFF, dtype=np.uint32)
    mask[-1] = tail
    assert ((v ^ vn) == mask).all()


def test_vote_even_m_negation_differs_only_on_ties():
    rng = np.random.default_rng(42)
    M, d = 4, 32 * 20
    packed = [rng.integers(0, 1 << 32, size=20, dtype=np.uint32) for _ in range(M)]
    v, tally = oracle.majority_vote(packed, d, 0, return_tally=True)
    vn = oracle.majority_vote(packed, d, (1 << M) - 1)
    same = oracle.unpack(v, d) == oracle.unpack(vn, d)
    assert np.array_equal(same, tally == 0)
    assert np.all(oracle.unpack(v, d)[tally == 0] == 1)     # ties vote +1


@pytest.mark.parametrize("M,n_adv", [(3, 1), (7, 3), (15, 7), (63, 31)])
def test_unanimous_honest_coordinate_survives_minority_of_inverters(M, n_adv):
    # M odd, fewer than M/2 inverting workers: where all honest workers agree, the vote
    # is the honest sign (Theorem 2's setting with alpha < 1/2).
    rng = np.random.default_rng(M)
    d = 1000
    honest = rng.standard_normal(d).astype(np.float32)
    w = oracle.sign_pack(honest)
    flip = 0
    for m in rng.choice(M, size=n_adv, replace=False):
        flip |= 1 << int(m)
    vote = oracle.majority_vote([w.copy() for _ in range(M)], d, flip)
    assert vote.tolist() == w.tolist()
    # one more inverter and the vote is the complement on every valid bit
    extra = next(m for m in range(M) if not (flip >> m) & 1)
    vote2 = oracle.majority_vote([w.copy() for _ in range(M)], d, flip | (1 << extra))
    assert np.array_equal(oracle.unpack(vote2, d), -oracle.unpack(w, d))


def test_duplicating_every_worker_keeps_non_tie_coordinates():
    rng = np.random.default_rng(8)
    M, d = 5, 32 * 10
    packed = [rng.integers(0, 1 << 32, size=10, dtype=np.uint32) for _ in range(M)]
    v = oracle.majority_vote(packed, d)
    v2 = oracle.majority_vote(packed + [p.copy() for p in packed], d)
    assert v.tolist() == v2.tolist()


# ---- momentum -----------------------------------------------------------------------------

def test_beta_zero_is_signsgd():
    rng = np.random.default_rng(21)
    d = 3000
    g = rng.standard_normal(d).astype(np.float32)
    g[::7] = -0.0
    g[::11] = 0.0
    v = rng.standard_normal(d).astype(np.float32)
    w = oracle.signum_update(g, v, 0.0)
    assert w.tolist() == oracle.sign_pack(g).tolist()
    assert np.array_equal(v, g)          # as values (-0.0 == +0.0)


def test_momentum_geometric_series_closed_form():
    # constant gradient g from v = 0: v_k = (1 - beta^k) g.
    rng = np.random.default_rng(22)
    d, beta = 2000, 0.9
    g = rng.standard_normal(d).astype(np.float32)
    v = np.zeros(d, dtype=np.float32)
    for k in range(1, 41):
        oracle.signum_update(g, v, beta)
        want = (1.0 - np.float64(np.float32(beta)) ** k) * g.astype(np.float64)
        assert np.allclose(v, want, rtol=5e-6, atol=0), k


def test_momentum_is_two_rounded_multiplies_and_one_rounded_add():
    # numpy float32 arithmetic rounds every operation separately; a contracted (fused
    # multiply-add) evaluation gives different values on a measurable share of inputs.
    rng = np.random.default_rng(23)
    d = 1 << 18
    beta = np.float32(0.9)
    omb = np.float32(1.0) - beta
    g = rng.standard_normal(d).astype(np.float32)
    v0 = rng.standard_normal(d).astype(np.float32)
    # make many near-cancellations so that the sign itself depends on the rounding
    v0[: d // 2] = (-(omb * g[: d // 2]) / beta).astype(np.float32)
    v = v0.copy()
    w = oracle.signum_update(g, v, float(beta))
    two_step = (omb * g) + (beta * v0)
    assert two_step.dtype == np.float32
    assert np.array_equal(v.view(np.uint32), two_step.view(np.uint32))
    fused = (np.float64(omb) * g.astype(np.float64) + (beta * v0).astype(np.float64)).astype(np.float32)
    assert np.count_nonzero(fused != two_step) > 1000          # the test can tell them apart
    assert np.count_nonzero((fused >= 0) != (two_step >= 0)) > 10
    assert np.array_equal(oracle.unpack(w, d) > 0, two_step >= 0)


def test_momentum_keeps_denormals():
    g = np.array([1e-38, -1e-38, 1e-44], dtype=np.float32)
    v = np.zeros(3, dtype=np.float32)
    oracle.signum_update(g, v, 0.9)
    want = (np.float32(1.0) - np.float32(0.9)) * g
    assert np.array_equal(v.view(np.uint32), want.view(np.uint32))
    assert v[0] != 0 and v[1] != 0       # not flushed to zero


def test_first_step_signs_equal_gradient_signs():
    rng = np.random.default_rng(24)
    g = rng.standard_normal(5000).astype(np.float32)
    v = np.zeros_like(g)
    w = oracle.signum_update(g, v, 0.9)
    assert w.tolist() == oracle.sign_pack(g).tolist()


# ---- apply --------------------------------------------------------------------------------

def test_apply_moves_every_coordinate_by_lr():
    rng = np.random.default_rng(31)
    d, lr = 4099, 1e-3
    x0 = rng.standard_normal(d).astype(np.float32)
    vote = oracle.sign_pack(rng.standard_normal(d).astype(np.float32))
    x = x0.copy()
    oracle.apply_vote(x, vote, lr)
    s = oracle.unpack(vote, d).astype(np.float64)
    assert np.allclose(x.astype(np.float64), x0.astype(np.float64) - lr * s, rtol=0, atol=1.2e-7 * 4)
    # sum of the steps counts the votes: sum (x0 - x)/lr = 2 popcount(vote) - d
    pop = sum(bin(int(w)).count("1") for w in vote)
    total = ((x0.astype(np.float64) - x.astype(np.float64)) / lr).sum()
    assert abs(total - (2 * pop - d)) < 1.0


def test_apply_weight_decay_matches_float64_formula():
    rng = np.random.default_rng(32)
    d, lr, wd = 1000, 1e-2, 0.1
    x0 = rng.standard_normal(d).astype(np.float32)
    vote = oracle.sign_pack(rng.standard_normal(d).astype(np.float32))
    x = x0.copy()
    oracle.apply_vote(x, vote, lr, wd)
    s = oracle.unpack(vote, d).astype(np.float64)
    want = x0 - lr * (s + wd * x0.astype(np.float64))
    assert np.allclose(x, want, rtol=1e-6, atol=1e-7)


def test_single_worker_no_momentum_is_theorem_1_update():
    # M = 1, beta = 0: x <- x - eta sign(g).
    rng = np.random.default_rng(33)
    d, lr = 777, 0.5
    g = rng.standard_normal(d).astype(np.float32)
    x0 = rng.standard_normal(d).astype(np.float32)
    x = x0.copy()
    oracle.fused_step([g], None, x, beta=0.0, lr=lr)
    want = x0 - np.float32(lr) * np.where(g >= 0, 1, -1).astype(np.float32)
    assert np.array_equal(x, want)


# ---- fused step == the unfused chain --------------------------------------------------------

@pytest.mark.parametrize("M,momentum,flip,wd,bf16", [
    (1, False, 0, 0.0, False), (3, False, 0, 0.0, False), (7, False, 0x70, 0.0, False),
    (15, True, 0, 0.0, False), (16, True, 0, 0.0, True), (4, True, 0b0101, 0.01, False),
    (63, False, 0, 0.0, False)])
def test_fused_step_equals_unfused_chain(M, momentum, flip, wd, bf16):
    rng = np.random.default_rng(1000 + M)
    d, beta, lr = 32 * 40 + 8, 0.9, 1e-3
    x_f = rng.standard_normal(d).astype(np.float32)
    x_u = x_f.copy()
    mom_f = [rng.standard_normal(d).astype(np.float32) for _ in range(M)] if momentum else None
    mom_u = [v.copy() for v in mom_f] if momentum else None
    for step in range(3):
        grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
        if bf16:
            grads = [(g.view(np.uint32) >> 16).astype(np.uint16) for g in grads]
        vote_f = oracle.fused_step(grads, mom_f, x_f, beta, lr, wd, flip)
        if momentum:
            packed = [oracle.signum_update(grads[m], mom_u[m], beta) for m in range(M)]
        else:
            packed = [oracle.sign_pack(g) for g in grads]
        vote_u = oracle.majority_vote(packed, d, flip)
        oracle.apply_vote(x_u, vote_u, lr, wd)
        assert vote_f.tolist() == vote_u.tolist()
        assert np.array_equal(x_f.view(np.uint32), x_u.view(np.uint32))
        if momentum:
            for a, b in zip(mom_f, mom_u):
                assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


# ---- robustness -----------------------------------------------------------------------------

def test_positive_rescaling_changes_nothing():
    # sign(v * g) = sign(v) sign(g): a positive multiplier has no effect (proof of Theorem 2).
    rng = np.random.default_rng(41)
    M, d = 5, 2000
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
    x1 = rng.standard_normal(d).astype(np.float32)
    x2 = x1.copy()
    v1 = oracle.fused_step(grads, None, x1, 0.0, 1e-3)
    scaled = [g.copy() for g in grads]
    scaled[2] = (scaled[2] * np.exp(rng.standard_normal(d) * 3).astype(np.float32)).astype(np.float32)
    scaled[2][scaled[2] == 0] = np.copysign(np.float32(1e-30), grads[2][scaled[2] == 0])
    v2 = oracle.fused_step(scaled, None, x2, 0.0, 1e-3)
    assert v1.tolist() == v2.tolist()
    assert np.array_equal(x1, x2)


@pytest.mark.parametrize("poison", [np.inf, -np.inf, np.nan])
def test_one_poisoned_worker_cannot_corrupt_the_parameters(poison):
    rng = np.random.default_rng(43)
    M, d = 3, 1000
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
    grads[1][:] = poison
    moms = [np.zeros(d, dtype=np.float32) for _ in range(M)]
    x = rng.standard_normal(d).astype(np.float32)
    x0 = x.copy()
    for _ in range(3):
        oracle.fused_step(grads, moms, x, 0.9, 1e-2)
    assert np.all(np.isfinite(x))
    assert np.all(np.abs(x - x0) <= 3 * 1e-2 * 1.0001)
    assert np.all(np.isfinite(moms[0])) and np.all(np.isfinite(moms[2]))


def test_threads_do_not_change_results():
    rng = np.random.default_rng(44)
    M, d = 7, 32 * 300 + 17
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
    outs = []
    for n in (1, 4):
        oracle.set_threads(n)
        try:
            x = np.ones(d, dtype=np.float32)
            moms = [np.zeros(d, dtype=np.float32) for _ in range(M)]
            vote = oracle.fused_step(grads, moms, x, 0.9, 1e-3, 0.0, 0x3)
            outs.append((vote.copy(), x.copy(), [v.copy() for v in moms]))
        finally:
            oracle.set_threads(1)
    assert outs[0][0].tolist() == outs[1][0].tolist()
    assert np.array_equal(outs[0][1], outs[1][1])
    for a, b in zip(outs[0][2], outs[1][2]):
        assert np.array_equal(a, b)
