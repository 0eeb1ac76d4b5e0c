"""Statistical pins: input generator + oracle pack + oracle vote against the binomial model
in the proof of Theorem 2 (Z = G + B, G ~ Bin((1-alpha)M, p), B ~ Bin(alpha M, q), the vote
fails iff Z <= M/2), with Gaussian noise so that p = Phi(S), S = |signal| / sigma.
Expected rates are computed here by quadrature over the N(0,1) signal, not by any
implementation of the method."""
import math

import numpy as np
import pytest
import torch
from scipy import integrate, stats

import oracle
from paper_1810_05291_b200 import inputs


def single_worker_error(sigma: float) -> float:
    # P[sign(s + sigma n) != sign(s)], s, n ~ N(0,1): closed form arctan(sigma)/pi.
    return math.atan(sigma) / math.pi


def vote_error(M: int, sigma: float, n_adv: int) -> float:
    good = M - n_adv

    def fail_given_s(s):
        p = stats.norm.cdf(abs(s) / sigma)
        q = 1.0 - p
        # P[G + B <= (M-1)/2] for odd M
        pg = stats.binom.pmf(np.arange(good + 1), good, p)
        pb = stats.binom.pmf(np.arange(n_adv + 1), n_adv, q)
        pz = np.convolve(pg, pb)
        return pz[: (M - 1) // 2 + 1].sum() * stats.norm.pdf(s)

    val, _ = integrate.quad(fail_given_s, -10, 10, limit=400, points=[0.0])
    return val


def test_closed_forms_of_the_model():
    assert abs(single_worker_error(1.0) - 0.25) < 1e-12
    assert abs(single_worker_error(2.0) - 0.352416) < 1e-6
    assert abs(vote_error(3, 1.0, 0) - 3.0 / 16.0) < 1e-6
    assert abs(vote_error(15, 1.0, 0) - 0.098190) < 2e-6
    assert abs(vote_error(7, 2.0, 0) - 0.235961) < 2e-6
    assert abs(vote_error(7, 2.0, 3) - 0.443505) < 2e-6
    # the 1-worker vote is the single-worker sign
    assert abs(vote_error(1, 2.0, 0) - single_worker_error(2.0)) < 1e-6


def _rates(case, d):
    case.d = d
    dev = torch.device("cpu")
    s = inputs.signal(case, dev, 0)
    truth = (s >= 0).numpy()
    packed, single = [], []
    for m in range(case.M):
        g = inputs.worker_gradient(case, m, dev, 0, s).numpy()
        w = oracle.sign_pack(g)
        packed.append(w)
        single.append(np.mean((oracle.unpack(w, d) > 0) != truth))
    vote = oracle.majority_vote(packed, d, case.flip_mask)
    vote_err = np.mean((oracle.unpack(vote, d) > 0) != truth)
    return float(np.mean(single)), float(vote_err), s.numpy(), packed, vote


@pytest.mark.parametrize("which", ["cfg3", "cfg2"])
def test_sign_and_vote_error_rates_match_binomial_model(which):
    d = 1 << 21
    case = inputs.cfg3(d) if which == "cfg3" else inputs.cfg2(d)
    n_adv = bin(case.flip_mask).count("1")
    single, vote_err, s, packed, vote = _rates(case, d)
    se1 = math.sqrt(0.25 / (d * case.M))
    se2 = math.sqrt(0.25 / d)
    assert abs(single - single_worker_error(case.sigma)) < 6 * se1 + 1e-4
    assert abs(vote_err - vote_error(case.M, case.sigma, n_adv)) < 6 * se2


def test_vote_failure_obeys_the_star_bound_and_lemma_1():
    # Bin coordinates by SNR; in every bin the empirical failure rates stay under
    # 1/((1-2 alpha) sqrt(M) S) (proof of Theorem 2) and under Lemma 1's bound.
    d = 1 << 21
    case = inputs.cfg2(d)
    M, n_adv = case.M, bin(case.flip_mask).count("1")
    alpha = n_adv / M
    _, _, s, packed, vote = _rates(case, d)
    S = np.abs(s) / case.sigma
    truth = s >= 0
    vote_bad = (oracle.unpack(vote, d) > 0) != truth
    honest_bad = (oracle.unpack(packed[0], d) > 0) != truth
    edges = np.array([0.05, 0.1, 0.2, 0.4, 0.8, 1.2, 1.6, 2.0])
    for lo, hi in zip(edges[:-1], edges[1:]):
        sel = (S >= lo) & (S < hi)
        n = sel.sum()
        assert n > 1000
        slack = 5 * math.sqrt(0.25 / n)
        star = 1.0 / ((1 - 2 * alpha) * math.sqrt(M) * lo)
        assert vote_bad[sel].mean() <= min(star, 1.0) + slack
        lemma = (2.0 / 9.0) / lo ** 2 if lo > 2 / math.sqrt(3) else 0.5 - lo / (2 * math.sqrt(3))
        assert honest_bad[sel].mean() <= lemma + slack
