"""The five named workloads at full size, in the launch configuration the benchmark times.

The ResNet-50- and AlexNet-sized workloads (cfg2, cfg3, cfg4 and the even-M tie probe) are
compared with the CPU oracle over the WHOLE vector, element by element, at every step: packed
vote words, parameters and every worker's momentum. Only vectors longer than 2^26 coordinates
(the sweep's d = 2^28 and the > 2^31 vector) are compared on sampled windows instead (every
coordinate is independent, so a window of the inputs determines the same window of every output):
the first 2^20 coordinates, the last ones including the ragged word, and seeded windows in
between. On top of that the tests check what holds at any size: the fused step equals the unfused
chain bit for bit, padding bits are zero, and the empirical sign/vote error rates match the
binomial model in the proof of Theorem 2.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B
from paper_1810_05291_b200 import inputs
from tests.test_oracle_stats import single_worker_error, vote_error
from tests.util import (assert_f32_close, assert_f32_state, assert_words_equal, count_bit_mismatch, to_np,
                        words_tensor)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
WINDOW = 1 << 20
FULL_PARITY_MAX_D = 1 << 26      # up to here the oracle checks every coordinate


@pytest.fixture(scope="module", autouse=True)
def _oracle_threads():
    oracle.set_threads(min(16, oracle.max_threads()))
    yield
    oracle.set_threads(1)


@pytest.fixture(autouse=True)
def _free_gpu_memory():
    yield
    torch.cuda.empty_cache()


def windows(d: int, n_random: int = 6, seed: int = 0):
    """The coordinate ranges [a, b) the oracle is run on: the whole vector up to FULL_PARITY_MAX_D
    coordinates; beyond that word-aligned windows: first, last (with the ragged word), seeded others."""
    if d <= FULL_PARITY_MAX_D:
        return [(0, d)]
    out = [(0, WINDOW), (((d - WINDOW) // 32) * 32, d)]
    rng = np.random.default_rng(seed)
    for _ in range(n_random):
        a = int(rng.integers(0, (d - WINDOW) // 32)) * 32
        out.append((a, a + WINDOW))
    return out


def unpack_bits(words: torch.Tensor, d: int) -> torch.Tensor:
    """Test-side unpacking of packed words to a bool vector (bit i of word j = coordinate 32j+i)."""
    shifts = torch.arange(32, device=words.device, dtype=torch.int32)
    return ((words.view(-1, 1) >> shifts) & 1).view(-1)[:d].bool()


def unfused_chain(case, grads, moms, x, vote):
    packed = [words_tensor(case.d, DEV) for _ in range(case.M)]
    for m in range(case.M):
        if moms is not None:
            B.ss_signum_update(grads[m], moms[m], case.beta, packed[m])
        else:
            B.ss_sign_pack(grads[m], packed[m])
    B.ss_majority_vote(packed, case.d, case.flip_mask, vote)
    B.ss_apply_vote(x, vote, case.lr, case.weight_decay)
    return packed


def run_case(case, steps: int, stats: bool = False, check_chain: bool = True):
    d, M = case.d, case.M
    beta = case.beta if case.beta is not None else 0.0
    x = inputs.initial_params(case, DEV)
    moms = inputs.zero_momenta(case, DEV)
    vote = words_tensor(d, DEV, fill=-1)
    wins = windows(d, seed=case.cfg)
    ox = [to_np(x[a:b]) for a, b in wins]
    om = [[np.zeros(b - a, dtype=np.float32) for _ in range(M)] if moms is not None else None
          for a, b in wins]
    if check_chain:
        x_u = x.clone()
        x_va = x.clone()
        moms_u = [v.clone() for v in moms] if moms is not None else None
        vote_u = words_tensor(d, DEV, fill=-1)
        vote_va = words_tensor(d, DEV, fill=-1)
    result = {}
    for step in range(steps):
        s = inputs.signal(case, DEV, step)
        grads = [inputs.worker_gradient(case, m, DEV, step, s) for m in range(M)]
        B.ss_fused_step(grads, moms, x, beta, case.lr, case.weight_decay, case.flip_mask, vote)
        torch.cuda.synchronize()
        # the oracle, on the whole vector (or on sampled windows beyond FULL_PARITY_MAX_D)
        for wi, (a, b) in enumerate(wins):
            g_np = [to_np(g[a:b]) for g in grads]
            want = oracle.fused_step(g_np, om[wi], ox[wi], beta, case.lr, case.weight_decay, case.flip_mask)
            wa, wb = a // 32, (b + 31) // 32
            assert_words_equal(vote[wa:wb], want, "vote words, window %d, step %d" % (wi, step))
            assert_f32_state(x[a:b], ox[wi], "parameters, window %d, step %d" % (wi, step))
            if moms is not None:
                for m in range(M):
                    assert_f32_state(moms[m][a:b], om[wi][m], "momentum %d, window %d, step %d" % (m, wi, step))
        # whole vectors: padding, and the fused step against the unfused chain
        if d % 32:
            assert int(vote[-1].item()) & 0xFFFFFFFF & ~((1 << (d % 32)) - 1) == 0, "padding bits set"
        if check_chain:
            packed = unfused_chain(case, grads, moms_u, x_u, vote_u)
            assert torch.equal(vote, vote_u), "fused and unfused vote differ at step %d" % step
            assert torch.equal(x.view(torch.int32), x_u.view(torch.int32))
            # the same packed words through the one-pass vote + update
            B.ss_vote_apply(packed, x_va, case.lr, case.weight_decay, case.flip_mask, vote_va)
            assert torch.equal(vote, vote_va), "ss_vote_apply vote differs at step %d" % step
            assert torch.equal(x.view(torch.int32), x_va.view(torch.int32))
            if moms is not None:
                for a_, b_ in zip(moms, moms_u):
                    assert torch.equal(a_.view(torch.int32), b_.view(torch.int32))
        if stats and step == 0:
            truth = s >= 0
            if check_chain:
                errs = [float((unpack_bits(p, d) != truth).float().mean().item()) for p in packed]
                result["single"] = errs
            result["vote"] = float((unpack_bits(vote, d) != truth).float().mean().item())
        del grads, s
    return result


def test_cfg1_plain_vote_and_apply():
    case = inputs.cfg1()
    run_case(case, steps=1)


def test_cfg2_alexnet_sized_with_three_inverting_workers():
    case = inputs.cfg2()
    r = run_case(case, steps=1, stats=True)
    d = case.d
    # honest workers' sign error, inverters' sign error (= 1 - honest), and the vote's
    honest = [e for m, e in enumerate(r["single"]) if not (case.flip_mask >> m) & 1]
    tol = 5e-4
    for e in honest:
        assert abs(e - single_worker_error(2.0)) < tol
    assert abs(r["vote"] - vote_error(7, 2.0, 3)) < tol
    assert abs(vote_error(7, 2.0, 3) - 0.443505) < 1e-5
    # bound (*) of Theorem 2's proof is respected on average as well: the vote is right more often than not
    assert r["vote"] < 0.5


def test_cfg2_unanimous_honest_coordinates_survive_the_inverters():
    # where all 4 honest workers agree, 3 inverters cannot change the outcome
    case = inputs.cfg2(d=4_000_000 + 8)
    grads = inputs.gradients(case, DEV, 0)
    x = inputs.initial_params(case, DEV)
    vote = words_tensor(case.d, DEV)
    B.ss_fused_step(grads, None, x, 0.0, case.lr, 0.0, case.flip_mask, vote)
    signs = torch.stack([g >= 0 for g in grads[:4]])
    all_pos, all_neg = signs.all(dim=0), (~signs).all(dim=0)
    v = unpack_bits(vote, case.d)
    assert bool(v[all_pos].all()) and not bool(v[all_neg].any())
    assert int(all_pos.sum()) + int(all_neg.sum()) > case.d // 10


def test_cfg3_resnet50_sized_signum_four_steps():
    case = inputs.cfg3()
    r = run_case(case, steps=4, stats=True)
    tol = 5e-4
    # step 1 starts from zero momentum, so sign(v) = sign(g): the model's rates apply
    for e in r["single"]:
        assert abs(e - 0.25) < tol
    assert abs(r["vote"] - vote_error(15, 1.0, 0)) < tol
    assert abs(vote_error(15, 1.0, 0) - 0.098190) < 1e-5


def test_cfg4_bf16_heavy_tails_zeros_four_steps():
    case = inputs.cfg4()
    run_case(case, steps=4)


def test_cfg4_zero_prefix_votes_plus_one():
    case = inputs.cfg4(d=1_000_000 + 8)
    grads = inputs.gradients(case, DEV, 0)
    moms = inputs.zero_momenta(case, DEV)
    x = inputs.initial_params(case, DEV)
    x0 = x.clone()
    vote = words_tensor(case.d, DEV)
    B.ss_fused_step(grads, moms, x, case.beta, case.lr, 0.0, 0, vote)
    v = unpack_bits(vote, case.d)
    assert bool(v[:4096].all())                        # sign(0) = +1 for every worker
    assert torch.equal(x[:4096], x0[:4096] - case.lr)
    zero_share = float(torch.stack([(g == 0).float().mean() for g in grads]).mean().item())
    assert abs(zero_share - 0.10) < 0.01


def test_cfg4_even_m_tie_probe():
    case = inputs.cfg4(tie_probe=True)
    assert case.M == 16
    run_case(case, steps=4, check_chain=False)
    # count ties on a window with the oracle's integer tally and check that they vote +1
    d = 1 << 20
    small = inputs.cfg4(d=d, tie_probe=True)
    grads = inputs.gradients(small, DEV, 0)
    assert torch.equal(grads[15], grads[0])
    packed = [words_tensor(d, DEV) for _ in range(16)]
    for m in range(16):
        B.ss_sign_pack(grads[m], packed[m])
    vote = words_tensor(d, DEV)
    B.ss_majority_vote(packed, d, 0, vote)
    want, tally = oracle.majority_vote([to_np(p) for p in packed], d, 0, return_tally=True)
    assert_words_equal(vote, want)
    ties = tally == 0
    assert ties.sum() > 1000
    assert bool(unpack_bits(vote, d).cpu().numpy()[ties].all())


@pytest.mark.parametrize("M", inputs.SWEEP_M)
@pytest.mark.parametrize("log2d", [16, 20, 24])
def test_cfg5_sweep_full_parity(log2d, M):
    d = 1 << log2d
    case = inputs.cfg5(d, M)
    grads = inputs.gradients(case, DEV, 0)
    g_np = [to_np(g) for g in grads]
    # vote-only path on pre-packed words
    packed = [words_tensor(d, DEV) for _ in range(M)]
    for m in range(M):
        B.ss_sign_pack(grads[m], packed[m])
    vote = words_tensor(d, DEV, fill=-1)
    B.ss_majority_vote(packed, d, 0, vote)
    packed_np = [oracle.sign_pack(g) for g in g_np]
    for m in (0, M - 1):
        assert_words_equal(packed[m], packed_np[m], "packed signs of worker %d" % m)
    assert_words_equal(vote, oracle.majority_vote(packed_np, d), "vote-only path")
    # fused path
    x = inputs.initial_params(case, DEV)
    x_np = to_np(x)
    vote2 = words_tensor(d, DEV, fill=-1)
    B.ss_fused_step(grads, None, x, 0.0, case.lr, 0.0, 0, vote2)
    want = oracle.fused_step(g_np, None, x_np, 0.0, case.lr)
    assert_words_equal(vote2, want, "fused path")
    assert torch.equal(vote, vote2)
    assert count_bit_mismatch(x, x_np) == 0


@pytest.mark.parametrize("M", [1, 15, 63])
def test_cfg5_sweep_largest_d_on_windows(M):
    d = 1 << 28
    free, _ = torch.cuda.mem_get_info()
    if free < (M * d * 4 + 3 * d * 4) * 1.05:
        pytest.skip("not enough free device memory for M=%d, d=2^28" % M)
    case = inputs.cfg5(d, M)
    grads = [inputs.worker_gradient(case, m, DEV, 0, None) for m in range(M)]
    x = inputs.initial_params(case, DEV)
    wins = windows(d, seed=M)
    ox = [to_np(x[a:b]) for a, b in wins]
    vote = words_tensor(d, DEV, fill=-1)
    B.ss_fused_step(grads, None, x, 0.0, case.lr, 0.0, 0, vote)
    # vote-only path
    packed = [words_tensor(d, DEV) for _ in range(M)]
    for m in range(M):
        B.ss_sign_pack(grads[m], packed[m])
    vote2 = words_tensor(d, DEV, fill=-1)
    B.ss_majority_vote(packed, d, 0, vote2)
    assert torch.equal(vote, vote2)
    for wi, (a, b) in enumerate(wins):
        g_np = [to_np(g[a:b]) for g in grads]
        want = oracle.fused_step(g_np, None, ox[wi], 0.0, case.lr)
        assert_words_equal(vote[a // 32:(b + 31) // 32], want, "vote words, window %d" % wi)
        assert count_bit_mismatch(x[a:b], ox[wi]) == 0
    # the model's vote error for pure-noise inputs is 1/2 against any fixed reference; check the
    # vote is balanced instead: each bit is +1 with probability 1/2 for odd M
    share = float(unpack_bits(vote, d).float().mean().item())
    assert abs(share - 0.5) < 5e-4


def _window_table(begins, lrs, wds, a, b, d):
    """The segment table restricted to coordinates [a, b), with begins relative to a."""
    out_b, out_lr, out_wd = [], [], []
    n = len(begins)
    for k in range(n):
        lo, hi = begins[k], begins[k + 1] if k + 1 < n else d
        if hi > a and lo < b and hi > lo:
            out_b.append(max(lo, a) - a)
            out_lr.append(lrs[k])
            out_wd.append(wds[k])
    return out_b, out_lr, out_wd


def test_cfg3_as_a_fused_vector_of_161_tensors():
    """Tensor fusion at full size: the ResNet-50-sized vector cut into 161 tensors (that model's
    number of parameter tensors) at seeded, unaligned coordinates, each with its own learning rate
    and weight decay, against one oracle step per tensor on sampled windows."""
    case = inputs.cfg3()
    d, M, n_seg = case.d, case.M, 161
    rng = np.random.default_rng(161)
    begins = [0] + sorted(int(c) for c in rng.integers(1, d, size=n_seg - 1))
    lrs = [float(10.0 ** rng.uniform(-5, -3)) for _ in range(n_seg)]
    wds = [0.0 if k % 2 else float(10.0 ** rng.uniform(-4, -2)) for k in range(n_seg)]
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)
    x = inputs.initial_params(case, DEV)
    moms = inputs.zero_momenta(case, DEV)
    vote = words_tensor(d, DEV, fill=-1)
    # windows: the standard ones plus one around each of three tensor boundaries
    wins = windows(d, seed=161)
    for k in (1, 80, 160):
        a = max(0, (begins[k] - 5000) // 32 * 32)
        wins.append((a, min(d, a + 10_016)))
    ox = [to_np(x[a:b]) for a, b in wins]
    om = [[np.zeros(b - a, dtype=np.float32) for _ in range(M)] for a, b in wins]
    for step in range(2):
        s = inputs.signal(case, DEV, step)
        grads = [inputs.worker_gradient(case, m, DEV, step, s) for m in range(M)]
        B.ss_fused_step_segments(grads, moms, x, case.beta, tab, n_seg, 0, vote)
        torch.cuda.synchronize()
        for wi, (a, b) in enumerate(wins):
            wb, wl, ww = _window_table(begins, lrs, wds, a, b, d)
            want = oracle.fused_step_segments([to_np(g[a:b]) for g in grads], om[wi], ox[wi], case.beta,
                                              wb, wl, ww)
            if b - a >= 32 and a % 32 == 0 and (b % 32 == 0 or b == d):
                assert_words_equal(vote[a // 32:(b + 31) // 32], want, "vote, window %d" % wi)
            assert count_bit_mismatch(x[a:b], ox[wi]) == 0, "parameters, window %d, step %d" % (wi, step)
            for m in range(M):
                assert count_bit_mismatch(moms[m][a:b], om[wi][m]) == 0
        del grads, s


def test_cfg2_tally_margins_match_the_oracle_and_the_vote():
    case = inputs.cfg2()
    d, M = case.d, case.M
    grads = inputs.gradients(case, DEV, 0)
    packed = [words_tensor(d, DEV) for _ in range(M)]
    for m in range(M):
        B.ss_sign_pack(grads[m], packed[m])
    del grads
    tally = torch.full((d,), 99, dtype=torch.int8, device=DEV)
    vote = words_tensor(d, DEV, fill=-1)
    B.ss_vote_tally(packed, d, case.flip_mask, tally)
    B.ss_majority_vote(packed, d, case.flip_mask, vote)
    assert torch.equal(tally >= 0, unpack_bits(vote, d))           # the vote is the tally's sign
    assert bool(((tally.int() + M) % 2 == 0).all()) and int(tally.abs().max()) <= M
    for a, b in windows(d, n_random=3, seed=2):
        _, want = oracle.majority_vote([to_np(p[a // 32:(b + 31) // 32]) for p in packed], b - a,
                                       case.flip_mask, return_tally=True)
        assert np.array_equal(tally[a:b].cpu().numpy().astype(np.int32), want)


@pytest.mark.parametrize("M,momentum", [(1, False), (3, True)])
def test_more_than_two_to_the_31_coordinates(M, momentum):
    """A single vector longer than 2^31 coordinates (64-bit indexing inside one buffer), ragged
    end included, on windows at the start, across the 2^31 and 2^32-byte marks, and at the end."""
    d = (1 << 31) + 100_000 + 8
    need = (M * (2 if momentum else 1) + 1) * d * 4 * 1.1
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip("not enough free device memory")
    gen = torch.Generator(device=DEV).manual_seed(31)
    grads = [torch.randn(d, generator=gen, device=DEV) for _ in range(M)]
    x = torch.randn(d, generator=gen, device=DEV)
    moms = [torch.randn(d, generator=gen, device=DEV) * 0.1 for _ in range(M)] if momentum else None
    wins = [(0, 1 << 16), ((1 << 30) - 4096, (1 << 30) + 4096), ((1 << 31) - 4096, (1 << 31) + 4096),
            (d - 70_000 - 8 - (d - 70_000 - 8) % 32, d)]
    ox = [to_np(x[a:b]) for a, b in wins]
    om = [[to_np(v[a:b]) for v in moms] if momentum else None for a, b in wins]
    vote = words_tensor(d, DEV, fill=-1)
    B.ss_fused_step(grads, moms, x, 0.9, 1e-3, 0.0, 0, vote)
    packed = [words_tensor(d, DEV, fill=-1) for _ in range(M)]
    for m in range(M):
        B.ss_sign_pack(grads[m], packed[m])
    torch.cuda.synchronize()
    for wi, (a, b) in enumerate(wins):
        g_np = [to_np(g[a:b]) for g in grads]
        want = oracle.fused_step(g_np, om[wi], ox[wi], 0.9, 1e-3)
        assert_words_equal(vote[a // 32:(b + 31) // 32], want, "vote words, window %d" % wi)
        assert count_bit_mismatch(x[a:b], ox[wi]) == 0
        if momentum:
            for m in range(M):
                assert count_bit_mismatch(moms[m][a:b], om[wi][m]) == 0
        assert_words_equal(packed[0][a // 32:(b + 31) // 32], oracle.sign_pack(g_np[0]), "pack, window %d" % wi)
    assert int(vote[-1].item()) & 0xFFFFFFFF & ~((1 << (d % 32)) - 1) == 0
