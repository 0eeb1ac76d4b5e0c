"""Parity of the CUDA library with the CPU oracle, element by element, through the C ABI.

Packed words and vote words must be bit-exact. fp32 momentum and parameters must agree within
1e-6 relative per element (they are in fact expected to be bit-identical, which is reported
and asserted separately, because both sides run the same sequence of rounded operations)."""
import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B
from paper_1810_05291_b200 import inputs
from tests import golden_io
from tests.util import (GuardedWords, assert_f32_close, assert_words_equal, check_guard,
                        count_bit_mismatch, guarded_f32, to_np, words_tensor)

pytestmark = pytest.mark.gpu

GOLD = golden_io.load()
DEV = "cuda:0"

AWKWARD_D = [1, 31, 32, 33, 127, 128, 4097, 100_003, 262_144 + 40]
ALL_M = [1, 2, 3, 4, 5, 7, 8, 15, 16, 31, 63, 64]


@pytest.fixture(scope="module", autouse=True)
def _oracle_threads():
    oracle.set_threads(min(16, oracle.max_threads()))
    yield
    oracle.set_threads(1)


def _rand(d, seed, dtype=torch.float32, specials=True):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    g = torch.randn(d, generator=gen, device=DEV)
    if specials and d >= 16:
        idx = torch.randint(0, d, (max(1, d // 9),), generator=gen, device=DEV)
        vals = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 1e-42, -1e-42, 1e-30],
                            device=DEV)
        g[idx] = vals[torch.randint(0, len(vals), (idx.numel(),), generator=gen, device=DEV)]
    return g.to(dtype).contiguous()


# ---- hand vectors through the C ABI ---------------------------------------------------------

@pytest.mark.parametrize("rec", GOLD["pack"], ids=lambda r: "%s-d%d" % (r[0], len(r[1])))
def test_pack_hand_vectors(rec):
    kind, arr, want = rec
    if kind == "f32":
        g = torch.from_numpy(arr.copy()).to(DEV)
    else:
        g = torch.from_numpy(arr.view(np.int16).copy()).to(DEV).view(torch.bfloat16)
    out = words_tensor(g.numel(), DEV, fill=-1)
    B.ss_sign_pack(g, out)
    assert_words_equal(out, want)


@pytest.mark.parametrize("rec", GOLD["vote"], ids=lambda r: "d%d-M%d-f%x" % (r[0], len(r[2]), r[1]))
def test_vote_hand_vectors(rec):
    d, flip, workers, want = rec
    packed = [torch.from_numpy(w.view(np.int32).copy()).to(DEV) for w in workers]
    out = words_tensor(d, DEV, fill=-1)
    B.ss_majority_vote(packed, d, flip, out)
    assert_words_equal(out, want)


@pytest.mark.parametrize("rec", GOLD["momentum"])
def test_momentum_hand_vectors(rec):
    beta, g, v0, v1, bit = rec
    gt = torch.tensor([g], device=DEV)
    vt = torch.tensor([v0], device=DEV)
    out = words_tensor(1, DEV, fill=-1)
    B.ss_signum_update(gt, vt, beta, out)
    assert vt.item() == v1
    assert out.item() == bit


@pytest.mark.parametrize("rec", GOLD["apply"])
def test_apply_hand_vectors(rec):
    x0, bit, lr, wd, x1 = rec
    x = torch.tensor([x0], device=DEV)
    B.ss_apply_vote(x, torch.tensor([bit], dtype=torch.int32, device=DEV), lr, wd)
    assert x.item() == x1


# ---- per-kernel parity on awkward shapes -----------------------------------------------------

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [0, 1, 4], ids=["aligned", "unaligned", "off-by-4-elements"])
@pytest.mark.parametrize("d", AWKWARD_D + [32 * 4096 + 8, 1_000_000])
def test_sign_pack(d, misalign, dtype):
    g = _rand(d + misalign, 100 + d, dtype)[misalign:]
    out = GuardedWords(d, DEV, misalign_words=misalign)
    B.ss_sign_pack(g, out.view)
    assert_words_equal(out.view, oracle.sign_pack(to_np(g)))
    out.check()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [0, 1, 4], ids=["aligned", "unaligned", "off-by-4-elements"])
@pytest.mark.parametrize("d", AWKWARD_D)
def test_signum_update(d, misalign, dtype):
    g = _rand(d + misalign, 200 + d, dtype)[misalign:]
    v_src = _rand(d, 300 + d, specials=False)
    full, v, lo = guarded_f32(v_src, misalign)
    v_np = to_np(v)
    g_np = to_np(g)
    out = GuardedWords(d, DEV)
    for step in range(3):
        B.ss_signum_update(g, v, 0.9, out.view)
        want = oracle.signum_update(g_np, v_np, 0.9)
        assert_words_equal(out.view, want, "packed sign(v) step %d" % step)
        assert_f32_close(v, v_np, "momentum step %d" % step)
        assert count_bit_mismatch(v, v_np) == 0
    out.check()
    check_guard(full, lo, d)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("n_dests", [1, 3, 8])
@pytest.mark.parametrize("d", [1, 33, 4097, 100_003, 32 * 4096 + 8])
def test_signum_update_push(d, n_dests, misalign, dtype):
    g = _rand(d + misalign, 210 + d, dtype)[misalign:]
    full, v, lo = guarded_f32(_rand(d, 310 + d, specials=False), misalign)
    v_np, g_np = to_np(v), to_np(g)
    outs = [GuardedWords(d, DEV) for _ in range(n_dests)]
    for step in range(2):
        B.ss_signum_update_push(g, v, 0.9, [o.view for o in outs])
        want = oracle.signum_update(g_np, v_np, 0.9)
        for o in outs:
            assert_words_equal(o.view, want, "pushed words step %d" % step)
            o.check()
        assert count_bit_mismatch(v, v_np) == 0
    check_guard(full, lo, d)


@pytest.mark.parametrize("M", ALL_M)
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("d", [1, 33, 127, 128, 4097, 100_003])
def test_majority_vote(d, misalign, M):
    W = B.ss_packed_words(d)
    gen = torch.Generator(device=DEV).manual_seed(17 * d + M)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W + misalign,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32)[misalign:] for _ in range(M)]
    flip = int(torch.randint(0, 1 << 30, (1,), generator=gen, device=DEV).item()) & ((1 << M) - 1)
    for f in (0, flip):
        out = GuardedWords(d, DEV, misalign_words=misalign)
        B.ss_majority_vote(packed, d, f, out.view)
        assert_words_equal(out.view, oracle.majority_vote([to_np(p) for p in packed], d, f))
        out.check()


@pytest.mark.parametrize("M", ALL_M)
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("d", [1, 3, 33, 127, 1023, 1027, 4097, 100_003])
def test_vote_tally(d, misalign, M):
    W = B.ss_packed_words(d)
    gen = torch.Generator(device=DEV).manual_seed(29 * d + M)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32) for _ in range(M)]
    flip = int(torch.randint(0, 1 << 30, (1,), generator=gen, device=DEV).item()) & ((1 << M) - 1)
    pad = 64
    full = torch.full((d + 2 * pad + misalign,), 99, dtype=torch.int8, device=DEV)
    out = full[pad + misalign: pad + misalign + d]
    for f in (0, flip):
        B.ss_vote_tally(packed, d, f, out)
        vote, tally = oracle.majority_vote([to_np(p) for p in packed], d, f, return_tally=True)
        got = out.cpu().numpy().astype(np.int32)
        assert np.array_equal(got, tally)
        assert bool((full[: pad + misalign] == 99).all()) and bool((full[pad + misalign + d:] == 99).all())
        # the packed vote is the sign of the tally
        words = words_tensor(d, DEV, fill=-1)
        B.ss_majority_vote(packed, d, f, words)
        assert_words_equal(words, oracle.sign_pack(tally.astype(np.float32)))


@pytest.mark.parametrize("wd", [0.0, 0.01])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("d", AWKWARD_D)
def test_apply_vote(d, misalign, wd):
    x_src = _rand(d, 400 + d, specials=False)
    full, x, lo = guarded_f32(x_src, misalign)
    vote = oracle.sign_pack(to_np(_rand(d, 500 + d, specials=False)))
    vt = torch.from_numpy(vote.view(np.int32).copy()).to(DEV)
    x_np = to_np(x)
    B.ss_apply_vote(x, vt, 1e-3, wd)
    oracle.apply_vote(x_np, vote, 1e-3, wd)
    assert_f32_close(x, x_np, "parameters")
    assert count_bit_mismatch(x, x_np) == 0
    check_guard(full, lo, d)


@pytest.mark.parametrize("M", ALL_M)
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
@pytest.mark.parametrize("d", [1, 3, 33, 127, 1023, 1024, 1027, 4097, 100_003])
def test_vote_apply(d, misalign, M):
    W = B.ss_packed_words(d)
    gen = torch.Generator(device=DEV).manual_seed(23 * d + M)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W + misalign,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32)[misalign:] for _ in range(M)]
    flip = int(torch.randint(0, 1 << 30, (1,), generator=gen, device=DEV).item()) & ((1 << M) - 1)
    packed_np = [to_np(p) for p in packed]
    for f, wd, want_words in ((0, 0.0, True), (flip, 0.02, True), (flip, 0.0, False)):
        full, x, lo = guarded_f32(_rand(d, 600 + d + M, specials=False), misalign)
        x_np = to_np(x)
        out = GuardedWords(d, DEV, misalign_words=misalign)
        B.ss_vote_apply(packed, x, 1e-3, wd, f, out.view if want_words else None)
        vote = oracle.majority_vote(packed_np, d, f)
        oracle.apply_vote(x_np, vote, 1e-3, wd)
        if want_words:
            assert_words_equal(out.view, vote)
        out.check()
        assert_f32_close(x, x_np, "parameters")
        assert count_bit_mismatch(x, x_np) == 0
        check_guard(full, lo, d)


@pytest.mark.parametrize("M", [2, 6, 9, 14, 17, 27, 30, 33, 62])
def test_vote_and_vote_apply_for_worker_counts_between_the_compiled_ones(M):
    """Worker counts that have no kernel of their own run the next larger compiled capacity with
    the absent workers switched off: vote, tally sign and parameters against the oracle."""
    d = 64 * 32 * 5 + 32 * 3 + 5                       # full 64-word tiles, then a ragged end
    W = B.ss_packed_words(d)
    gen = torch.Generator(device=DEV).manual_seed(1000 + M)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32) for _ in range(M)]
    packed_np = [to_np(p) for p in packed]
    flip = (0x5A5A5A5A5A5A5A5A >> 3) & ((1 << M) - 1)
    want = oracle.majority_vote(packed_np, d, flip)
    out = GuardedWords(d, DEV)
    B.ss_majority_vote(packed, d, flip, out.view)
    assert_words_equal(out.view, want, "ss_majority_vote")
    out.check()
    full, x, lo = guarded_f32(_rand(d, 900 + M, specials=False), 0)
    x_np = to_np(x)
    oracle.apply_vote(x_np, want, 1e-3, 0.01)
    out2 = GuardedWords(d, DEV)
    B.ss_vote_apply(packed, x, 1e-3, 0.01, flip, out2.view)
    assert_words_equal(out2.view, want, "ss_vote_apply")
    out2.check()
    assert count_bit_mismatch(x, x_np) == 0
    check_guard(full, lo, d)


@pytest.mark.parametrize("M", [3, 15, 20, 64])
@pytest.mark.parametrize("packed_off,vote_off", [(2, 0), (0, 2), (1, 0), (0, 1), (2, 2), (3, 1)])
def test_vote_apply_with_packed_words_off_the_16_byte_grid(M, packed_off, vote_off):
    """The parameters 16-byte aligned, the packed inputs or the vote output shifted by whole
    words: 8-byte shifts keep the 64-bit loads, odd shifts take the word-at-a-time kernel."""
    d = 64 * 32 * 7 + 32 * 40 + 9
    W = B.ss_packed_words(d)
    gen = torch.Generator(device=DEV).manual_seed(2000 + M + packed_off)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W + packed_off,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32)[packed_off:] for _ in range(M)]
    packed_np = [to_np(p) for p in packed]
    flip = 0b101 & ((1 << M) - 1)
    want = oracle.majority_vote(packed_np, d, flip)
    full, x, lo = guarded_f32(_rand(d, 950 + M, specials=False), 0)
    x_np = to_np(x)
    oracle.apply_vote(x_np, want, 1e-3, 0.0)
    out = GuardedWords(d, DEV, misalign_words=vote_off)
    B.ss_vote_apply(packed, x, 1e-3, 0.0, flip, out.view)
    assert_words_equal(out.view, want)
    out.check()
    assert count_bit_mismatch(x, x_np) == 0
    check_guard(full, lo, d)


def test_vote_apply_equals_vote_then_apply_on_the_gpu():
    M, d = 15, 32 * 40_000 + 8
    gen = torch.Generator(device=DEV).manual_seed(77)
    W = B.ss_packed_words(d)
    packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV,
                            dtype=torch.int64).to(torch.int32) for _ in range(M)]
    xa = _rand(d, 78, specials=False)
    xb = xa.clone()
    va, vb = words_tensor(d, DEV, fill=-1), words_tensor(d, DEV, fill=-1)
    B.ss_vote_apply(packed, xa, 1e-4, 0.0, 0b101, va)
    B.ss_majority_vote(packed, d, 0b101, vb)
    B.ss_apply_vote(xb, vb, 1e-4, 0.0)
    assert torch.equal(va, vb)
    assert torch.equal(xa.view(torch.int32), xb.view(torch.int32))


# ---- the fused step ---------------------------------------------------------------------------

def _fused_case(M, d, dtype, momentum, flip, wd, misalign, steps=2, seed=0):
    grads_all = [[_rand(d + misalign, seed + 1000 * s + m, dtype)[misalign:] for m in range(M)]
                 for s in range(steps)]
    xf, x, xlo = guarded_f32(_rand(d, seed + 7, specials=False), misalign)
    moms = mom_guards = None
    if momentum:
        mom_guards = [guarded_f32(_rand(d, seed + 50 + m, specials=False), misalign) for m in range(M)]
        moms = [t[1] for t in mom_guards]
    x_np = to_np(x)
    moms_np = [to_np(v) for v in moms] if momentum else None
    for s in range(steps):
        out = GuardedWords(d, DEV)
        B.ss_fused_step(grads_all[s], moms, x, 0.9, 1e-3, wd, flip, out.view)
        want = oracle.fused_step([to_np(g) for g in grads_all[s]], moms_np, x_np, 0.9, 1e-3, wd, flip)
        assert_words_equal(out.view, want, "vote step %d" % s)
        assert_f32_close(x, x_np, "parameters step %d" % s)
        assert count_bit_mismatch(x, x_np) == 0
        if momentum:
            for m in range(M):
                assert_f32_close(moms[m], moms_np[m], "momentum[%d] step %d" % (m, s))
                assert count_bit_mismatch(moms[m], moms_np[m]) == 0
        out.check()
    check_guard(xf, xlo, d)
    if momentum:
        for full, _, lo in mom_guards:
            check_guard(full, lo, d)


@pytest.mark.parametrize("momentum", [False, True], ids=["signsgd", "signum"])
@pytest.mark.parametrize("M", ALL_M)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_fused_step_all_worker_counts(M, momentum, dtype):
    flip = (0x5A5A5A5A5A5A5A5A if M > 2 else 0) & ((1 << M) - 1)
    if M % 2 == 1 and bin(flip).count("1") * 2 > M:
        flip = 0
    _fused_case(M, 32 * 1024 * 3 + 8, dtype, momentum, flip, 0.0, 0, seed=M * 31)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("misalign", [0, 1, 4], ids=["aligned", "unaligned", "off-by-4-elements"])
@pytest.mark.parametrize("d", AWKWARD_D)
@pytest.mark.parametrize("M,momentum", [(3, False), (15, True), (6, True)])
def test_fused_step_awkward_shapes(d, misalign, dtype, M, momentum):
    _fused_case(M, d, dtype, momentum, 1 if M > 2 else 0, 0.0, misalign, seed=d + M)


@pytest.mark.parametrize("M,momentum", [(7, False), (15, True)])
def test_fused_step_weight_decay(M, momentum):
    _fused_case(M, 70_001, torch.float32, momentum, 0, 0.05, 0, steps=3, seed=99)


def test_fused_step_without_vote_output():
    M, d = 7, 50_000
    grads = [_rand(d, 3000 + m) for m in range(M)]
    x = _rand(d, 3100, specials=False)
    x2 = x.clone()
    out = words_tensor(d, DEV)
    B.ss_fused_step(grads, None, x, 0.0, 1e-3, 0.0, 0, out)
    B.ss_fused_step(grads, None, x2, 0.0, 1e-3, 0.0, 0, None)
    assert torch.equal(x, x2)


@pytest.mark.parametrize("M,momentum,dtype", [(3, False, torch.float32), (15, True, torch.float32),
                                              (16, True, torch.bfloat16), (5, True, torch.float32)])
def test_fused_equals_unfused_chain_on_the_gpu(M, momentum, dtype):
    d = 32 * 5000 + 8
    flip = 1 if M > 2 else 0
    grads = [_rand(d, 4000 + m, dtype) for m in range(M)]
    x_f = _rand(d, 4100, specials=False)
    x_u = x_f.clone()
    mom_f = [_rand(d, 4200 + m, specials=False) for m in range(M)] if momentum else None
    mom_u = [v.clone() for v in mom_f] if momentum else None
    vote_f, vote_u = words_tensor(d, DEV), words_tensor(d, DEV)
    B.ss_fused_step(grads, mom_f, x_f, 0.9, 1e-3, 0.0, flip, vote_f)
    packed = [words_tensor(d, DEV) for _ in range(M)]
    for m in range(M):
        if momentum:
            B.ss_signum_update(grads[m], mom_u[m], 0.9, packed[m])
        else:
            B.ss_sign_pack(grads[m], packed[m])
    B.ss_majority_vote(packed, d, flip, vote_u)
    B.ss_apply_vote(x_u, vote_u, 1e-3, 0.0)
    assert torch.equal(vote_f, vote_u)
    assert torch.equal(x_f.view(torch.int32), x_u.view(torch.int32))
    if momentum:
        for a, b in zip(mom_f, mom_u):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_beta_zero_equals_sign_pack():
    d = 100_000
    g = _rand(d, 5000)
    v = _rand(d, 5001, specials=False)
    a, b = words_tensor(d, DEV), words_tensor(d, DEV)
    B.ss_signum_update(g, v, 0.0, a)
    B.ss_sign_pack(g, b)
    assert torch.equal(a, b)
    fin = ~torch.isnan(g)
    assert torch.equal(v[fin], g[fin])


def test_empty_input_is_a_no_op():
    g = torch.zeros(0, device=DEV)
    out = torch.zeros(0, dtype=torch.int32, device=DEV)
    B.ss_sign_pack(g, out)
    B.ss_apply_vote(g, out, 0.1)
    B.ss_fused_step([g], None, g, 0.0, 0.1, 0.0, 0, out)
    torch.cuda.synchronize()


def test_poisoned_worker_cannot_corrupt_parameters():
    M, d = 3, 40_000
    grads = [_rand(d, 6000 + m, specials=False) for m in range(M)]
    grads[1].fill_(float("inf"))
    grads[1][::2] = float("nan")
    moms = [torch.zeros(d, device=DEV) for _ in range(M)]
    x = _rand(d, 6100, specials=False)
    x0 = x.clone()
    for _ in range(3):
        B.ss_fused_step(grads, moms, x, 0.9, 1e-2)
    assert bool(torch.isfinite(x).all())
    assert bool(((x - x0).abs() <= 3e-2 * 1.0001).all())


def test_runs_on_a_non_default_stream():
    d, M = 300_000, 7
    grads = [_rand(d, 7000 + m) for m in range(M)]
    x = _rand(d, 7100, specials=False)
    x_np = to_np(x)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    out = words_tensor(d, DEV)
    with torch.cuda.stream(s):
        B.ss_fused_step(grads, None, x, 0.0, 1e-3, 0.0, 0, out)
    s.synchronize()
    want = oracle.fused_step([to_np(g) for g in grads], None, x_np, 0.0, 1e-3)
    assert_words_equal(out, want)
    assert count_bit_mismatch(x, x_np) == 0


def test_host_entry_point_matches_device_entry_point():
    M, d = 7, 200_000 + 8
    case = inputs.cfg3(d)
    case.M = M
    grads = inputs.gradients(case, DEV, 0)
    host = [g.cpu().pin_memory() for g in grads]
    staging = [torch.empty_like(g) for g in grads]
    x1, x2 = inputs.initial_params(case, DEV), inputs.initial_params(case, DEV)
    m1 = [torch.zeros(d, device=DEV) for _ in range(M)]
    m2 = [torch.zeros(d, device=DEV) for _ in range(M)]
    v1, v2 = words_tensor(d, DEV), words_tensor(d, DEV)
    hv = torch.zeros(B.ss_packed_words(d), dtype=torch.int32).pin_memory()
    B.ss_fused_step(grads, m1, x1, 0.9, 1e-4, 0.0, 0, v1)
    B.ss_fused_step_host(host, staging, m2, x2, 0.9, 1e-4, 0.0, 0, v2, hv)
    torch.cuda.synchronize()
    assert torch.equal(v1, v2) and torch.equal(v1.cpu(), hv)
    assert torch.equal(x1, x2)
    for a, b in zip(m1, m2):
        assert torch.equal(a, b)


def test_unfused_chain_replays_from_a_cuda_graph():
    """The kernels only enqueue work on the caller's stream, so a whole iteration of the unfused
    chain can be recorded once into a CUDA graph and replayed; the replays must give what the
    same calls give when issued one by one."""
    M, d = 7, 32 * 20_000 + 8
    grads = [_rand(d, 8000 + m, specials=False) for m in range(M)]
    x_e = _rand(d, 8100, specials=False)
    x_g = x_e.clone()
    mom_e = [torch.zeros(d, device=DEV) for _ in range(M)]
    mom_g = [torch.zeros(d, device=DEV) for _ in range(M)]
    packed = [words_tensor(d, DEV) for _ in range(M)]
    vote_e, vote_g = words_tensor(d, DEV), words_tensor(d, DEV)

    def chain(moms, x, vote):
        for m in range(M):
            B.ss_signum_update(grads[m], moms[m], 0.9, packed[m])
        B.ss_vote_apply(packed, x, 1e-3, 0.0, 0b10, vote)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            chain(mom_g, x_g, vote_g)
    torch.cuda.current_stream().wait_stream(side)
    # capture does not run the work: the graph's buffers are still untouched
    assert torch.equal(x_g, x_e)
    for step in range(3):
        graph.replay()
        chain(mom_e, x_e, vote_e)
        torch.cuda.synchronize()
        assert torch.equal(vote_g, vote_e)
        assert torch.equal(x_g.view(torch.int32), x_e.view(torch.int32))
        for a, b in zip(mom_g, mom_e):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("flip,wd", [(0, 0.0), (1, 0.0), (0, 0.05), (1, 0.05)])
@pytest.mark.parametrize("d,misalign", [(1, 0), (33, 0), (4097, 0), (4097, 1), (100_003, 0), (32 * 4096 + 8, 0)])
def test_single_worker_signsgd_step(d, misalign, flip, wd, dtype):
    """M = 1 without momentum (Theorem 1's update) has a kernel of its own."""
    _fused_case(1, d, dtype, False, flip, wd, misalign, steps=2, seed=900 + d)
    g = _rand(d, 950 + d, dtype)
    xa = _rand(d, 951 + d, specials=False)
    xb = xa.clone()
    B.ss_fused_step([g], None, xa, 0.0, 1e-3, wd, flip, words_tensor(d, DEV))
    B.ss_fused_step([g], None, xb, 0.0, 1e-3, wd, flip, None)       # without the packed output
    assert torch.equal(xa.view(torch.int32), xb.view(torch.int32))


@pytest.mark.parametrize("threads,blocks_per_sm", [(128, 0), (64, 1), (256, 2), (192, 3)])
def test_results_do_not_depend_on_the_launch_shape(threads, blocks_per_sm):
    """Block size and the persistent-grid option change only how the tiles are walked."""
    try:
        B.ss_set_launch_option("threads", threads)
        B.ss_set_launch_option("blocks_per_sm", blocks_per_sm)
        d = 148 * 3 * 256 * 4 * 5 + 32 * 7 + 8       # several grid-stride rounds and a ragged word
        _fused_case(15, d, torch.float32, True, 0b100, 0.0, 0, steps=1, seed=1234)
        _fused_case(7, d, torch.bfloat16, False, 0, 0.01, 0, steps=1, seed=1235)
        _fused_case(1, d, torch.float32, False, 0, 0.0, 0, steps=1, seed=1236)
        _fused_case(5, 100_003, torch.float32, True, 0, 0.0, 1, steps=1, seed=1237)
        g = _rand(d, 1238, torch.bfloat16)
        out = words_tensor(d, DEV, fill=-1)
        B.ss_sign_pack(g, out)
        assert_words_equal(out, oracle.sign_pack(to_np(g)))
        W = B.ss_packed_words(d)
        gen = torch.Generator(device=DEV).manual_seed(1239)
        packed = [torch.randint(-(1 << 31), 1 << 31, (W,), generator=gen, device=DEV,
                                dtype=torch.int64).to(torch.int32) for _ in range(7)]
        x = _rand(d, 1240, specials=False)
        x_np = to_np(x)
        vote = words_tensor(d, DEV, fill=-1)
        B.ss_vote_apply(packed, x, 1e-3, 0.0, 0b1, vote)
        want = oracle.majority_vote([to_np(p) for p in packed], d, 0b1)
        oracle.apply_vote(x_np, want, 1e-3, 0.0)
        assert_words_equal(vote, want)
        assert count_bit_mismatch(x, x_np) == 0
        tally = torch.zeros(d, dtype=torch.int8, device=DEV)
        B.ss_vote_tally(packed, d, 0b1, tally)
        assert np.array_equal(tally.cpu().numpy().astype(np.int32),
                              oracle.majority_vote([to_np(p) for p in packed], d, 0b1, return_tally=True)[1])
    finally:
        B.ss_set_launch_option("threads", 0)
        B.ss_set_launch_option("blocks_per_sm", 0)


@pytest.mark.parametrize("from_mib", [1, 1 << 20], ids=["plain-gradient-loads", "evict-first-gradient-loads"])
def test_results_do_not_depend_on_the_gradient_load_policy(from_mib):
    """The unrolled kernels without momentum exist twice, with plain and with evict-first gradient
    loads, chosen by the size of the call; the option forces either one at a size the oracle can check."""
    try:
        B.ss_set_launch_option("plain_loads_from_mib", from_mib)
        d = 32 * 4096 * 9 + 8                                  # 4.7 MB per fp32 worker
        for M in (1, 3, 7, 15, 16):
            _fused_case(M, d, torch.float32, False, 0b1 if M > 2 else 0, 0.0, 0, steps=1, seed=4000 + M)
        _fused_case(7, d, torch.bfloat16, False, 0, 0.0, 4, steps=1, seed=4100)    # 8-byte aligned bf16: quad form
        _fused_case(15, d, torch.bfloat16, False, 0, 0.02, 0, steps=1, seed=4101)  # octet form
        _fused_case(15, d, torch.float32, True, 0, 0.0, 0, steps=1, seed=4102)     # momentum: unaffected
    finally:
        B.ss_set_launch_option("plain_loads_from_mib", 0)


def test_two_streams_run_independent_steps_side_by_side():
    """The library keeps no state between calls, so steps on different streams and buffers may
    overlap on the GPU."""
    M, d = 7, 32 * 60_000 + 8
    sets = []
    for k in range(2):
        grads = [_rand(d, 9000 + 10 * k + m, specials=False) for m in range(M)]
        x = _rand(d, 9100 + k, specials=False)
        moms = [torch.zeros(d, device=DEV) for _ in range(M)]
        sets.append((grads, moms, x, words_tensor(d, DEV), to_np(x), [np.zeros(d, dtype=np.float32) for _ in range(M)]))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for s in streams:
        s.wait_stream(torch.cuda.current_stream())
    for step in range(4):
        for k, s in enumerate(streams):
            grads, moms, x, vote, _, _ = sets[k]
            with torch.cuda.stream(s):
                B.ss_fused_step(grads, moms, x, 0.9, 1e-3, 0.0, 0, vote)
    torch.cuda.synchronize()
    for grads, moms, x, vote, x_np, m_np in sets:
        g_np = [to_np(g) for g in grads]
        for step in range(4):
            want = oracle.fused_step(g_np, m_np, x_np, 0.9, 1e-3)
        assert_words_equal(vote, want)
        assert count_bit_mismatch(x, x_np) == 0
