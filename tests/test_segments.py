"""Tensor fusion: one flat vector made of several tensors, each with its own learning rate and
weight decay (Section 4 merges small tensors into one buffer before compression).

The CPU half pins the oracle's per-tensor loop: equal hyper-parameters everywhere reduce to the
plain step, and a hand-worked two-tensor example. The GPU half checks ss_fused_step_segments and
ss_apply_vote_segments against that loop, with tensors that start at arbitrary coordinates (inside
quads and words), empty tensors, one tensor, and hundreds of small ones.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B


def _inputs(M, d, seed, momentum):
    rng = np.random.default_rng(seed)
    grads = [rng.standard_normal(d).astype(np.float32) for _ in range(M)]
    x = rng.standard_normal(d).astype(np.float32)
    moms = [rng.standard_normal(d).astype(np.float32) * 0.1 for _ in range(M)] if momentum else None
    return grads, moms, x


def _table(d, n, seed):
    rng = np.random.default_rng(seed)
    cuts = np.sort(rng.integers(1, max(2, d), size=n - 1)) if n > 1 else np.array([], dtype=np.int64)
    begins = [0] + [int(c) for c in cuts]
    lrs = [float(10.0 ** rng.uniform(-4, -2)) for _ in range(n)]
    wds = [0.0 if k % 3 == 0 else float(10.0 ** rng.uniform(-3, -1)) for k in range(n)]
    return begins, lrs, wds


# ---- CPU: the per-tensor loop ------------------------------------------------------------------

@pytest.mark.parametrize("momentum", [False, True])
def test_equal_hyperparameters_reduce_to_the_plain_step(momentum):
    M, d = 5, 1000
    g, v, x = _inputs(M, d, 1, momentum)
    v2 = [a.copy() for a in v] if momentum else None
    x2 = x.copy()
    vote_a = oracle.fused_step(g, v, x, 0.9, 1e-3, 0.01, 0b00100)
    vote_b = oracle.fused_step_segments(g, v2, x2, 0.9, [0, 17, 17, 640], [1e-3] * 4, [0.01] * 4, 0b00100)
    assert np.array_equal(vote_a, vote_b)
    assert np.array_equal(x.view(np.uint32), x2.view(np.uint32))
    if momentum:
        for a, b in zip(v, v2):
            assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_hand_worked_two_tensor_example():
    # M = 1, signSGD: tensor 0 = coordinates 0..2 with lr 0.5, no decay; tensor 1 = coordinates
    # 3..5 with lr 0.25 and weight decay 0.5. All values are exact binary fractions.
    g = [np.array([1.0, -2.0, 0.0, 3.0, -1.0, -4.0], dtype=np.float32)]
    x = np.array([1.0, 1.0, 1.0, 2.0, 2.0, -4.0], dtype=np.float32)
    vote = oracle.fused_step_segments(g, None, x, 0.0, [0, 3], [0.5, 0.25], [0.0, 0.5])
    assert vote.tolist() == [0b001101]
    # tensor 0: x - (+-0.5);  tensor 1: x - 0.25 * (s + 0.5 x)
    assert x.tolist() == [0.5, 1.5, 0.5, 2.0 - 0.25 * (1 + 1.0), 2.0 - 0.25 * (-1 + 1.0),
                          -4.0 - 0.25 * (-1 - 2.0)]


def test_upload_rejects_bad_tables_without_a_gpu():
    L = B.lib()
    fake = ctypes.c_void_p(0x1000)

    def status(begins, d):
        host = (B.ss_segment * len(begins))()
        for k, b in enumerate(begins):
            host[k].begin = b
        return L.ss_segments_upload(ctypes.cast(host, ctypes.c_void_p), len(begins), d, fake, None)

    assert status([1, 5], 10) == B.SS_ERR_INVALID_ARG        # first tensor must start at 0
    assert status([0, 7, 5], 10) == B.SS_ERR_INVALID_ARG     # begins must not decrease
    assert status([0, 11], 10) == B.SS_ERR_INVALID_ARG       # begin beyond d
    assert L.ss_segments_upload(None, 1, 10, fake, None) == B.SS_ERR_INVALID_ARG
    host = (B.ss_segment * 1)()
    assert L.ss_segments_upload(ctypes.cast(host, ctypes.c_void_p), 0, 10, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_segments_upload(ctypes.cast(host, ctypes.c_void_p), 1, 10, ctypes.c_void_p(0x1004), None) \
        == B.SS_ERR_MISALIGNED


# ---- GPU ---------------------------------------------------------------------------------------

DEV = "cuda:0"


def _to_dev(a):
    return torch.from_numpy(a.copy()).to(DEV)


@pytest.mark.gpu
@pytest.mark.parametrize("M,momentum", [(1, False), (3, False), (15, True), (6, True), (16, True)])
@pytest.mark.parametrize("d,n_seg", [(1, 1), (33, 2), (4097, 5), (100_003, 161), (262_184, 40), (70_000, 1)])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
def test_fused_step_segments_matches_per_tensor_steps(M, momentum, d, n_seg, misalign):
    g, v, x = _inputs(M, d, 10 * d + M, momentum)
    begins, lrs, wds = _table(d, n_seg, d + n_seg)
    if n_seg >= 5:
        begins[2] = begins[1]                      # an empty tensor
    flip = 0b10 if M > 2 else 0
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)

    def dev(a):                                     # optionally off the 16-byte grid
        t = torch.zeros(d + misalign, device=DEV)
        t[misalign:] = _to_dev(a)
        return t[misalign:]

    gd = [dev(a) for a in g]
    vd = [dev(a) for a in v] if momentum else None
    xd = dev(x)
    vote = torch.full((B.ss_packed_words(d),), -1, dtype=torch.int32, device=DEV)
    for step in range(2):
        B.ss_fused_step_segments(gd, vd, xd, 0.9, tab, n_seg, flip, vote)
        want = oracle.fused_step_segments(g, v, x, 0.9, begins, lrs, wds, flip)
        assert np.array_equal(vote.cpu().numpy().view(np.uint32), want), "vote, step %d" % step
        assert np.array_equal(xd.cpu().numpy().view(np.uint32), x.view(np.uint32)), "x, step %d" % step
        if momentum:
            for a, b in zip(vd, v):
                assert np.array_equal(a.cpu().numpy().view(np.uint32), b.view(np.uint32))


@pytest.mark.gpu
@pytest.mark.parametrize("M,momentum", [(3, False), (15, True), (6, True)])
@pytest.mark.parametrize("d,n_seg", [(4097, 5), (100_003, 161)])
def test_fused_step_segments_with_bf16_gradients(M, momentum, d, n_seg):
    """bf16 gradients on aligned pointers run kernels of their own (eight coordinates per thread);
    the per-tensor learning rates must reach both quads of every octet."""
    g32, v, x = _inputs(M, d, 20 * d + M, momentum)
    gd = [torch.from_numpy(a).to(DEV).to(torch.bfloat16) for a in g32]
    g = [t.cpu().view(torch.int16).numpy().view(np.uint16).copy() for t in gd]   # raw bf16 for the checker
    begins, lrs, wds = _table(d, n_seg, d + n_seg + 1)
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)
    vd = [_to_dev(a) for a in v] if momentum else None
    xd = _to_dev(x)
    vote = torch.full((B.ss_packed_words(d),), -1, dtype=torch.int32, device=DEV)
    for step in range(2):
        B.ss_fused_step_segments(gd, vd, xd, 0.9, tab, n_seg, 0b100, vote)
        want = oracle.fused_step_segments(g, v, x, 0.9, begins, lrs, wds, 0b100)
        assert np.array_equal(vote.cpu().numpy().view(np.uint32), want), "vote, step %d" % step
        assert np.array_equal(xd.cpu().numpy().view(np.uint32), x.view(np.uint32)), "x, step %d" % step
        if momentum:
            for a, b in zip(vd, v):
                assert np.array_equal(a.cpu().numpy().view(np.uint32), b.view(np.uint32))


@pytest.mark.gpu
@pytest.mark.parametrize("d,n_seg", [(1, 1), (127, 3), (100_003, 161)])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
def test_apply_vote_segments(d, n_seg, misalign):
    rng = np.random.default_rng(d)
    x = rng.standard_normal(d).astype(np.float32)
    vote = oracle.sign_pack(rng.standard_normal(d).astype(np.float32))
    begins, lrs, wds = _table(d, n_seg, 3 * d)
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)
    xt = torch.zeros(d + misalign, device=DEV)
    xt[misalign:] = _to_dev(x)
    xd = xt[misalign:]
    B.ss_apply_vote_segments(xd, torch.from_numpy(vote.view(np.int32).copy()).to(DEV), tab, n_seg)
    want = x.copy()                                 # the oracle's apply, tensor by tensor
    for k in range(n_seg):
        a, b = begins[k], begins[k + 1] if k + 1 < n_seg else d
        if b > a:
            bits = oracle.unpack(vote, d)[a:b]
            sub_vote = oracle.sign_pack(bits.astype(np.float32))
            oracle.apply_vote(want[a:b], sub_vote, lrs[k], wds[k])
    assert np.array_equal(xd.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.gpu
@pytest.mark.parametrize("M", [1, 7, 12])
@pytest.mark.parametrize("d,n_seg", [(3, 2), (1027, 4), (100_003, 161)])
@pytest.mark.parametrize("misalign", [0, 1], ids=["aligned", "unaligned"])
def test_vote_apply_segments(M, d, n_seg, misalign):
    rng = np.random.default_rng(d + M)
    W = B.ss_packed_words(d)
    packed_np = [rng.integers(0, 1 << 32, size=W, dtype=np.uint64).astype(np.uint32) for _ in range(M)]
    packed = [torch.from_numpy(p.view(np.int32).copy()).to(DEV) for p in packed_np]
    x = rng.standard_normal(d).astype(np.float32)
    begins, lrs, wds = _table(d, n_seg, 5 * d + M)
    tab = B.segment_table(n_seg, DEV)
    B.ss_segments_upload(begins, lrs, wds, d, tab)
    xt = torch.zeros(d + misalign, device=DEV)
    xt[misalign:] = _to_dev(x)
    xd = xt[misalign:]
    vote_out = torch.full((W,), -1, dtype=torch.int32, device=DEV)
    flip = 0b100 if M > 2 else 0
    B.ss_vote_apply_segments(packed, xd, tab, n_seg, flip, vote_out)
    vote = oracle.majority_vote(packed_np, d, flip)
    bits = oracle.unpack(vote, d)
    want = x.copy()
    for k in range(n_seg):
        a, b = begins[k], begins[k + 1] if k + 1 < n_seg else d
        if b > a:
            oracle.apply_vote(want[a:b], oracle.sign_pack(bits[a:b].astype(np.float32)), lrs[k], wds[k])
    assert np.array_equal(vote_out.cpu().numpy().view(np.uint32), vote)
    assert np.array_equal(xd.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.gpu
def test_flat_layout_front_end_runs_a_model_shaped_step():
    from paper_1810_05291_b200.fusion import FlatLayout
    shapes = [(64, 3, 7, 7), (64,), (64,), (128, 64, 3, 3), (128,), (1000, 128), (1000,)]
    lrs = [1e-3 if len(s) > 1 else 2e-3 for s in shapes]
    wds = [5e-4 if len(s) > 1 else 0.0 for s in shapes]
    lay = FlatLayout(shapes, lrs, wds, DEV, align=4)
    M = 7
    gen = torch.Generator(device=DEV).manual_seed(5)
    x = torch.randn(lay.d, generator=gen, device=DEV)
    grads = [torch.randn(lay.d, generator=gen, device=DEV) for _ in range(M)]
    moms = [lay.flat() for _ in range(M)]
    x_np = x.cpu().numpy().copy()
    g_np = [t.cpu().numpy().copy() for t in grads]
    m_np = [np.zeros(lay.d, dtype=np.float32) for _ in range(M)]
    views = lay.views(x)
    assert [tuple(v.shape) for v in views] == [tuple(s) for s in shapes]
    assert views[3].data_ptr() == x.data_ptr() + 4 * lay.begins[3]
    vote = torch.zeros(B.ss_packed_words(lay.d), dtype=torch.int32, device=DEV)
    for _ in range(3):
        lay.step(grads, moms, x, 0.9, 0, vote)
        want = oracle.fused_step_segments(g_np, m_np, x_np, 0.9, lay.begins, lrs, wds)
        assert np.array_equal(vote.cpu().numpy().view(np.uint32), want)
        assert np.array_equal(x.cpu().numpy().view(np.uint32), x_np.view(np.uint32))
    lay.set_hyperparameters([v * 0.1 for v in lrs], wds)
    lay.step(grads, moms, x, 0.9)
    oracle.fused_step_segments(g_np, m_np, x_np, 0.9, lay.begins, [v * 0.1 for v in lrs], wds)
    assert np.array_equal(x.cpu().numpy().view(np.uint32), x_np.view(np.uint32))
