"""The allocation-free host step, ss_fused_step_host_static, against ss_fused_step_host.

Some users of the library may not allocate device memory when they need a step (the device has
been given to a framework's allocator, or their rules forbid allocating after start-up), so they
cannot pass staging buffers. The static variant stages the gradients in a fixed array inside the
library. This file checks, through the C ABI, that it gives the same packed vote, parameters and
momenta as the entry point with caller-provided staging, on two calls in a row that reuse the
shared array with different shapes, and that requests beyond the fixed size are refused.
The file name sorts last so that a run that stops at the first failure has already run the rest.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_1810_05291_b200 import binding as B
from paper_1810_05291_b200 import inputs
from tests.util import assert_f32_close, assert_words_equal, count_bit_mismatch, to_np

DEV = "cuda:0"


def _run_pair(M, d, dtype, momentum, flip, step):
    case = inputs.cfg3(d)
    case.M, case.dtype = M, dtype
    grads = inputs.gradients(case, DEV, step)
    host = [g.cpu().pin_memory() for g in grads]
    W = B.ss_packed_words(d)
    outs = []
    for static in (False, True):
        x = inputs.initial_params(case, DEV)
        moms = [torch.full((d,), 0.01 * (m + 1), device=DEV) for m in range(M)] if momentum else None
        vote = torch.full((W,), -1, dtype=torch.int32, device=DEV)
        hv = torch.full((W,), -1, dtype=torch.int32).pin_memory()
        if static:
            B.ss_fused_step_host_static(host, moms, x, 0.9, 1e-4, 0.0, flip, vote, hv)
        else:
            staging = [torch.empty_like(g) for g in grads]
            B.ss_fused_step_host(host, staging, moms, x, 0.9, 1e-4, 0.0, flip, vote, hv)
        torch.cuda.synchronize()
        outs.append((x, moms, vote, hv))
    (x1, m1, v1, h1), (x2, m2, v2, h2) = outs
    assert torch.equal(v1, v2), "packed vote differs"
    assert torch.equal(h1, h2) and torch.equal(h2, v2.cpu()), "vote copied to the host differs"
    assert_f32_close(x2, to_np(x1), "parameters")
    assert torch.equal(x1, x2)
    if momentum:
        for a, b in zip(m1, m2):
            assert_f32_close(b, to_np(a), "momentum")
            assert torch.equal(a, b)


@pytest.mark.gpu
def test_static_staging_matches_caller_staging_on_two_calls_in_a_row():
    # first call: larger shape; second call: fewer workers, shorter and ragged vectors, bf16, an
    # inverting worker -- whatever the first call left in the shared array must not leak in
    _run_pair(M=15, d=32 * 9000 + 8, dtype=torch.float32, momentum=True, flip=0, step=0)
    _run_pair(M=7, d=100_003, dtype=torch.bfloat16, momentum=True, flip=0x10, step=1)
    _run_pair(M=3, d=4097, dtype=torch.float32, momentum=False, flip=0, step=2)


def _run_against_the_checker(M, d, dtype, flip, step, x, moms, x_np, moms_np):
    """One static-staging step on the device and the same step in the CPU checker, compared
    element by element: packed vote (on the device and as copied to the host), parameters, momenta."""
    case = inputs.cfg3(d)
    case.M, case.dtype = M, dtype
    grads = inputs.gradients(case, DEV, step)
    host = [g.cpu().pin_memory() for g in grads]
    W = B.ss_packed_words(d)
    vote = torch.full((W,), -1, dtype=torch.int32, device=DEV)
    hv = torch.full((W,), -1, dtype=torch.int32).pin_memory()
    B.ss_fused_step_host_static(host, moms, x, 0.9, 1e-4, 0.0, flip, vote, hv)
    torch.cuda.synchronize()
    want = oracle.fused_step([to_np(g) for g in grads], moms_np, x_np, 0.9, 1e-4, 0.0, flip)
    assert_words_equal(vote, want, "packed vote")
    assert np.array_equal(hv.numpy().view(np.uint32), want), "vote copied to the host"
    assert_f32_close(x, x_np, "parameters")
    assert count_bit_mismatch(x, x_np) == 0
    for v, v_np in zip(moms, moms_np):
        assert_f32_close(v, v_np, "momentum")
        assert count_bit_mismatch(v, v_np) == 0


@pytest.mark.gpu
def test_static_staging_matches_the_cpu_checker_and_takes_no_device_memory():
    """Two calls in a row with different shapes against the CPU checker directly, and the property
    the entry point exists for: once the first call on the device has been made, further calls
    leave the amount of free device memory exactly where it was."""
    shapes = [(15, 32 * 9000 + 8, torch.float32, 0), (5, 77_777, torch.bfloat16, 0b00100)]
    state = []
    for M, d, dtype, flip in shapes:
        x = torch.randn(d, device=DEV, generator=torch.Generator(device=DEV).manual_seed(d))
        moms = [torch.zeros(d, device=DEV) for _ in range(M)]
        state.append((x, moms, to_np(x), [np.zeros(d, dtype=np.float32) for _ in range(M)]))
    (M, d, dtype, flip), (x, moms, x_np, moms_np) = shapes[0], state[0]
    _run_against_the_checker(M, d, dtype, flip, 0, x, moms, x_np, moms_np)   # also the set-up call
    host_sets = []
    for (M, d, dtype, flip) in shapes:               # host buffers made before the measurement
        case = inputs.cfg3(d)
        case.M, case.dtype = M, dtype
        host_sets.append([g.cpu().pin_memory() for g in inputs.gradients(case, DEV, 7)])
    votes = [torch.zeros(B.ss_packed_words(d), dtype=torch.int32, device=DEV) for (_, d, _, _) in shapes]
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        for (M, d, dtype, flip), (x, moms, _, _), host, vote in zip(shapes, state, host_sets, votes):
            B.ss_fused_step_host_static(host, moms, x, 0.9, 1e-4, 0.0, flip, vote, None)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "a call changed the free device memory by %d bytes" % (free_before - free_after)
    # those calls moved the state; bring the checker's copy along, then compare once more per shape
    for (M, d, dtype, flip), (x, moms, x_np, moms_np), host in zip(shapes, state, host_sets):
        for _ in range(3):
            oracle.fused_step([to_np(h) for h in host], moms_np, x_np, 0.9, 1e-4, 0.0, flip)
    for step, ((M, d, dtype, flip), (x, moms, x_np, moms_np)) in enumerate(zip(shapes, state)):
        _run_against_the_checker(M, d, dtype, flip, 20 + step, x, moms, x_np, moms_np)


@pytest.mark.gpu
def test_static_staging_refuses_requests_beyond_its_size():
    M = 3
    d = B.SS_STATIC_STAGING_BYTES // 4 // M + 64        # M * d * 4 bytes > the fixed array
    host = [torch.zeros(d) for _ in range(M)]
    x = torch.zeros(d, device=DEV)
    vote = torch.zeros(B.ss_packed_words(d), dtype=torch.int32, device=DEV)
    with pytest.raises(B.SignSGDError) as ei:
        B.ss_fused_step_host_static(host, None, x, 0.0, 1e-3, 0.0, 0, vote, None)
    assert ei.value.status == B.SS_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((x == 0).all())                          # nothing was enqueued


def test_static_staging_argument_errors_need_no_gpu():
    L = B.lib()
    fake = ctypes.c_void_p(0x1000)
    arr = (ctypes.c_void_p * 1)(0x1000)
    big = B.SS_STATIC_STAGING_BYTES // 4 + 1
    assert L.ss_fused_step_host_static(arr, 0, None, 1, big, 0.0, 0, fake, 0.1, 0.0, fake, None, None) == B.SS_ERR_UNSUPPORTED
    assert L.ss_fused_step_host_static(arr, 0, None, 0, 8, 0.0, 0, fake, 0.1, 0.0, fake, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step_host_static(None, 0, None, 1, 8, 0.0, 0, fake, 0.1, 0.0, fake, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step_host_static(arr, 0, None, 1, 8, 0.0, 2, fake, 0.1, 0.0, fake, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step_host_static(None, 0, None, 1, 0, 0.0, 0, None, 0.1, 0.0, None, None, None) == B.SS_OK
