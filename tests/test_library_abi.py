"""The C-ABI library without a GPU: it loads, exports every symbol the header declares, and
rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_1810_05291_b200 import binding as B
from paper_1810_05291_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    libbuild.build()
    return B.lib()


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names.update(re.findall(r"\b(ss_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(L):
    names = declared_symbols()
    assert {"ss_sign_pack", "ss_majority_vote", "ss_signum_update", "ss_apply_vote",
            "ss_fused_step"} <= names
    for n in names:
        assert hasattr(L, n), "libsignsgd.so does not export %s" % n
    assert names == set(B.EXPORTS), "header and binding disagree on the entry points"


def test_every_entry_point_has_its_argument_types_declared(L):
    for n in B.EXPORTS:
        assert getattr(L, n).argtypes is not None or n in ("ss_last_cuda_error",), "%s: argtypes not set" % n


def test_packed_words(L):
    assert B.ss_packed_words(0) == 0
    assert B.ss_packed_words(1) == 1
    assert B.ss_packed_words(32) == 1
    assert B.ss_packed_words(33) == 2
    assert B.ss_packed_words(25_557_032) == 798_658
    assert B.ss_packed_words(61_100_840) == 1_909_402
    assert B.ss_packed_words(-5) == -1


def test_status_strings(L):
    assert B.ss_status_string(0) == "SS_OK"
    for code in (-1, -2, -3, -4):
        assert B.ss_status_string(code).startswith("SS_ERR_")
    assert B.ss_status_string(99) == "unknown status"


def test_argument_errors_are_reported_before_any_cuda_call(L):
    fake = ctypes.c_void_p(0x1000)          # aligned, never dereferenced: validation fails first
    arr1 = (ctypes.c_void_p * 1)(0x1000)
    null_arr = (ctypes.c_void_p * 1)(None)
    # null pointers
    assert L.ss_sign_pack(None, 0, 10, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step(None, 0, None, 1, 10, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_sign_pack(fake, 0, 10, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step(arr1, 0, None, 1, 10, 0.0, 0, None, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step(null_arr, 0, None, 1, 10, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    # worker count and size out of range
    assert L.ss_fused_step(arr1, 0, None, 0, 10, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step(arr1, 0, None, 65, 10, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_fused_step(arr1, 0, None, 1, -1, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_majority_vote(arr1, 0, 10, 0, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_apply_vote(fake, fake, -3, 0.1, 0.0, None) == B.SS_ERR_INVALID_ARG
    # flip_mask names a worker that does not exist
    assert L.ss_fused_step(arr1, 0, None, 1, 10, 0.0, 2, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_majority_vote(arr1, 1, 10, 2, fake, None) == B.SS_ERR_INVALID_ARG
    # bad dtype
    assert L.ss_sign_pack(fake, 7, 10, fake, None) == B.SS_ERR_INVALID_ARG
    # misaligned below the element size
    odd = ctypes.c_void_p(0x1002)
    assert L.ss_sign_pack(odd, 0, 10, ctypes.c_void_p(0x9000), None) == B.SS_ERR_MISALIGNED
    assert L.ss_apply_vote(ctypes.c_void_p(0x1001), ctypes.c_void_p(0x9000), 10, 0.1, 0.0, None) == B.SS_ERR_MISALIGNED
    # overlapping buffers
    assert L.ss_apply_vote(fake, fake, 10, 0.1, 0.0, None) == B.SS_ERR_INVALID_ARG
    # d == 0 is a no-op
    assert L.ss_sign_pack(fake, 0, 0, None, None) == B.SS_OK
    assert L.ss_sign_pack(None, 0, 0, None, None) == B.SS_OK
    assert L.ss_fused_step(None, 0, None, 1, 0, 0.0, 0, None, 0.1, 0.0, None, None) == B.SS_OK
    assert L.ss_fused_step(None, 0, None, 0, 0, 0.0, 0, None, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_apply_vote(None, None, 0, 0.1, 0.0, None) == B.SS_OK
    assert L.ss_majority_vote(arr1, 1, 0, 0, None, None) == B.SS_OK


def test_host_entry_points_check_every_argument_before_the_first_copy(L):
    """ss_fused_step_host and its static-staging sibling: a bad momentum, parameter or vote buffer
    must be reported before any copy is enqueued. With fake pointers and no GPU in reach, a call
    that got as far as a copy would come back as SS_ERR_CUDA (or crash) instead."""
    vp = ctypes.c_void_p
    d, M = 64, 2
    host = (vp * M)(0x10000, 0x20000)
    stage = (vp * M)(0x30000, 0x40000)
    mom_ok = (vp * M)(0x50000, 0x60000)
    x, vote = vp(0x70000), vp(0x80000)

    def host_call(staging=stage, momenta=mom_ok, param=x, words=vote, dd=d, flip=0):
        return L.ss_fused_step_host(host, 0, staging, momenta, M, dd, 0.9, flip, param, 0.1, 0.0, words, None, None)

    def static_call(momenta=mom_ok, param=x, words=vote, dd=d, flip=0):
        return L.ss_fused_step_host_static(host, 0, momenta, M, dd, 0.9, flip, param, 0.1, 0.0, words, None, None)

    for call in (host_call, static_call):
        assert call(momenta=(vp * M)(0x50000, None)) == B.SS_ERR_INVALID_ARG          # NULL momentum
        assert call(momenta=(vp * M)(0x50002, 0x60000)) == B.SS_ERR_MISALIGNED        # below 4 bytes
        assert call(momenta=(vp * M)(0x50000, 0x50080)) == B.SS_ERR_INVALID_ARG       # momenta overlap
        assert call(momenta=(vp * M)(0x50000, 0x70040)) == B.SS_ERR_INVALID_ARG       # momentum on param
        assert call(words=vp(0x50004)) == B.SS_ERR_INVALID_ARG                        # vote on a momentum
        assert call(words=vp(0x70010)) == B.SS_ERR_INVALID_ARG                        # vote on param
        assert call(words=vp(0x80002)) == B.SS_ERR_MISALIGNED
        assert call(param=vp(0x70001)) == B.SS_ERR_MISALIGNED
        assert call(flip=4) == B.SS_ERR_INVALID_ARG
        assert call(dd=(1 << 62) + 5) == B.SS_ERR_INVALID_ARG                         # d that would wrap d * 4
        assert call(dd=(1 << 40) + 1) == B.SS_ERR_INVALID_ARG
    assert host_call(staging=(vp * M)(0x30000, None)) == B.SS_ERR_INVALID_ARG
    assert host_call(staging=(vp * M)(0x30000, 0x30040)) == B.SS_ERR_INVALID_ARG      # staging overlap
    assert host_call(staging=(vp * M)(0x30000, 0x50000)) == B.SS_ERR_INVALID_ARG      # staging on a momentum
    assert host_call(staging=(vp * M)(0x30000, 0x7FFF0)) == B.SS_ERR_INVALID_ARG      # staging on the vote
    # the static variant's size limit is tested without forming a product that could wrap
    assert static_call(dd=(B.SS_STATIC_STAGING_BYTES // 4) // M + 64) == B.SS_ERR_UNSUPPORTED
    assert static_call(dd=1 << 40) == B.SS_ERR_UNSUPPORTED


def test_sizes_that_would_wrap_a_byte_count_are_refused(L):
    fake = ctypes.c_void_p(0x1000)
    arr1 = (ctypes.c_void_p * 1)(0x1000)
    for d in ((1 << 62) + 8, (1 << 63) - 1, (1 << 40) + 1):
        assert L.ss_sign_pack(fake, 0, d, fake, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_fused_step(arr1, 0, None, 1, d, 0.0, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_majority_vote(arr1, 1, d, 0, fake, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_apply_vote(fake, fake, d, 0.1, 0.0, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_vote_apply(arr1, 1, d, 0, fake, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_signum_update_push(fake, 0, fake, 0.9, d, arr1, 1, None) == B.SS_ERR_INVALID_ARG
        assert L.ss_vote_tally(arr1, 1, d, 0, fake, None) == B.SS_ERR_INVALID_ARG


def test_step_arguments_may_not_alias_what_the_step_writes(L):
    vp = ctypes.c_void_p
    g = (vp * 2)(0x10000, 0x20000)
    x = vp(0x70000)
    # a momentum buffer on another worker's gradient
    assert L.ss_fused_step(g, 0, (vp * 2)(0x50000, 0x10040), 2, 64, 0.9, 0, x, 0.1, 0.0, None, None) == B.SS_ERR_INVALID_ARG
    # the packed output of ss_signum_update on its momentum
    assert L.ss_signum_update(vp(0x10000), 0, vp(0x50000), 0.9, 64, vp(0x50010), None) == B.SS_ERR_INVALID_ARG


def test_flag_exchange_argument_errors(L):
    vp = ctypes.c_void_p
    fake, arr = vp(0x1000), (vp * 2)(0x1000, 0x2000)
    assert L.ss_flags_wait(fake, 3, 1, B.SS_FLAGS_MAX_TIMEOUT_NS + 1, fake, None) == B.SS_ERR_INVALID_ARG  # no long waits
    assert L.ss_flags_wait(fake, 0, 1, 1000, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_wait(fake, 65, 1, 1000, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_wait(None, 3, 1, 1000, fake, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_wait(fake, 3, 1, 1000, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_wait(vp(0x1002), 3, 1, 1000, fake, None) == B.SS_ERR_MISALIGNED
    assert L.ss_flags_signal(None, 2, 0, 1, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_signal(arr, 0, 0, 1, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_signal(arr, 65, 0, 1, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_signal(arr, 2, 64, 1, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_signal((vp * 2)(0x1000, None), 2, 0, 1, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_flags_signal((vp * 2)(0x1000, 0x2001), 2, 0, 1, None) == B.SS_ERR_MISALIGNED
    assert L.ss_vote_apply_guarded(arr, 2, 64, 0, vp(0x70000), 0.1, 0.0, None, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_vote_apply_guarded(arr, 2, 64, 0, vp(0x70000), 0.1, 0.0, None, vp(0x9001), None) == B.SS_ERR_MISALIGNED
    assert L.ss_vote_apply_guarded(arr, 2, 64, 0, vp(0x70000), 0.1, 0.0, None, vp(0x70010), None) == B.SS_ERR_INVALID_ARG  # guard inside param
    assert L.ss_vote_apply_guarded(arr, 2, 64, 0, vp(0x70000), 0.1, 0.0, vp(0x80000), vp(0x80004), None) == B.SS_ERR_INVALID_ARG  # guard inside the vote
    seg = vp(0x90000)
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), seg, 1, None, None, None) == B.SS_ERR_INVALID_ARG
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), seg, 1, None, vp(0x9001), None) == B.SS_ERR_MISALIGNED
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), seg, 1, None, vp(0x70010), None) == B.SS_ERR_INVALID_ARG
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), seg, 0, None, vp(0xA0000), None) == B.SS_ERR_INVALID_ARG  # empty table
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), None, 1, None, vp(0xA0000), None) == B.SS_ERR_INVALID_ARG
    assert L.ss_vote_apply_guarded_segments(arr, 2, 64, 0, vp(0x70000), vp(0x90004), 1, None, vp(0xA0000), None) == B.SS_ERR_MISALIGNED


def test_launch_option_validation(L):
    assert L.ss_set_launch_option(b"threads", 100) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"threads", 512) == B.SS_ERR_INVALID_ARG      # kernels are built for <= 256
    assert L.ss_set_launch_option(b"threads", 1024) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"threads", 256) == B.SS_OK
    assert L.ss_set_launch_option(b"blocks_per_sm", 4097) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"plain_loads_from_mib", -1) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"plain_loads_from_mib", (1 << 20) + 1) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"plain_loads_from_mib", 1) == B.SS_OK
    assert L.ss_set_launch_option(b"plain_loads_from_mib", 0) == B.SS_OK
    assert L.ss_set_launch_option(b"nope", 1) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(None, 1) == B.SS_ERR_INVALID_ARG
    assert L.ss_set_launch_option(b"threads", 128) == B.SS_OK
    assert L.ss_set_launch_option(b"threads", 0) == B.SS_OK
    assert L.ss_set_launch_option(b"blocks_per_sm", 0) == B.SS_OK


def test_binding_refuses_cpu_tensors(L):
    import torch
    g = torch.zeros(64)
    w = torch.zeros(2, dtype=torch.int32)
    with pytest.raises(ValueError):
        B.ss_sign_pack(g, w)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libsignsgd.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.ss_packed_words(5)


def test_the_product_never_reaches_for_the_cpu_checker():
    """The CPU oracle is test infrastructure: nothing under the package may import, load or name it,
    and the binding must refuse to run without the CUDA library rather than fall back."""
    pkg = os.path.join(ROOT, "paper_1810_05291_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text.lower(), "%s mentions the oracle" % fn
    missing = os.path.join(pkg, "no_such_dir", "libsignsgd.so")
    saved_path, saved_lib = B.LIB_PATH, B._lib
    try:
        B.LIB_PATH, B._lib = missing, None
        with pytest.raises(RuntimeError):
            B.lib()
    finally:
        B.LIB_PATH, B._lib = saved_path, saved_lib
