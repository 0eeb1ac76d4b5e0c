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


def test_launch_option_validation(L):
    assert L.ss_set_launch_option(b"threads", 100) == B.SS_ERR_INVALID_ARG
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
