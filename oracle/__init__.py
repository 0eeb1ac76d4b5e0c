"""CPU oracle for Signum / signSGD with majority vote (Algorithm 1) -- numpy front end.

TEST INFRASTRUCTURE ONLY: the slow, plain CPU definition the CUDA library is checked
against. Nothing on the product path imports this package; only the tests, the smoke
check and the benchmark's CPU-baseline leg do. It shares no code with the CUDA path.

The arithmetic lives in ``signsgd_oracle.cpp`` (Algorithm 1) and ``ternary_oracle.cpp`` (the
comparison codec of Appendix B), plain C++, one coordinate at a time; this module only compiles
them with g++ on first use, loads it with ctypes and passes
numpy arrays through. Arrays: gradients ``float32`` or raw bf16 bit patterns as
``uint16``; momenta and parameters ``float32`` (updated in place); packed signs and
votes ``uint32`` with ``ceil(d/32)`` words, coordinate ``32 j + i`` at bit ``i`` of word ``j``.
"""

from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "signsgd_oracle.cpp")
_SRC_TERNARY = os.path.join(_HERE, "ternary_oracle.cpp")   # the comparison codec of Appendix B
_LIB = os.path.join(_HERE, "libsignsgd_oracle.so")
_lock = threading.Lock()
_lib = None

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (-O2 -ffp-contract=off: no fused multiply-add, so the
    momentum is two rounded multiplies and one rounded add as Algorithm 1's line is read)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_TERNARY))):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-fPIC", "-shared", "-o", tmp, _SRC, _SRC_TERNARY]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        vp, i64, i32, u64, f32 = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint64,
                                  ctypes.c_float)
        lib.oracle_set_threads.argtypes = [i32]
        lib.oracle_set_threads.restype = None
        lib.oracle_get_threads.restype = i32
        lib.oracle_max_threads.restype = i32
        lib.oracle_packed_words.argtypes = [i64]
        lib.oracle_packed_words.restype = i64
        lib.oracle_sign_pack.argtypes = [vp, i32, i64, vp]
        lib.oracle_sign_pack.restype = None
        lib.oracle_unpack.argtypes = [vp, i64, vp]
        lib.oracle_unpack.restype = None
        lib.oracle_majority_vote.argtypes = [vp, i32, i64, u64, vp, vp]
        lib.oracle_majority_vote.restype = None
        lib.oracle_signum_update.argtypes = [vp, i32, vp, f32, i64, vp]
        lib.oracle_signum_update.restype = None
        lib.oracle_apply_vote.argtypes = [vp, vp, i64, f32, f32]
        lib.oracle_apply_vote.restype = None
        lib.oracle_fused_step.argtypes = [vp, i32, vp, i32, i64, f32, u64, vp, f32, f32, vp]
        lib.oracle_fused_step.restype = None
        lib.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        lib.oracle_philox4x32_10.restype = None
        lib.oracle_ternary_draws.argtypes = [u64, i64, vp]
        lib.oracle_ternary_draws.restype = None
        lib.oracle_absmax.argtypes = [vp, i32, i64]
        lib.oracle_absmax.restype = f32
        lib.oracle_ternary_words.argtypes = [i64]
        lib.oracle_ternary_words.restype = i64
        lib.oracle_ternary_pack.argtypes = [vp, i32, i64, f32, vp, vp]
        lib.oracle_ternary_pack.restype = None
        lib.oracle_ternary_unpack.argtypes = [vp, i64, f32, vp]
        lib.oracle_ternary_unpack.restype = None
        _lib = lib
        return lib


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(_load().oracle_get_threads())


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def packed_words(d: int) -> int:
    return int(_load().oracle_packed_words(int(d)))


def _grad(a: np.ndarray):
    if a.dtype == np.float32:
        dt = F32
    elif a.dtype == np.uint16:
        dt = BF16
    else:
        raise TypeError("gradient must be float32 or uint16 (raw bf16), got %s" % a.dtype)
    if a.ndim != 1 or not a.flags.c_contiguous:
        raise ValueError("gradient must be a contiguous 1-D array")
    return dt


def _check(a: np.ndarray, dtype, n: int, name: str):
    if a.dtype != dtype or a.ndim != 1 or not a.flags.c_contiguous or a.shape[0] != n:
        raise ValueError("%s must be a contiguous 1-D %s array of %d elements" % (name, np.dtype(dtype), n))
    if not a.flags.writeable:
        raise ValueError("%s must be writeable" % name)


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _ptr_array(arrs):
    arr = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    return arr


def sign_pack(grad: np.ndarray) -> np.ndarray:
    dt = _grad(grad)
    d = grad.shape[0]
    out = np.zeros(packed_words(d), dtype=np.uint32)
    _load().oracle_sign_pack(_ptr(grad), dt, d, _ptr(out))
    return out


def unpack(words: np.ndarray, d: int) -> np.ndarray:
    _check(words, np.uint32, packed_words(d), "words")
    out = np.zeros(d, dtype=np.int8)
    _load().oracle_unpack(_ptr(words), d, _ptr(out))
    return out


def majority_vote(packed, d: int, flip_mask: int = 0, return_tally: bool = False):
    M = len(packed)
    W = packed_words(d)
    for p in packed:
        _check(p, np.uint32, W, "packed[m]")
    vote = np.zeros(W, dtype=np.uint32)
    tally = np.zeros(d, dtype=np.int32) if return_tally else None
    _load().oracle_majority_vote(_ptr_array(packed), M, d, int(flip_mask), _ptr(vote),
                                 _ptr(tally) if return_tally else None)
    return (vote, tally) if return_tally else vote


def signum_update(grad: np.ndarray, momentum: np.ndarray, beta: float) -> np.ndarray:
    dt = _grad(grad)
    d = grad.shape[0]
    _check(momentum, np.float32, d, "momentum")
    out = np.zeros(packed_words(d), dtype=np.uint32)
    _load().oracle_signum_update(_ptr(grad), dt, _ptr(momentum), float(beta), d, _ptr(out))
    return out


def apply_vote(param: np.ndarray, vote: np.ndarray, lr: float, weight_decay: float = 0.0) -> None:
    d = param.shape[0]
    _check(param, np.float32, d, "param")
    _check(vote, np.uint32, packed_words(d), "vote")
    _load().oracle_apply_vote(_ptr(param), _ptr(vote), d, float(lr), float(weight_decay))


def fused_step(grads, momenta, param: np.ndarray, beta: float, lr: float,
               weight_decay: float = 0.0, flip_mask: int = 0) -> np.ndarray:
    """One iteration of Algorithm 1 over M simulated workers. ``momenta=None`` is signSGD."""
    M = len(grads)
    dts = {_grad(g) for g in grads}
    if len(dts) != 1:
        raise TypeError("all gradients must share one dtype")
    d = grads[0].shape[0]
    for g in grads:
        if g.shape[0] != d:
            raise ValueError("all gradients must have d elements")
    _check(param, np.float32, d, "param")
    if momenta is not None:
        if len(momenta) != M:
            raise ValueError("need one momentum buffer per worker")
        for v in momenta:
            _check(v, np.float32, d, "momenta[m]")
    vote = np.zeros(packed_words(d), dtype=np.uint32)
    _load().oracle_fused_step(_ptr_array(grads), dts.pop(),
                              _ptr_array(momenta) if momenta is not None else None,
                              M, d, float(beta), int(flip_mask), _ptr(param), float(lr),
                              float(weight_decay), _ptr(vote))
    return vote


def fused_step_segments(grads, momenta, param: np.ndarray, beta: float, begins, lrs, weight_decays,
                        flip_mask: int = 0) -> np.ndarray:
    """Algorithm 1 on a flat vector that is the concatenation of several tensors, each with its
    own eta and lambda (Section 4 merges small tensors into one buffer before compression; the
    merged step must equal one step per tensor). Written as exactly that: one ``fused_step`` per
    tensor on that tensor's slice of every buffer. Tensor k covers coordinates
    [begins[k], begins[k+1]), the last one runs to d. Returns the packed vote of the whole vector
    (the vote depends on neither eta nor lambda), computed by a separate whole-vector step on
    copies."""
    d = param.shape[0]
    n = len(begins)
    scratch_m = [v.copy() for v in momenta] if momenta is not None else None
    vote = fused_step(grads, scratch_m, param.copy(), beta, 0.0, 0.0, flip_mask)
    for k in range(n):
        a = int(begins[k])
        b = int(begins[k + 1]) if k + 1 < n else d
        if b <= a:
            continue
        fused_step([g[a:b] for g in grads],
                   [v[a:b] for v in momenta] if momenta is not None else None,
                   param[a:b], beta, float(lrs[k]), float(weight_decays[k]), flip_mask)
    return vote


# ---- the comparison codec of Appendix B: 1-bit max-norm QSGD (ternary, two bits per coordinate) ----

def philox4x32_10(counter, key) -> np.ndarray:
    """One block of the counter-based generator: 4 counter words, 2 key words -> 4 output words."""
    c = np.asarray(counter, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    if c.shape != (4,) or k.shape != (2,):
        raise ValueError("counter has 4 words, key has 2")
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def ternary_draws(seed: int, d: int) -> np.ndarray:
    """The 32-bit draw of every coordinate 0..d-1 under a seed."""
    r = np.zeros(int(d), dtype=np.uint32)
    _load().oracle_ternary_draws(int(seed), int(d), _ptr(r))
    return r


def absmax(grad: np.ndarray) -> float:
    """||g||_inf over the elements that are not NaN, as fp32."""
    dt = _grad(grad)
    return float(_load().oracle_absmax(_ptr(grad), dt, grad.shape[0]))


def ternary_words(d: int) -> int:
    return int(_load().oracle_ternary_words(int(d)))


def ternary_pack(grad: np.ndarray, gmax: float = None, seed: int = None, draws: np.ndarray = None) -> np.ndarray:
    """1-bit max-norm QSGD code of a gradient: two bits per coordinate, 16 per uint32 word. The
    draws are either given (one uint32 per coordinate) or generated from ``seed``."""
    dt = _grad(grad)
    d = grad.shape[0]
    if gmax is None:
        gmax = absmax(grad)
    if draws is None:
        if seed is None:
            raise ValueError("give either the draws or a seed")
        draws = ternary_draws(seed, d)
    _check(draws, np.uint32, d, "draws")
    codes = np.zeros(ternary_words(d), dtype=np.uint32)
    _load().oracle_ternary_pack(_ptr(grad), dt, d, float(np.float32(gmax)), _ptr(draws), _ptr(codes))
    return codes


def ternary_unpack(codes: np.ndarray, d: int, scale: float) -> np.ndarray:
    _check(codes, np.uint32, ternary_words(d), "codes")
    out = np.zeros(int(d), dtype=np.float32)
    _load().oracle_ternary_unpack(_ptr(codes), int(d), float(np.float32(scale)), _ptr(out))
    return out
