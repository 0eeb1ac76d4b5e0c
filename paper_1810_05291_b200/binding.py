"""Python names for the C ABI of libsignsgd.so -- argument marshalling only.

Each function below has the name and the argument order of its C entry point (see
``include/signsgd.h``) and does nothing but check tensor types, take ``data_ptr()`` and the
current CUDA stream, call into the library and raise on a non-zero status. All arithmetic
of Algorithm 1 happens in the CUDA kernels. There is no CPU fallback: if the library has
not been built (``python -m paper_1810_05291_b200.build``), the first call raises.

Tensors: gradients ``float32`` or ``bfloat16``; momenta and parameters ``float32``; packed
signs and votes ``int32`` (bit pattern of the uint32 words), ``ceil(d/32)`` of them.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsignsgd.so")

SS_F32 = 0
SS_BF16 = 1
SS_MAX_WORKERS = 64
SS_STATIC_STAGING_BYTES = 64 << 20
SS_FLAGS_MAX_TIMEOUT_NS = 2_000_000_000

SS_OK = 0
SS_ERR_INVALID_ARG = -1
SS_ERR_MISALIGNED = -2
SS_ERR_UNSUPPORTED = -3
SS_ERR_CUDA = -4

EXPORTS = ("ss_packed_words", "ss_status_string", "ss_last_cuda_error", "ss_sign_pack",
           "ss_majority_vote", "ss_signum_update", "ss_apply_vote", "ss_fused_step",
           "ss_segments_upload", "ss_fused_step_segments", "ss_apply_vote_segments",
           "ss_vote_apply", "ss_vote_apply_segments", "ss_signum_update_push", "ss_vote_tally", "ss_fused_step_host", "ss_fused_step_host_static", "ss_set_launch_option",
           "ss_ternary_words", "ss_absmax", "ss_ternary_pack", "ss_ternary_unpack",
           "ss_flags_signal", "ss_flags_wait", "ss_flags_signal_wait", "ss_vote_apply_guarded",
           "ss_vote_apply_guarded_segments")


class ss_segment(ctypes.Structure):
    """One tensor of a fused flat vector: first coordinate, learning rate, weight decay."""
    _fields_ = [("begin", ctypes.c_int64), ("lr", ctypes.c_float), ("weight_decay", ctypes.c_float)]


SEGMENT_BYTES = ctypes.sizeof(ss_segment)  # 16

_lib = None


class SignSGDError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ss_status_string(status).decode()
        if status == SS_ERR_CUDA:
            msg += " [cudaError %d]" % lib().ss_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


def lib() -> ctypes.CDLL:
    """Load libsignsgd.so (once). Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "libsignsgd.so is missing (%s). Build it with `python -m paper_1810_05291_b200.build`; "
            "this package has no CPU or PyTorch fallback." % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i64, i32, u64, f32 = (ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint64,
                              ctypes.c_float)
    L.ss_packed_words.argtypes = [i64]
    L.ss_packed_words.restype = i64
    L.ss_status_string.argtypes = [i32]
    L.ss_status_string.restype = ctypes.c_char_p
    L.ss_last_cuda_error.argtypes = []
    L.ss_last_cuda_error.restype = i32
    L.ss_sign_pack.argtypes = [vp, i32, i64, vp, vp]
    L.ss_majority_vote.argtypes = [vp, i32, i64, u64, vp, vp]
    L.ss_signum_update.argtypes = [vp, i32, vp, f32, i64, vp, vp]
    L.ss_apply_vote.argtypes = [vp, vp, i64, f32, f32, vp]
    L.ss_fused_step.argtypes = [vp, i32, vp, i32, i64, f32, u64, vp, f32, f32, vp, vp]
    L.ss_fused_step_host.argtypes = [vp, i32, vp, vp, i32, i64, f32, u64, vp, f32, f32, vp, vp, vp]
    L.ss_fused_step_host_static.argtypes = [vp, i32, vp, i32, i64, f32, u64, vp, f32, f32, vp, vp, vp]
    L.ss_set_launch_option.argtypes = [ctypes.c_char_p, i32]
    L.ss_segments_upload.argtypes = [vp, i32, i64, vp, vp]
    L.ss_fused_step_segments.argtypes = [vp, i32, vp, i32, i64, f32, u64, vp, vp, i32, vp, vp]
    L.ss_apply_vote_segments.argtypes = [vp, vp, i64, vp, i32, vp]
    L.ss_signum_update_push.argtypes = [vp, i32, vp, f32, i64, vp, i32, vp]
    L.ss_vote_tally.argtypes = [vp, i32, i64, u64, vp, vp]
    L.ss_vote_apply.argtypes = [vp, i32, i64, u64, vp, f32, f32, vp, vp]
    L.ss_vote_apply_segments.argtypes = [vp, i32, i64, u64, vp, vp, i32, vp, vp]
    L.ss_ternary_words.argtypes = [i64]
    L.ss_ternary_words.restype = i64
    L.ss_absmax.argtypes = [vp, i32, i64, vp, vp]
    L.ss_ternary_pack.argtypes = [vp, i32, i64, vp, u64, vp, vp]
    L.ss_ternary_unpack.argtypes = [vp, i64, vp, vp, vp]
    L.ss_flags_signal.argtypes = [vp, i32, i32, ctypes.c_uint32, vp]
    L.ss_flags_wait.argtypes = [vp, i32, ctypes.c_uint32, u64, vp, vp]
    L.ss_vote_apply_guarded.argtypes = [vp, i32, i64, u64, vp, f32, f32, vp, vp, vp]
    L.ss_vote_apply_guarded_segments.argtypes = [vp, i32, i64, u64, vp, vp, i32, vp, vp, vp]
    L.ss_flags_signal_wait.argtypes = [vp, i32, i32, vp, i32, ctypes.c_uint32, u64, vp, vp]
    for name in ("ss_flags_signal", "ss_flags_wait", "ss_flags_signal_wait", "ss_vote_apply_guarded",
                 "ss_vote_apply_guarded_segments"):
        getattr(L, name).restype = i32
    for name in ("ss_absmax", "ss_ternary_pack", "ss_ternary_unpack"):
        getattr(L, name).restype = i32
    for name in ("ss_sign_pack", "ss_majority_vote", "ss_signum_update", "ss_apply_vote",
                 "ss_fused_step", "ss_fused_step_host", "ss_fused_step_host_static",
                 "ss_set_launch_option", "ss_segments_upload", "ss_fused_step_segments",
                 "ss_apply_vote_segments", "ss_vote_apply", "ss_vote_apply_segments",
                 "ss_signum_update_push", "ss_vote_tally"):
        getattr(L, name).restype = i32
    _lib = L
    return L


# ---- marshalling helpers ------------------------------------------------------------------

def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SS_F32
    if t.dtype == torch.bfloat16:
        return SS_BF16
    raise TypeError("gradient dtype must be float32 or bfloat16, got %s" % t.dtype)


def _dev(t: torch.Tensor, dtype, name: str, n: Optional[int] = None) -> int:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (name, dtype, t.dtype))
    if t.dim() != 1 or not t.is_contiguous():
        raise ValueError("%s must be a contiguous 1-D tensor" % name)
    if n is not None and t.numel() != n:
        raise ValueError("%s must have %d elements, has %d" % (name, n, t.numel()))
    return t.data_ptr()


def _words(t: torch.Tensor, d: int, name: str) -> int:
    return _dev(t, torch.int32, name, ss_packed_words(d))


def _ptr_array(ptrs: Sequence[int]):
    return (ctypes.c_void_p * len(ptrs))(*ptrs)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status: int, where: str) -> None:
    if status != SS_OK:
        raise SignSGDError(status, where)


# ---- the entry points -----------------------------------------------------------------------

def ss_packed_words(d: int) -> int:
    return int(lib().ss_packed_words(int(d)))


def ss_status_string(status: int) -> str:
    return lib().ss_status_string(int(status)).decode()


def ss_set_launch_option(key: str, value: int) -> None:
    _check(lib().ss_set_launch_option(key.encode(), int(value)), "ss_set_launch_option")


def ss_sign_pack(grad: torch.Tensor, out_words: torch.Tensor, stream=None) -> None:
    d = grad.numel()
    _check(lib().ss_sign_pack(_dev(grad, None, "grad"), _dtype_code(grad), d,
                              _words(out_words, d, "out_words"), _stream(stream)), "ss_sign_pack")


def ss_majority_vote(packed: Sequence[torch.Tensor], d: int, flip_mask: int,
                     vote_words: torch.Tensor, stream=None) -> None:
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    _check(lib().ss_majority_vote(_ptr_array(ptrs), len(ptrs), int(d), int(flip_mask),
                                  _words(vote_words, d, "vote_words"), _stream(stream)),
           "ss_majority_vote")


def ss_signum_update(grad: torch.Tensor, momentum: torch.Tensor, beta: float,
                     out_words: torch.Tensor, stream=None) -> None:
    d = grad.numel()
    _check(lib().ss_signum_update(_dev(grad, None, "grad"), _dtype_code(grad),
                                  _dev(momentum, torch.float32, "momentum", d), float(beta), d,
                                  _words(out_words, d, "out_words"), _stream(stream)),
           "ss_signum_update")


def ss_signum_update_push(grad: torch.Tensor, momentum: torch.Tensor, beta: float,
                          dests: Sequence[torch.Tensor], stream=None) -> None:
    """``dests`` may be tensors on this GPU or raw integer addresses of peer buffers."""
    d = grad.numel()
    ptrs = [p if isinstance(p, int) else _words(p, d, "dests[%d]" % i) for i, p in enumerate(dests)]
    _check(lib().ss_signum_update_push(_dev(grad, None, "grad"), _dtype_code(grad),
                                       _dev(momentum, torch.float32, "momentum", d), float(beta), d,
                                       _ptr_array(ptrs), len(ptrs), _stream(stream)),
           "ss_signum_update_push")


def ss_vote_tally(packed: Sequence[torch.Tensor], d: int, flip_mask: int, tally_out: torch.Tensor,
                  stream=None) -> None:
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    _check(lib().ss_vote_tally(_ptr_array(ptrs), len(ptrs), int(d), int(flip_mask),
                               _dev(tally_out, torch.int8, "tally_out", int(d)), _stream(stream)),
           "ss_vote_tally")


def ss_apply_vote(param: torch.Tensor, vote_words: torch.Tensor, lr: float,
                  weight_decay: float = 0.0, stream=None) -> None:
    d = param.numel()
    _check(lib().ss_apply_vote(_dev(param, torch.float32, "param"), _words(vote_words, d, "vote_words"),
                               d, float(lr), float(weight_decay), _stream(stream)), "ss_apply_vote")


def ss_vote_apply(packed: Sequence[torch.Tensor], param: torch.Tensor, lr: float,
                  weight_decay: float = 0.0, flip_mask: int = 0,
                  vote_words_out: Optional[torch.Tensor] = None, stream=None) -> None:
    d = param.numel()
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    w_ptr = None if vote_words_out is None else _words(vote_words_out, d, "vote_words_out")
    _check(lib().ss_vote_apply(_ptr_array(ptrs), len(ptrs), d, int(flip_mask),
                               _dev(param, torch.float32, "param"), float(lr), float(weight_decay),
                               w_ptr, _stream(stream)), "ss_vote_apply")


def _step_args(grads, momenta, param, vote_words_out):
    """Marshalling shared by the fused-step entry points: (dtype code, gradient pointer array,
    momentum pointer array or None, vote pointer or None, M, d)."""
    M = len(grads)
    d = param.numel()
    codes = {_dtype_code(g) for g in grads}
    if len(codes) != 1:
        raise TypeError("all gradients must share one dtype")
    g_ptrs = [_dev(g, None, "grads[%d]" % m, d) for m, g in enumerate(grads)]
    v_arr = None
    if momenta is not None:
        if len(momenta) != M:
            raise ValueError("need one momentum buffer per worker")
        v_arr = _ptr_array([_dev(v, torch.float32, "momenta[%d]" % m, d) for m, v in enumerate(momenta)])
    w_ptr = None if vote_words_out is None else _words(vote_words_out, d, "vote_words_out")
    return codes.pop(), _ptr_array(g_ptrs), v_arr, w_ptr, M, d


def ss_fused_step(grads: Sequence[torch.Tensor], momenta: Optional[Sequence[torch.Tensor]],
                  param: torch.Tensor, beta: float, lr: float, weight_decay: float = 0.0,
                  flip_mask: int = 0, vote_words_out: Optional[torch.Tensor] = None,
                  stream=None) -> None:
    code, g_arr, v_arr, w_ptr, M, d = _step_args(grads, momenta, param, vote_words_out)
    _check(lib().ss_fused_step(g_arr, code, v_arr, M, d, float(beta),
                               int(flip_mask), _dev(param, torch.float32, "param"), float(lr),
                               float(weight_decay), w_ptr, _stream(stream)), "ss_fused_step")


def segment_table(n_segments: int, device) -> torch.Tensor:
    """Device storage for a table of n_segments ss_segment entries (16 bytes each)."""
    return torch.zeros(2 * int(n_segments), dtype=torch.int64, device=device)


def _segments(t: torch.Tensor, n_segments: int) -> int:
    if not t.is_cuda or t.dtype != torch.int64 or not t.is_contiguous() or t.numel() < 2 * n_segments:
        raise ValueError("segments_dev must come from segment_table(n_segments, device)")
    return t.data_ptr()


def ss_segments_upload(begins: Sequence[int], lrs: Sequence[float], weight_decays: Sequence[float],
                       d: int, segments_dev: torch.Tensor, stream=None) -> None:
    n = len(begins)
    if len(lrs) != n or len(weight_decays) != n:
        raise ValueError("begins, lrs and weight_decays must have one entry per tensor")
    host = (ss_segment * max(n, 1))()
    for k in range(n):
        host[k].begin, host[k].lr, host[k].weight_decay = int(begins[k]), float(lrs[k]), float(weight_decays[k])
    _check(lib().ss_segments_upload(ctypes.cast(host, ctypes.c_void_p), n, int(d),
                                    _segments(segments_dev, n), _stream(stream)), "ss_segments_upload")


def ss_fused_step_segments(grads: Sequence[torch.Tensor], momenta: Optional[Sequence[torch.Tensor]],
                           param: torch.Tensor, beta: float, segments_dev: torch.Tensor,
                           n_segments: int, flip_mask: int = 0,
                           vote_words_out: Optional[torch.Tensor] = None, stream=None) -> None:
    code, g_arr, v_arr, w_ptr, M, d = _step_args(grads, momenta, param, vote_words_out)
    _check(lib().ss_fused_step_segments(g_arr, code, v_arr, M, d, float(beta),
                                        int(flip_mask), _dev(param, torch.float32, "param"),
                                        _segments(segments_dev, n_segments), int(n_segments), w_ptr,
                                        _stream(stream)), "ss_fused_step_segments")


def ss_vote_apply_segments(packed: Sequence[torch.Tensor], param: torch.Tensor,
                           segments_dev: torch.Tensor, n_segments: int, flip_mask: int = 0,
                           vote_words_out: Optional[torch.Tensor] = None, stream=None) -> None:
    d = param.numel()
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    w_ptr = None if vote_words_out is None else _words(vote_words_out, d, "vote_words_out")
    _check(lib().ss_vote_apply_segments(_ptr_array(ptrs), len(ptrs), d, int(flip_mask),
                                        _dev(param, torch.float32, "param"),
                                        _segments(segments_dev, n_segments), int(n_segments), w_ptr,
                                        _stream(stream)), "ss_vote_apply_segments")


def ss_apply_vote_segments(param: torch.Tensor, vote_words: torch.Tensor, segments_dev: torch.Tensor,
                           n_segments: int, stream=None) -> None:
    d = param.numel()
    _check(lib().ss_apply_vote_segments(_dev(param, torch.float32, "param"),
                                        _words(vote_words, d, "vote_words"), d,
                                        _segments(segments_dev, n_segments), int(n_segments),
                                        _stream(stream)), "ss_apply_vote_segments")


def _host_step_args(host_grads, momenta, param, host_vote_out):
    """Marshalling shared by the two host-gradient entry points: (dtype code, host pointer array,
    momentum pointer array or None, host vote pointer or None, M, d)."""
    M = len(host_grads)
    d = param.numel()
    codes = {_dtype_code(g) for g in host_grads}
    if len(codes) != 1:
        raise TypeError("all gradients must share one dtype")
    h_ptrs = []
    for m, g in enumerate(host_grads):
        if g.is_cuda or g.dim() != 1 or not g.is_contiguous() or g.numel() != d:
            raise ValueError("host_grads[%d] must be a contiguous 1-D host tensor of d elements" % m)
        h_ptrs.append(g.data_ptr())
    v_arr = None
    if momenta is not None:
        if len(momenta) != M:
            raise ValueError("need one momentum buffer per worker")
        v_arr = _ptr_array([_dev(v, torch.float32, "momenta[%d]" % m, d) for m, v in enumerate(momenta)])
    hv = None
    if host_vote_out is not None:
        if (host_vote_out.is_cuda or host_vote_out.dtype != torch.int32
                or host_vote_out.numel() != ss_packed_words(d) or not host_vote_out.is_contiguous()):
            raise ValueError("host_vote_out must be a contiguous host int32 tensor of ceil(d/32) words")
        hv = host_vote_out.data_ptr()
    return codes.pop(), _ptr_array(h_ptrs), v_arr, hv, M, d


def ss_fused_step_host(host_grads: Sequence[torch.Tensor], staging: Sequence[torch.Tensor],
                       momenta: Optional[Sequence[torch.Tensor]], param: torch.Tensor, beta: float,
                       lr: float, weight_decay: float, flip_mask: int,
                       vote_words_dev: torch.Tensor, host_vote_out: Optional[torch.Tensor],
                       stream=None) -> None:
    code, h_arr, v_arr, hv, M, d = _host_step_args(host_grads, momenta, param, host_vote_out)
    if len(staging) != M:
        raise ValueError("need one staging buffer per worker")
    s_ptrs = [_dev(s, host_grads[0].dtype, "staging[%d]" % m, d) for m, s in enumerate(staging)]
    _check(lib().ss_fused_step_host(h_arr, code, _ptr_array(s_ptrs), v_arr, M, d,
                                    float(beta), int(flip_mask), _dev(param, torch.float32, "param"),
                                    float(lr), float(weight_decay),
                                    _words(vote_words_dev, d, "vote_words_dev"), hv, _stream(stream)),
           "ss_fused_step_host")


def ss_fused_step_host_static(host_grads: Sequence[torch.Tensor],
                              momenta: Optional[Sequence[torch.Tensor]], param: torch.Tensor,
                              beta: float, lr: float, weight_decay: float, flip_mask: int,
                              vote_words_dev: torch.Tensor, host_vote_out: Optional[torch.Tensor],
                              stream=None) -> None:
    """ss_fused_step_host for callers that may not allocate device memory: the gradients are
    staged in a fixed array inside the library (at most SS_STATIC_STAGING_BYTES for all M workers
    together), so no staging tensors are passed. The first call on a device looks up that array's
    address (and, with lazy module loading, is what reserves the array); make it during start-up.
    Calls that overlap on the GPU race on the array."""
    code, h_arr, v_arr, hv, M, d = _host_step_args(host_grads, momenta, param, host_vote_out)
    _check(lib().ss_fused_step_host_static(h_arr, code, v_arr, M, d, float(beta),
                                           int(flip_mask), _dev(param, torch.float32, "param"),
                                           float(lr), float(weight_decay),
                                           _words(vote_words_dev, d, "vote_words_dev"), hv,
                                           _stream(stream)), "ss_fused_step_host_static")


# ---- the comparison codec of Appendix B (1-bit max-norm QSGD) -------------------------------

def ss_ternary_words(d: int) -> int:
    return int(lib().ss_ternary_words(int(d)))


def ss_absmax(grad: torch.Tensor, absmax_dev: torch.Tensor, stream=None) -> None:
    _check(lib().ss_absmax(_dev(grad, None, "grad"), _dtype_code(grad), grad.numel(),
                           _dev(absmax_dev, torch.float32, "absmax_dev", 1), _stream(stream)), "ss_absmax")


def ss_ternary_pack(grad: torch.Tensor, absmax_dev: torch.Tensor, seed: int, out_codes: torch.Tensor,
                    stream=None) -> None:
    d = grad.numel()
    _check(lib().ss_ternary_pack(_dev(grad, None, "grad"), _dtype_code(grad), d,
                                 _dev(absmax_dev, torch.float32, "absmax_dev", 1), int(seed),
                                 _dev(out_codes, torch.int32, "out_codes", ss_ternary_words(d)),
                                 _stream(stream)), "ss_ternary_pack")


def ss_ternary_unpack(codes: torch.Tensor, scale_dev: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    d = out.numel()
    _check(lib().ss_ternary_unpack(_dev(codes, torch.int32, "codes", ss_ternary_words(d)), d,
                                   _dev(scale_dev, torch.float32, "scale_dev", 1),
                                   _dev(out, torch.float32, "out"), _stream(stream)), "ss_ternary_unpack")


# ---- flag-ordered exchange (one worker per GPU) -------------------------------------------------

def flag_array(device) -> torch.Tensor:
    """Storage for one worker's flag array: SS_MAX_WORKERS words, zeroed (epoch 0 = nothing arrived)."""
    return torch.zeros(SS_MAX_WORKERS, dtype=torch.int32, device=device)


def ss_flags_signal(flags: Sequence, index: int, epoch: int, stream=None) -> None:
    """``flags`` may be tensors on this GPU or raw integer addresses of peers' flag arrays."""
    ptrs = [p if isinstance(p, int) else _dev(p, torch.int32, "flags[%d]" % i) for i, p in enumerate(flags)]
    _check(lib().ss_flags_signal(_ptr_array(ptrs), len(ptrs), int(index), int(epoch) & 0xFFFFFFFF,
                                 _stream(stream)), "ss_flags_signal")


def ss_flags_wait(flags_local: torch.Tensor, M: int, epoch: int, timeout_ns: int, status_dev: torch.Tensor,
                  stream=None) -> None:
    _check(lib().ss_flags_wait(_dev(flags_local, torch.int32, "flags_local"), int(M), int(epoch) & 0xFFFFFFFF,
                               int(timeout_ns), _dev(status_dev, torch.int32, "status_dev", 1),
                               _stream(stream)), "ss_flags_wait")


def ss_flags_signal_wait(flags: Sequence, index: int, flags_local: torch.Tensor, M: int, epoch: int,
                         timeout_ns: int, status_dev: torch.Tensor, stream=None) -> None:
    ptrs = [p if isinstance(p, int) else _dev(p, torch.int32, "flags[%d]" % i) for i, p in enumerate(flags)]
    _check(lib().ss_flags_signal_wait(_ptr_array(ptrs), len(ptrs), int(index),
                                      _dev(flags_local, torch.int32, "flags_local"), int(M),
                                      int(epoch) & 0xFFFFFFFF, int(timeout_ns),
                                      _dev(status_dev, torch.int32, "status_dev", 1), _stream(stream)),
           "ss_flags_signal_wait")


def ss_vote_apply_guarded(packed: Sequence[torch.Tensor], param: torch.Tensor, lr: float,
                          weight_decay: float, flip_mask: int, vote_words_out: Optional[torch.Tensor],
                          skip_if_nonzero_dev: torch.Tensor, stream=None) -> None:
    d = param.numel()
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    w_ptr = None if vote_words_out is None else _words(vote_words_out, d, "vote_words_out")
    _check(lib().ss_vote_apply_guarded(_ptr_array(ptrs), len(ptrs), d, int(flip_mask),
                                       _dev(param, torch.float32, "param"), float(lr), float(weight_decay),
                                       w_ptr, _dev(skip_if_nonzero_dev, torch.int32, "skip_if_nonzero_dev", 1),
                                       _stream(stream)), "ss_vote_apply_guarded")


def ss_vote_apply_guarded_segments(packed: Sequence[torch.Tensor], param: torch.Tensor,
                                   segments_dev: torch.Tensor, n_segments: int, flip_mask: int,
                                   vote_words_out: Optional[torch.Tensor], skip_if_nonzero_dev: torch.Tensor,
                                   stream=None) -> None:
    d = param.numel()
    ptrs = [_words(p, d, "packed[%d]" % m) for m, p in enumerate(packed)]
    w_ptr = None if vote_words_out is None else _words(vote_words_out, d, "vote_words_out")
    _check(lib().ss_vote_apply_guarded_segments(_ptr_array(ptrs), len(ptrs), d, int(flip_mask),
                                                _dev(param, torch.float32, "param"),
                                                _segments(segments_dev, n_segments), int(n_segments), w_ptr,
                                                _dev(skip_if_nonzero_dev, torch.int32, "skip_if_nonzero_dev", 1),
                                                _stream(stream)), "ss_vote_apply_guarded_segments")
