"""Shared helpers for the parity tests: tensor <-> numpy conversion for the CPU checker and
runners that push one case through the CUDA library and through the checker."""
import numpy as np
import torch

import oracle
from paper_1810_05291_b200 import binding as B

REL_TOL = 1e-6       # fp32 state: |delta| <= 1e-6 relative per element
ABS_FLOOR = 1e-12    # absolute floor for exact zeros


def to_np(t: torch.Tensor) -> np.ndarray:
    """Same bytes on the host: fp32 -> float32, bf16 -> uint16 bit patterns, int32 words -> uint32."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    if t.dtype == torch.int32:
        return t.numpy().view(np.uint32).copy()
    return t.numpy().copy()


def words_tensor(d: int, device, fill: int = 0) -> torch.Tensor:
    return torch.full((B.ss_packed_words(d),), fill, dtype=torch.int32, device=device)


def assert_words_equal(got: torch.Tensor, want: np.ndarray, what: str = "words"):
    g = to_np(got)
    if not np.array_equal(g, want):
        bad = np.nonzero(g != want)[0]
        raise AssertionError("%s differ in %d of %d words; first at word %d: got %08x want %08x"
                             % (what, bad.size, want.size, bad[0], g[bad[0]], want[bad[0]]))


def assert_f32_close(got, want: np.ndarray, what: str = "fp32 state"):
    """|delta| <= 1e-6 relative per element; NaNs must sit at the same places."""
    g = got if isinstance(got, np.ndarray) else to_np(got)
    assert g.shape == want.shape
    nan_g, nan_w = np.isnan(g), np.isnan(want)
    assert np.array_equal(nan_g, nan_w), "%s: NaN pattern differs" % what
    fin = ~nan_w
    gd, wd = g[fin].astype(np.float64), want[fin].astype(np.float64)
    inf = np.isinf(wd)
    assert np.array_equal(gd[inf], wd[inf]), "%s: infinities differ" % what
    err = np.abs(gd[~inf] - wd[~inf])
    bound = REL_TOL * np.abs(wd[~inf]) + ABS_FLOOR
    if np.any(err > bound):
        i = int(np.argmax(err - bound))
        raise AssertionError("%s: %d elements beyond 1e-6 relative; worst got %r want %r"
                             % (what, int(np.sum(err > bound)), gd[~inf][i], wd[~inf][i]))


def count_bit_mismatch(got: torch.Tensor, want: np.ndarray) -> int:
    """Elements whose fp32 bit patterns differ. A NaN on both sides counts as equal: the NaN
    payload is the one thing IEEE 754 leaves to the implementation (x86 keeps the operand's
    payload, the GPU returns the canonical NaN)."""
    g = got if isinstance(got, np.ndarray) else to_np(got)
    both_nan = np.isnan(g) & np.isnan(want)
    return int(np.count_nonzero((g.view(np.uint32) != want.view(np.uint32)) & ~both_nan))


def assert_f32_state(got: torch.Tensor, want: np.ndarray, what: str = "fp32 state"):
    """Both bars on one device-to-host copy: within 1e-6 relative per element, and (because both
    sides run the same rounded operation sequence) bit-identical apart from NaN payloads."""
    g = to_np(got)
    assert_f32_close(g, want, what)
    n = count_bit_mismatch(g, want)
    assert n == 0, "%s: %d elements differ in their bit patterns" % (what, n)


class GuardedWords:
    """A packed-word output buffer with canary words on both sides, to catch out-of-range writes."""
    CANARY = 0x5A5A5A5A
    PAD = 64

    def __init__(self, d: int, device, misalign_words: int = 0):
        W = B.ss_packed_words(d)
        self.full = torch.full((W + 2 * self.PAD + misalign_words,), self.CANARY, dtype=torch.int32,
                               device=device)
        lo = self.PAD + misalign_words
        self.view = self.full[lo: lo + W]
        self.lo, self.W = lo, W

    def check(self):
        f = self.full.cpu()
        assert bool((f[: self.lo] == self.CANARY).all()), "write before the output buffer"
        assert bool((f[self.lo + self.W:] == self.CANARY).all()), "write past the output buffer"


def guarded_f32(src: torch.Tensor, misalign: int = 0):
    """Copy of src placed inside a larger buffer with NaN-free canaries; returns (full, view, lo)."""
    pad = 64
    d = src.numel()
    full = torch.full((d + 2 * pad + misalign,), 12345.0, dtype=src.dtype, device=src.device)
    lo = pad + misalign
    full[lo: lo + d] = src
    return full, full[lo: lo + d], lo


def check_guard(full: torch.Tensor, lo: int, d: int):
    f = full.cpu().float()
    assert bool((f[:lo] == 12345.0).all()), "write before the buffer"
    assert bool((f[lo + d:] == 12345.0).all()), "write past the buffer"


def oracle_step(grads_np, momenta_np, x_np, case):
    """One oracle iteration on host copies; returns the packed vote."""
    return oracle.fused_step(grads_np, momenta_np, x_np,
                             beta=case.beta if case.beta is not None else 0.0, lr=case.lr,
                             weight_decay=case.weight_decay, flip_mask=case.flip_mask)
