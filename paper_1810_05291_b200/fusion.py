"""Tensor fusion: many parameter tensors laid out back to back in one flat vector.

Section 4 of the paper notes that merging small tensors into one buffer before compression saved
compression and communication cost. Here that buffer is the flat vector the C ABI works on: a
``FlatLayout`` places a model's tensors one after another, hands out per-tensor views of any flat
buffer (parameters, one gradient buffer per worker, one momentum buffer per worker), and holds
the device table of per-tensor learning rate and weight decay that ``ss_fused_step_segments``
reads. This module only computes offsets and marshals the table; the arithmetic is in the kernels.
"""

from __future__ import annotations

from typing import List, Sequence

import torch

from . import binding as B


class FlatLayout:
    def __init__(self, shapes: Sequence[Sequence[int]], lrs: Sequence[float],
                 weight_decays: Sequence[float], device, align: int = 4, kernels=None):
        """``align``: every tensor starts at a multiple of this many coordinates (4 keeps fp32
        views 16-byte aligned; 1 packs them with no padding). Padding coordinates belong to the
        tensor before them and take its hyper-parameters. ``kernels``: the object whose ``ss_*``
        functions are called, by default the binding of the CUDA library (the host-side tests
        pass a stand-in)."""
        self.B = kernels if kernels is not None else B
        if not (len(shapes) == len(lrs) == len(weight_decays)) or len(shapes) == 0:
            raise ValueError("need one shape, lr and weight_decay per tensor")
        if align < 1:
            raise ValueError("align must be >= 1")
        self.shapes = [tuple(int(s) for s in sh) for sh in shapes]
        self.numels = [int(torch.Size(sh).numel()) for sh in self.shapes]
        self.begins: List[int] = []
        at = 0
        for n in self.numels:
            self.begins.append(at)
            at += -(-n // align) * align
        self.d = at
        self.device = torch.device(device)
        self.n_segments = len(self.shapes)
        self.segments_dev = self.B.segment_table(self.n_segments, self.device)
        self.set_hyperparameters(lrs, weight_decays)

    def set_hyperparameters(self, lrs: Sequence[float], weight_decays: Sequence[float], stream=None) -> None:
        """(Re)writes the device table, e.g. when a learning-rate schedule moves."""
        self.lrs = [float(v) for v in lrs]
        self.weight_decays = [float(v) for v in weight_decays]
        self.B.ss_segments_upload(self.begins, self.lrs, self.weight_decays, self.d, self.segments_dev, stream)

    def flat(self, dtype=torch.float32) -> torch.Tensor:
        return torch.zeros(self.d, dtype=dtype, device=self.device)

    def views(self, flat: torch.Tensor) -> List[torch.Tensor]:
        """Per-tensor views of a flat buffer laid out by this object."""
        if flat.numel() != self.d or flat.dim() != 1:
            raise ValueError("flat buffer must have %d elements" % self.d)
        return [flat[b: b + n].view(sh) for b, n, sh in zip(self.begins, self.numels, self.shapes)]

    def step(self, grads, momenta, param, beta: float, flip_mask: int = 0, vote_words_out=None,
             stream=None) -> None:
        """One iteration of Algorithm 1 over the whole model in one launch."""
        self.B.ss_fused_step_segments(grads, momenta, param, beta, self.segments_dev, self.n_segments,
                                 flip_mask, vote_words_out, stream)
