"""Algorithm 1 as a ``torch.optim.Optimizer``: Signum (or signSGD) with majority vote, one worker
per process, over a model's own parameter tensors.

The model's parameters are moved into one flat vector (``fusion.FlatLayout``; Section 4 of the
paper merges tensors into one buffer before compression) and every ``p.data`` / ``p.grad`` becomes a
view of the flat parameter / gradient buffer, so that ``backward()`` accumulates straight into the
buffer the kernels read and one optimiser step is one pass of the hot path:

* one process (no process group, or a group of one): ``ss_fused_step_segments`` with M = 1;
* M processes: ``MajorityVoteWorker`` -- momentum and sign packing of the local gradient, the
  exchange of the packed signs (``allgather``, ``sharded`` or ``push``), vote and update with each
  tensor's own learning rate and weight decay.

Every replica applies the same vote to the same parameters, so the replicas stay bit-identical
without ever exchanging a parameter. This module moves no number itself: flattening, views and
hyper-parameter tables only; the arithmetic is in the kernels.
"""

from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist

from .distributed import MajorityVoteWorker
from .fusion import FlatLayout


class SignumVote(torch.optim.Optimizer):
    """``lr`` and ``weight_decay`` may differ per parameter group (they go to the per-tensor table
    the kernels read, and a scheduler may change ``lr`` between steps); ``momentum`` is the beta of
    Algorithm 1 and is one number for the whole model (``None``: signSGD, no momentum buffers).

    A parameter whose ``grad`` is ``None`` at ``step()`` votes with a zero gradient, i.e. +1 under
    the one-bit sign. ``zero_grad`` always zeroes in place: the gradients must stay views of the
    flat buffer. ``mode`` is the layout of the exchange between the workers (``"allgather"``,
    ``"sharded"``, or ``"push"``, which is connected over the process group at construction with
    ``push_barrier`` = ``"collective"``, ``"signal"`` or ``"flags"``; with ``"flags"`` call
    ``opt.worker.check()`` to learn of a step that a missing worker made this one skip). ``exchange``: run the worker-and-exchange
    path even in a group of one (default: only with more than one process). ``kernels`` /
    ``collectives`` replace the CUDA binding and ``torch.distributed`` (the host-side tests drive
    the optimiser on CPU ranks that way)."""

    def __init__(self, params, lr: float = 1e-4, momentum: Optional[float] = 0.9, weight_decay: float = 0.0,
                 mode: str = "allgather", group=None, world: Optional[int] = None, rank: Optional[int] = None,
                 kernels=None, collectives=None, exchange: Optional[bool] = None, push_barrier: str = "collective"):
        if lr < 0.0 or weight_decay < 0.0 or (momentum is not None and not 0.0 <= momentum < 1.0):
            raise ValueError("need lr >= 0, weight_decay >= 0 and 0 <= momentum < 1 (or None)")
        super().__init__(params, dict(lr=lr, weight_decay=weight_decay))
        if kernels is None:
            from . import binding as kernels
            kernels.lib()
        self.B = kernels
        self.beta = momentum
        tensors = [p for g in self.param_groups for p in g["params"]]
        if len(tensors) == 0:
            raise ValueError("no parameters")
        device = tensors[0].device
        for p in tensors:
            if p.dtype != torch.float32 or p.device != device:
                raise ValueError("all parameters must be float32 tensors on one device")
        if world is None:
            world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
        if rank is None:
            rank = dist.get_rank(group) if world > 1 else 0
        lrs, wds = self._hyperparameters()
        self.layout = FlatLayout([tuple(p.shape) for p in tensors], lrs, wds, device, kernels=kernels)
        self._table = (lrs, wds)
        self.flat_param = self.layout.flat()
        self.flat_grad = self.layout.flat()
        self.flat_momentum = self.layout.flat() if momentum is not None else None
        self._param_views = self.layout.views(self.flat_param)
        self._grad_views = self.layout.views(self.flat_grad)
        moms = self.layout.views(self.flat_momentum) if momentum is not None else [None] * len(tensors)
        with torch.no_grad():
            for p, pv, gv, mv in zip(tensors, self._param_views, self._grad_views, moms):
                pv.copy_(p.data)
                if p.grad is not None:
                    gv.copy_(p.grad)
                p.data = pv
                p.grad = gv
                if mv is not None:
                    self.state[p]["momentum_buffer"] = mv
        self._tensors = tensors
        self.vote = torch.zeros(self.B.ss_packed_words(self.layout.d), dtype=torch.int32, device=device)
        self.worker = None
        if world > 1 if exchange is None else exchange:
            self.worker = MajorityVoteWorker(self.flat_param, momentum, lr, weight_decay, mode, group, world, rank,
                                             collectives, kernels, layout=self.layout)
            if momentum is not None:
                self.worker.momentum = self.flat_momentum
            if mode == "push":
                if push_barrier not in ("collective", "signal", "flags"):
                    raise ValueError("push_barrier must be 'collective', 'signal' or 'flags'")
                self.worker.connect_push(group, barrier=push_barrier)

    def _hyperparameters(self):
        lrs, wds = [], []
        for g in self.param_groups:
            lrs += [float(g["lr"])] * len(g["params"])
            wds += [float(g["weight_decay"])] * len(g["params"])
        return lrs, wds

    def _gather_grads(self) -> None:
        """Gradients that are not (or no longer) views of the flat buffer are brought back into it."""
        for p, gv in zip(self._tensors, self._grad_views):
            if p.grad is None:
                gv.zero_()
                p.grad = gv
            elif p.grad.data_ptr() != gv.data_ptr() or p.grad.shape != gv.shape:
                gv.copy_(p.grad)
                p.grad = gv

    @torch.no_grad()
    def step(self, closure=None, flip_mask: int = 0):
        """``flip_mask``: the adversary model of Section 3.3 (bit m set: worker m sends inverted signs)."""
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        table = self._hyperparameters()
        if table != self._table:                 # a scheduler moved a learning rate
            self.layout.set_hyperparameters(*table)
            self._table = table
        self._gather_grads()
        if self.worker is None:
            moms = [self.flat_momentum] if self.flat_momentum is not None else None
            self.layout.step([self.flat_grad], moms, self.flat_param, self.beta if self.beta is not None else 0.0,
                             flip_mask, self.vote)
        else:
            self.vote = self.worker.step(self.flat_grad, flip_mask)
        return loss

    def zero_grad(self, set_to_none: bool = False) -> None:
        self.flat_grad.zero_()
        for p, gv in zip(self._tensors, self._grad_views):
            p.grad = gv

    def load_state_dict(self, state_dict) -> None:
        super().load_state_dict(state_dict)
        # the loaded momenta are fresh tensors: copy them into the flat buffer and point the state back at its views
        if self.flat_momentum is not None:
            for p, mv in zip(self._tensors, self.layout.views(self.flat_momentum)):
                loaded = self.state[p].get("momentum_buffer")
                if loaded is not None and loaded.data_ptr() != mv.data_ptr():
                    mv.copy_(loaded)
                self.state[p]["momentum_buffer"] = mv
        self._table = None                       # the groups' hyper-parameters may have changed: re-upload at the next step
