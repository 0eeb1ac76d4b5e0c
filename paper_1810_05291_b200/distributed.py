"""One worker of Algorithm 1 per GPU: the exchange of packed signs between the kernels.

With the M workers on M GPUs, an iteration of Algorithm 1 has exactly one exchange step: every
worker pushes the d sign bits of its momentum and receives the d bits of the vote (2 M d bits
per iteration over the whole system, Appendix B). Two layouts of that exchange are provided,
both carried by ``torch.distributed`` collectives (NCCL on GPUs); received words always land in
this GPU's own memory before a kernel reads them.

``allgather``  every worker receives all M packed vectors (d/8 bytes from each peer) and runs
               ``ss_vote_apply`` locally: one collective, (M-1) d/8 bytes received per worker.
``sharded``    the parameter server split across the workers (the future-work item of the
               paper's discussion section): worker r is the server for the r-th slice of the
               words. An all-to-all brings every worker's slice r to worker r, which votes on
               it (``ss_majority_vote``); an all-gather returns the voted slices, and
               ``ss_apply_vote`` updates the parameters: about 2 (M-1)/M d/8 bytes per worker.

``push``       the all-gather folded into the producing kernel: ``ss_signum_update_push`` stores
               each packed word straight into this worker's slot of every worker's receive
               buffer (plain peer stores over NVLink), a barrier across the workers follows, and
               ``ss_vote_apply`` reads the local receive buffer. ``connect_push`` sets up the
               peer addresses and the barrier (by default a one-element all-reduce in stream
               order); ``set_push_destinations`` takes them from the caller. Signum only.

``PackedExchange`` holds the buffers and the slice arithmetic and works on any device (the
multi-process CPU tests drive it over gloo); ``MajorityVoteWorker`` adds the kernels and needs
CUDA tensors. There is no CPU path for the arithmetic.
"""

from __future__ import annotations

from typing import List, Optional

import torch
import torch.distributed as dist


def packed_words(d: int) -> int:
    return (int(d) + 31) // 32


class PackedExchange:
    """Buffers and collectives for the packed sign words of one worker."""

    def __init__(self, d: int, world: int, rank: int, device, mode: str = "allgather", group=None,
                 collectives=None):
        if mode not in ("allgather", "sharded", "push"):
            raise ValueError("mode must be 'allgather', 'sharded' or 'push'")
        if world < 1 or not 0 <= rank < world or d < 0:
            raise ValueError("bad world/rank/d")
        self.d, self.world, self.rank, self.mode, self.group = int(d), world, rank, mode, group
        self.coll = collectives if collectives is not None else dist
        self.W = packed_words(d)
        # words per server slice, rounded up to 4 so that every worker's row of the gathered
        # buffer and every slice starts on a 16-byte boundary (the kernels' wide loads need it)
        self.slice_words = 4 * -(-max(self.W, 1) // (4 * world))
        self.W_pad = self.slice_words * world               # local buffer, padded with zero words
        kw = dict(dtype=torch.int32, device=device)
        self.local = torch.zeros(self.W_pad, **kw)          # this worker's packed sign(v)
        if mode in ("allgather", "push"):
            self.gathered = torch.zeros(world * self.W_pad, **kw)
        else:
            self.recv = torch.zeros(world * self.slice_words, **kw)
            self.vote_slice = torch.zeros(self.slice_words, **kw)
            self.vote_pad = torch.zeros(self.W_pad, **kw)

    # ---- views ------------------------------------------------------------------------------
    def local_words(self) -> torch.Tensor:
        """Where the worker-side kernel writes this worker's ceil(d/32) words."""
        return self.local[: self.W]

    def worker_rows(self) -> List[torch.Tensor]:
        """allgather mode, after gather(): worker m's packed vector, m = 0..M-1."""
        return [self.gathered[m * self.W_pad: m * self.W_pad + self.W] for m in range(self.world)]

    def slot(self, m: int) -> torch.Tensor:
        """push mode: the part of this worker's receive buffer that worker m writes."""
        return self.gathered[m * self.W_pad: m * self.W_pad + self.W]

    def slice_coordinates(self) -> int:
        """sharded mode: how many of the d coordinates fall in this worker's server slice."""
        first = 32 * self.rank * self.slice_words
        return max(0, min(self.d - first, 32 * self.slice_words))

    def slice_rows(self) -> List[torch.Tensor]:
        """sharded mode, after scatter_slices(): worker m's words of this worker's slice."""
        n = packed_words(self.slice_coordinates())
        return [self.recv[m * self.slice_words: m * self.slice_words + n] for m in range(self.world)]

    def slice_vote(self) -> torch.Tensor:
        """sharded mode: where the server-side kernel writes this slice's vote words."""
        return self.vote_slice[: packed_words(self.slice_coordinates())]

    def vote_words(self) -> torch.Tensor:
        """sharded mode, after gather_vote(): the packed vote of the whole vector."""
        return self.vote_pad[: self.W]

    # ---- collectives ------------------------------------------------------------------------
    def gather(self) -> None:
        self.coll.all_gather_into_tensor(self.gathered, self.local, group=self.group)

    def scatter_slices(self) -> None:
        self.coll.all_to_all_single(self.recv, self.local, group=self.group)

    def gather_vote(self) -> None:
        self.coll.all_gather_into_tensor(self.vote_pad, self.vote_slice, group=self.group)

    def bytes_received_per_step(self) -> int:
        """Bytes this worker receives from its peers per iteration (excludes its own share)."""
        if self.mode in ("allgather", "push"):
            return (self.world - 1) * self.W_pad * 4
        return 2 * (self.world - 1) * self.slice_words * 4


class MajorityVoteWorker:
    """Algorithm 1 as seen from one worker: momentum and sign packing of the local gradient,
    the exchange, then vote and parameter update. State (x, v) lives on this worker's GPU.

    ``kernels`` is the object whose ``ss_*`` functions do the arithmetic: by default the binding
    of the CUDA library (tensors must then be CUDA tensors; there is no CPU path). The host-side
    tests pass a stand-in so that the order of kernels and collectives can be driven on CPU ranks.
    ``on_phase`` (optional) is called with a label after every kernel or collective of a step has
    been enqueued -- the benchmark records a CUDA event there to split a step into kernel time
    and exchange time. ``layout`` (optional ``fusion.FlatLayout``): the parameter vector is a model's
    tensors back to back, each updated with its own learning rate and weight decay."""

    STATUS_RING = 256                # flag-ordered push: steps whose wait status is kept on the device

    def __init__(self, param: torch.Tensor, beta: Optional[float], lr: float,
                 weight_decay: float = 0.0, mode: str = "allgather", group=None, world=None,
                 rank=None, collectives=None, kernels=None, on_phase=None, layout=None):
        if kernels is None:
            from . import binding as kernels
            if not param.is_cuda:
                raise ValueError("MajorityVoteWorker needs CUDA tensors: the arithmetic has no CPU path")
            kernels.lib()
        self.B = kernels
        self.x = param
        self.d = param.numel()
        self.beta, self.lr, self.weight_decay = beta, float(lr), float(weight_decay)
        if world is None:
            world = dist.get_world_size(group)
        if rank is None:
            rank = dist.get_rank(group)
        self.momentum = torch.zeros_like(param) if beta is not None else None
        self.ex = PackedExchange(self.d, world, rank, param.device, mode, group, collectives)
        self.vote = torch.zeros(self.ex.W, dtype=torch.int32, device=param.device)
        self.push_dests = None
        self.barrier = None
        self.flags = None            # flag-ordered push: see set_flag_exchange
        self.epoch = 0
        self.checked_epoch = 0       # flag-ordered push: last step that check() has passed
        self.on_phase = on_phase
        # a fusion.FlatLayout of the parameter vector: the update then takes each tensor's own
        # learning rate and weight decay from its device table and lr / weight_decay are unused
        self.layout = layout
        if layout is not None and layout.d != self.d:
            raise ValueError("the layout describes %d coordinates, the parameter vector has %d" % (layout.d, self.d))
        if mode == "push" and beta is None:
            raise ValueError("push mode carries the momentum kernel: use it with Signum (beta set)")

    def _vote_apply(self, rows, flip_mask: int, stream) -> None:
        if self.layout is not None:
            self.B.ss_vote_apply_segments(rows, self.x, self.layout.segments_dev, self.layout.n_segments,
                                          flip_mask, self.vote, stream)
        else:
            self.B.ss_vote_apply(rows, self.x, self.lr, self.weight_decay, flip_mask, self.vote, stream)

    def _phase(self, label: str) -> None:
        if self.on_phase is not None:
            self.on_phase(label)

    def set_push_destinations(self, dests, barrier) -> None:
        """push mode: ``dests[m]`` is the address (tensor or int) of this worker's slot in worker
        m's receive buffer; ``barrier()`` must return only when every worker's push kernel has
        completed (or, if it is stream-ordered, must order everything enqueued after it behind
        every worker's push kernel), and is called again after the update so that no worker's next
        push overtakes another worker's reads."""
        if len(dests) != self.ex.world:
            raise ValueError("need one destination per worker")
        self.push_dests = list(dests)
        self.barrier = barrier

    def set_flag_exchange(self, recv_bufs, dests, flag_dests, flags_local, timeout_ns: int = 1_000_000_000,
                          signal_with_wait: bool = False) -> None:
        """push mode without any collective: the flag-ordered exchange of ``ss_flags_signal`` /
        ``ss_flags_wait``. ``recv_bufs`` are this worker's two receive buffers (used alternately by
        the parity of the step, world * W_pad words each); ``dests[parity][m]`` is the address
        (tensor or int) of this worker's slot in worker m's buffer of that parity;
        ``flag_dests[m]`` is worker m's flag array and ``flags_local`` this worker's own. After a
        step whose wait ran out of time the update is skipped as a whole; ``check()`` tells, for
        every step since the last check.
        ``signal_with_wait``: raise the flag in the launch that waits (``ss_flags_signal_wait``, one
        launch fewer per step) instead of right after the push; only for workers whose ``finish``
        follows their own ``pack_local`` without waiting for other workers' calls on this host."""
        world = self.ex.world
        if len(recv_bufs) != 2 or len(dests) != 2 or any(len(x) != world for x in dests) or len(flag_dests) != world:
            raise ValueError("need two receive buffers, two lists of one destination per worker, one flag array per worker")
        # one status word per step, in a ring: a step whose wait ran out stays on record until
        # check() has looked at it (finish() calls check() itself before it reuses a word)
        self.flags = dict(recv=list(recv_bufs), dests=[list(dests[0]), list(dests[1])], flag_dests=list(flag_dests),
                          local=flags_local, timeout_ns=int(timeout_ns), fused=bool(signal_with_wait),
                          status=torch.zeros(self.STATUS_RING, dtype=torch.int32, device=self.x.device))
        self.checked_epoch = self.epoch

    def step_status(self) -> torch.Tensor:
        """Flag-ordered push: the status word (a one-element view) of the current step."""
        slot = self.epoch % self.STATUS_RING
        return self.flags["status"][slot: slot + 1]

    def check(self) -> None:
        """Flag-ordered push: waits for the stream and raises if the wait of any step since the
        last successful check ran out of time (RuntimeError naming the first such step and the
        lowest worker whose packed signs had not arrived). The parameter update of such a step was
        skipped on this worker, so its replica no longer follows the others'."""
        self._check_through(self.epoch)

    def _check_through(self, last_epoch: int) -> None:
        if self.flags is None:
            return
        if self.x.is_cuda:
            torch.cuda.synchronize(self.x.device)
        ring = self.flags["status"].tolist()
        for epoch in range(self.checked_epoch + 1, last_epoch + 1):
            status = ring[epoch % self.STATUS_RING]
            if status != 0:
                raise RuntimeError("majority vote step %d: the packed signs of worker %d did not arrive within "
                                   "%.3f s; the parameter update of that step was skipped"
                                   % (epoch, status - 1, self.flags["timeout_ns"] * 1e-9))
        self.checked_epoch = last_epoch

    def connect_push(self, group=None, barrier: str = "collective", timeout_ns: int = 1_000_000_000) -> None:
        """push mode across GPUs: allocates the receive buffer in symmetric memory
        (``torch.distributed._symmetric_memory``), exchanges its addresses over ``group``, and
        points this worker's push at its own slot in every peer's buffer. Every worker of the
        group must call this once, after the process group exists.

        ``barrier="collective"`` (default): the barrier between the push and the reads is a
        one-element all-reduce of the process group (NCCL on GPUs), enqueued in stream order: it
        starts when this worker's push kernel has finished and completes only when every worker
        has reached it, and a worker that never arrives ends it with the process group's timeout
        error on the host. ``barrier="signal"``: the symmetric-memory handle's own barrier, a
        spin on a flag in the peers' signal pads inside a kernel, with the library's own timeout;
        lower latency, kept as an explicit choice. ``barrier="flags"``: no barrier and no collective
        at all: two receive buffers used alternately and one flag per worker, raised by
        ``ss_flags_signal`` after the push and awaited, for at most ``timeout_ns``, by
        ``ss_flags_wait`` before the vote (see ``set_flag_exchange``)."""
        import torch.distributed._symmetric_memory as symm
        if self.ex.mode != "push":
            raise RuntimeError("connect_push is for push mode")
        if barrier not in ("collective", "signal", "flags"):
            raise ValueError("barrier must be 'collective', 'signal' or 'flags'")
        group = group if group is not None else dist.group.WORLD
        ex = self.ex
        if barrier == "flags":
            n_buf = ex.world * ex.W_pad
            n_flags = self.B.SS_MAX_WORKERS
            buf = symm.empty(2 * n_buf + n_flags, dtype=torch.int32, device=self.x.device)
            buf.zero_()
            handle = symm.rendezvous(buf, group)
            self._symmetric = (buf, handle)
            base = [int(handle.buffer_ptrs[m]) for m in range(ex.world)]
            slot = ex.rank * ex.W_pad * 4
            dests = [[base[m] + parity * n_buf * 4 + slot for m in range(ex.world)] for parity in (0, 1)]
            flag_dests = [base[m] + 2 * n_buf * 4 for m in range(ex.world)]
            # every worker's buffers and flags are zero before anyone pushes: a host-side barrier,
            # once, at set-up
            if self.x.is_cuda:
                torch.cuda.synchronize(self.x.device)
            dist.barrier(group)
            self.set_flag_exchange([buf[:n_buf], buf[n_buf:2 * n_buf]], dests, flag_dests,
                                   buf[2 * n_buf: 2 * n_buf + n_flags], timeout_ns, signal_with_wait=True)
            return
        buf = symm.empty(ex.world * ex.W_pad, dtype=torch.int32, device=self.x.device)
        buf.zero_()
        handle = symm.rendezvous(buf, group)
        ex.gathered = buf
        slot_bytes = ex.W_pad * 4
        dests = [int(handle.buffer_ptrs[m]) + ex.rank * slot_bytes for m in range(ex.world)]
        self._symmetric = (buf, handle)
        if barrier == "signal":
            self.set_push_destinations(dests, handle.barrier)
        else:
            self.set_push_destinations(dests, collective_barrier(group, self.x.device, ex.coll))

    def pack_local(self, grad: torch.Tensor, stream=None) -> None:
        """Worker side: v <- (1 - beta) g + beta v, sign(v) packed into the send buffer."""
        if self.ex.mode == "push" and self.flags is not None:
            self.epoch += 1
            fl = self.flags
            self.B.ss_signum_update_push(grad, self.momentum, self.beta, fl["dests"][self.epoch & 1], stream)
            self._phase("kernel:pack")
            if not fl["fused"]:
                self.B.ss_flags_signal(fl["flag_dests"], self.ex.rank, self.epoch, stream)
                self._phase("exchange:signal")
            return
        if self.ex.mode == "push":
            if self.push_dests is None:
                raise RuntimeError("push mode: call set_push_destinations, set_flag_exchange or connect_push first")
            self.B.ss_signum_update_push(grad, self.momentum, self.beta, self.push_dests, stream)
        elif self.momentum is not None:
            self.B.ss_signum_update(grad, self.momentum, self.beta, self.ex.local_words(), stream)
        else:
            self.B.ss_sign_pack(grad, self.ex.local_words(), stream)
        self._phase("kernel:pack")

    def serve(self, flip_mask: int = 0, stream=None) -> None:
        """sharded mode: receive every worker's words of this worker's slice and vote on them
        (this worker acting as the parameter server of its slice). No-op in the other modes."""
        ex = self.ex
        if ex.mode != "sharded":
            return
        ex.scatter_slices()
        self._phase("exchange:all_to_all")
        n = ex.slice_coordinates()
        if n > 0:
            self.B.ss_majority_vote(ex.slice_rows(), n, flip_mask, ex.slice_vote(), stream)
        self._phase("kernel:vote")

    def finish(self, flip_mask: int = 0, stream=None) -> torch.Tensor:
        """Receive what the update needs (all packed vectors, or the voted slices), update the
        parameters, and return the packed vote of the whole vector."""
        B, ex = self.B, self.ex
        if ex.mode == "push" and self.flags is not None:
            fl = self.flags
            if self.epoch - self.checked_epoch >= self.STATUS_RING:
                self._check_through(self.epoch - 1)   # this step's word still holds an unchecked step's status
            status = self.step_status()
            ex.gathered = fl["recv"][self.epoch & 1]
            if fl["fused"]:
                B.ss_flags_signal_wait(fl["flag_dests"], ex.rank, fl["local"], ex.world, self.epoch,
                                       fl["timeout_ns"], status, stream)
            else:
                B.ss_flags_wait(fl["local"], ex.world, self.epoch, fl["timeout_ns"], status, stream)
            self._phase("exchange:wait")
            if self.layout is not None:
                B.ss_vote_apply_guarded_segments(ex.worker_rows(), self.x, self.layout.segments_dev,
                                                 self.layout.n_segments, flip_mask, self.vote, status, stream)
            else:
                B.ss_vote_apply_guarded(ex.worker_rows(), self.x, self.lr, self.weight_decay, flip_mask,
                                        self.vote, status, stream)
            self._phase("kernel:vote_apply")
            return self.vote
        if ex.mode == "push":
            self.barrier()
            self._phase("exchange:barrier")
            self._vote_apply(ex.worker_rows(), flip_mask, stream)
            self._phase("kernel:vote_apply")
            self.barrier()
            self._phase("exchange:barrier")
            return self.vote
        if ex.mode == "allgather":
            ex.gather()
            self._phase("exchange:all_gather")
            self._vote_apply(ex.worker_rows(), flip_mask, stream)
            self._phase("kernel:vote_apply")
            return self.vote
        ex.gather_vote()
        self._phase("exchange:all_gather")
        if self.layout is not None:
            B.ss_apply_vote_segments(self.x, ex.vote_words(), self.layout.segments_dev, self.layout.n_segments, stream)
        else:
            B.ss_apply_vote(self.x, ex.vote_words(), self.lr, self.weight_decay, stream)
        self._phase("kernel:apply")
        return ex.vote_words()

    def step(self, grad: torch.Tensor, flip_mask: int = 0, stream=None) -> torch.Tensor:
        """One iteration. Kernels run on the current stream (or ``stream``, which must then be
        the stream the collectives see as current)."""
        self._phase("start")
        self.pack_local(grad, stream)
        self.serve(flip_mask, stream)
        return self.finish(flip_mask, stream)


def collective_barrier(group, device, collectives=None):
    """A barrier made of a one-element all-reduce over ``group``: stream-ordered on GPUs (NCCL
    enqueues it behind the work already on the current stream and the stream waits for it), and
    bounded by the process group's timeout rather than by a device-side spin."""
    coll = collectives if collectives is not None else dist
    token = torch.zeros(1, dtype=torch.int32, device=device)

    def barrier() -> None:
        coll.all_reduce(token, group=group)

    return barrier
