#!/usr/bin/env python
"""Benchmark of the fused Signum step (momentum -> sign -> majority vote -> update, one kernel).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl ours|reference]
    python bench.py --mode worker-per-gpu --layout allgather|sharded|push [--gpus N]
    python bench.py --table named|sweep|<workloads> [--entries ...]

A step is one call of ss_fused_step over one batch of synthetic gradients: M = 15 workers,
d = 25,557,032 (ResNet-50-sized) fp32, per-worker momentum, beta = 0.9, lr = 1e-4. With more than
one rank every rank runs the same workload on its own GPU (the path shards by coordinate and needs
no collective), timing is the maximum over ranks, and rank 0 prints one JSON line. The ranks come
from a launcher (torch.distributed.run sets RANK / LOCAL_RANK / WORLD_SIZE) or, when --gpus N is
given to a plain process, from this script starting them itself.

--mode worker-per-gpu measures the other multi-GPU form, Algorithm 1 with one worker per GPU and
the packed signs exchanged between them, in three layouts of that exchange.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused pack+vote+apply params/s"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM bytes per coordinate (dram__bytes_read.sum + dram__bytes_write.sum) of the fused kernels,
# from ncu captures at d = 8,388,608 (larger than L2; traffic is proportional to d because every
# coordinate is touched exactly once). Keyed by (M, gradient bytes, momentum). Each entry carries
# the hash of the kernel sources at the time of the capture (kernel_source_hash below); when the
# sources have changed since, the entry no longer describes the kernel that runs and
# roofline.traffic is reported as null until the counters are taken again.
NCU_DRAM_BYTES_PER_COORD = {
    (15, 4, True): {"bytes_per_coord": (1.040224e9 + 487.41e6) / 8388608, "capture_d": 8388608,
                    "sources": "f32", "source_hash": "54a1c01e5932fd89"},
    (15, 2, True): {"bytes_per_coord": (788.586e6 + 483.21e6) / 8388608, "capture_d": 8388608,
                    "sources": "bf16", "source_hash": "16344c2aad055820"},
}
KERNEL_SOURCES = {
    "f32": ("step_kernel.cuh", "bitslice.cuh", "common.cuh"),
    "bf16": ("step_oct_kernel.cuh", "step_kernel.cuh", "bitslice.cuh", "common.cuh"),
}


def kernel_source_hash(which: str) -> str:
    """sha256 (first 16 hex digits) over the sources that define the fused kernel of a gradient dtype."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[which]:
        with open(os.path.join(ROOT, "paper_1810_05291_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def make_case(name: str, d_override=None):
    from paper_1810_05291_b200 import inputs
    if name == "cfg1":
        c = inputs.cfg1()
    elif name == "cfg2":
        c = inputs.cfg2()
    elif name == "cfg3":
        c = inputs.cfg3()
    elif name == "cfg4":
        c = inputs.cfg4()
    elif name == "cfg4tie":
        c = inputs.cfg4(tie_probe=True)
    elif name.startswith("sweep:"):          # sweep:<d>:<M>[:mom]
        parts = name.split(":")
        c = inputs.cfg5(int(parts[1]), int(parts[2]), momentum=len(parts) > 3)
    else:
        raise SystemExit("unknown workload %r" % name)
    if d_override:
        c.d = int(d_override)
    return c


def algorithmic_bytes(case) -> int:
    """Bytes one fused step must move: per coordinate, M gradients read, (with momentum) M
    momenta read and written, x read and written."""
    import torch
    gb = 4 if case.dtype == torch.float32 else 2
    per = case.M * gb + 8
    if case.beta is not None:
        per += case.M * 8
    return per * case.d


def ncu_traffic(case):
    """(bytes, note): DRAM bytes of one launch of the fused kernel on this workload, scaled by d
    from the recorded ncu capture of a smaller case of the same kernel; bytes is None when no
    capture is on record or the kernel sources have changed since it was taken."""
    import torch
    key = (case.M, 4 if case.dtype == torch.float32 else 2, case.beta is not None)
    rec = NCU_DRAM_BYTES_PER_COORD.get(key)
    if rec is None:
        return None, "no ncu capture on record for this kernel"
    now = kernel_source_hash(rec["sources"])
    if now != rec["source_hash"]:
        return None, ("kernel sources changed since the ncu capture (hash %s, capture %s): counters must be "
                      "taken again" % (now, rec["source_hash"]))
    return rec["bytes_per_coord"] * case.d, ("scaled by d from the recorded ncu capture at d=%d (sources %s)"
                                             % (rec["capture_d"], now))


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, torch copy read+write)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index          # what nvidia-smi -i accepts: an index or a GPU / MIG UUID
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1] or [l for (_, l) in self.lines]
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            p = [x.strip() for x in r.split(",")]
            if len(p) < 8:
                continue
            try:
                sm.append(float(p[0]))
                smax.append(float(p[1]))
                power.append(float(p[2]))
            except ValueError:
                continue
            for name, val in zip(names, p[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def time_oracle(case, steps: int, warmup: int, threads: int, budget_s: float = 12.0):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the first
    d_s coordinates of all M workers (every coordinate is independent), d_s chosen so that the
    run stays near budget_s seconds. Returns (params_per_s, d_s, threads_used, seconds_per_step)."""
    import numpy as np
    import torch

    import oracle
    from paper_1810_05291_b200 import inputs

    oracle.set_threads(threads)
    used = oracle.get_threads()
    probe_d = min(case.d, 1 << 21)

    def host_inputs(d_s):
        sub = make_case_like(case, d_s)
        grads = [to_host(g) for g in inputs.gradients(sub, "cpu", 0)]
        x = inputs.initial_params(sub, "cpu").numpy().copy()
        moms = [np.zeros(d_s, dtype=np.float32) for _ in range(sub.M)] if sub.beta is not None else None
        return sub, grads, moms, x

    def to_host(t):
        if t.dtype == torch.bfloat16:
            return t.view(torch.int16).numpy().view(np.uint16).copy()
        return t.numpy().copy()

    def run(sub, grads, moms, x, n):
        t0 = time.perf_counter()
        for _ in range(n):
            oracle.fused_step(grads, moms, x, sub.beta if sub.beta is not None else 0.0, sub.lr,
                              sub.weight_decay, sub.flip_mask)
        return (time.perf_counter() - t0) / n

    sub, grads, moms, x = host_inputs(probe_d)
    run(sub, grads, moms, x, 1)
    per_coord = run(sub, grads, moms, x, 2) / probe_d
    total_steps = max(1, steps + warmup)
    d_s = int(min(case.d, max(1 << 16, budget_s / (per_coord * total_steps))))
    if d_s < case.d:
        d_s = max(32, d_s - d_s % 32)
    if d_s != probe_d:
        sub, grads, moms, x = host_inputs(d_s)
    run(sub, grads, moms, x, max(1, warmup))
    sec = run(sub, grads, moms, x, max(1, steps))
    oracle.set_threads(1)
    return d_s / sec, d_s, used, sec


def make_case_like(case, d):
    import copy
    c = copy.copy(case)
    c.d = int(d)
    return c


def reference_arm(args) -> None:
    """The reference arm of this benchmark is the CPU oracle, timed as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    case = make_case(args.workload, args.d)
    cores = oracle.max_threads()
    value, d_s, used, sec = time_oracle(case, args.steps, args.warmup, cores)
    sample = "first %d of %d coordinates, all %d workers, per step" % (d_s, case.d, case.M)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3 * case.d / d_s,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": dtype_name(case), "data": "synthetic",
        "config": config_of(case, "host memory; CPU oracle"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def dtype_name(case) -> str:
    import torch
    return "f32" if case.dtype == torch.float32 else "bf16 gradients, f32 state"


def config_of(case, residency: str) -> dict:
    return {"workload": case.name, "M": case.M, "d": case.d, "beta": case.beta, "lr": case.lr,
            "weight_decay": case.weight_decay, "flip_mask": case.flip_mask,
            "entry_point": "ss_fused_step", "l2": residency}


# ---- per-entry-point table: every kernel of the path on the named workloads ------------------

def entry_bytes(case, entry: str) -> int:
    """Algorithmic bytes of one call of an entry point (what the method must move): gradients
    and fp32 state once each way they are needed, packed words at 4 bytes per 32 coordinates."""
    import torch
    gb = 4 if case.dtype == torch.float32 else 2
    d, M = case.d, case.M
    wb = ((d + 31) // 32) * 4
    mom = case.beta is not None
    if entry == "pack":
        return gb * d + wb
    if entry in ("signum_update", "signum_update_push"):
        return (gb + 8) * d + wb
    if entry == "vote":
        return (M + 1) * wb
    if entry == "apply":
        return 8 * d + wb
    if entry == "vote_apply":
        return M * wb + 8 * d
    if entry in ("fused", "fused_segments"):
        return algorithmic_bytes(case)
    tb = ((d + 15) // 16) * 4            # the ternary comparison codec: 2 bits per coordinate
    if entry == "absmax":
        return gb * d
    if entry == "ternary_pack":
        return gb * d + tb
    if entry == "ternary_unpack":
        return tb + 4 * d
    if entry == "chain":
        per_worker = entry_bytes(case, "signum_update" if mom else "pack")
        return M * per_worker + entry_bytes(case, "vote") + entry_bytes(case, "apply")
    if entry in ("chain_va", "chain_va_graph"):
        per_worker = entry_bytes(case, "signum_update" if mom else "pack")
        return M * per_worker + entry_bytes(case, "vote_apply")
    raise ValueError(entry)


def time_launches(fn, n: int, warmup: int, stream, flush=None):
    """Per-launch device times in ms: an event pair around every call of fn; when a flush buffer
    (larger than L2) is given it is overwritten and then read back between calls, outside the
    event pair, so that every call starts with an L2 that holds none of its data and no dirty
    lines whose write-back would be charged to it."""
    import torch

    def cold():
        flush.zero_()
        flush.max()

    for _ in range(warmup):
        if flush is not None:
            cold()
        fn()
    torch.cuda.synchronize()
    pairs = []
    for _ in range(n):
        if flush is not None:
            cold()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        pairs.append((a, b))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


def table_mode(args) -> None:
    """--table: one JSON line per (workload, entry point) with median and best launch time,
    achieved GB/s over the algorithmic bytes and the fraction of the measured copy bandwidth.
    Every call starts from a cold L2 (a 512 MB buffer is overwritten and read between calls)."""
    import torch

    from paper_1810_05291_b200 import binding as B
    from paper_1810_05291_b200 import inputs

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B.lib()
    if args.threads:
        B.ss_set_launch_option("threads", args.threads)
    if args.blocks_per_sm:
        B.ss_set_launch_option("blocks_per_sm", args.blocks_per_sm)
    stream = torch.cuda.current_stream()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    peak, peak_src = measured_peak()
    if args.table == "named":
        names = ["cfg1", "cfg2", "cfg3", "cfg4", "cfg4tie"]
        entries = ["pack", "signum_update", "vote", "apply", "vote_apply", "chain", "chain_va",
                   "chain_va_graph", "fused", "fused_segments"]
    elif args.table == "sweep":
        names = ["sweep:%d:%d" % (d, M) for d in inputs.SWEEP_D for M in inputs.SWEEP_M]
        entries = ["vote", "fused"]
    else:
        names = args.table.split(",")
        entries = ["pack", "signum_update", "vote", "apply", "vote_apply", "chain", "chain_va",
                   "chain_va_graph", "fused", "fused_segments"]
    if args.entries:
        entries = args.entries.split(",")
    rows = []
    for name in names:
        case = make_case(name, args.d)
        mom = case.beta is not None
        beta = case.beta if mom else 0.0
        grads = inputs.gradients(case, dev, 0)
        x = inputs.initial_params(case, dev)
        moms = inputs.zero_momenta(case, dev)
        W = B.ss_packed_words(case.d)
        packed = [torch.zeros(W, dtype=torch.int32, device=dev) for _ in range(case.M)]
        vote = torch.zeros(W, dtype=torch.int32, device=dev)
        for m in range(case.M):
            B.ss_sign_pack(grads[m], packed[m], stream)
        turn = [0]
        # a fused flat vector of 161 tensors (the number of parameter tensors of ResNet-50) at
        # seeded cut points, all with the workload's own lr and weight decay
        n_seg = 161
        cuts = torch.randint(1, max(2, case.d), (n_seg - 1,), generator=torch.Generator().manual_seed(5)).sort().values
        seg_begins = [0] + [int(c) for c in cuts]
        seg_table = B.segment_table(n_seg, dev)
        B.ss_segments_upload(seg_begins, [case.lr] * n_seg, [case.weight_decay] * n_seg, case.d, seg_table, stream)

        gmax = torch.zeros(1, device=dev)
        codes = torch.zeros(B.ss_ternary_words(case.d), dtype=torch.int32, device=dev)
        decoded = torch.empty(case.d, device=dev) if args.entries and "ternary_unpack" in entries else None
        B.ss_absmax(grads[0], gmax, stream)

        def call(entry):
            m = turn[0] % case.M
            turn[0] += 1
            if entry == "absmax":
                B.ss_absmax(grads[m], gmax, stream)
            elif entry == "ternary_pack":
                B.ss_ternary_pack(grads[m], gmax, 1000 + turn[0], codes, stream)
            elif entry == "ternary_unpack":
                B.ss_ternary_unpack(codes, gmax, decoded, stream)
            elif entry == "pack":
                B.ss_sign_pack(grads[m], packed[m], stream)
            elif entry == "signum_update":
                B.ss_signum_update(grads[m], moms[m], beta, packed[m], stream)
            elif entry == "signum_update_push":      # one destination: the same bytes as signum_update
                B.ss_signum_update_push(grads[m], moms[m], beta, [packed[m]], stream)
            elif entry == "vote":
                B.ss_majority_vote(packed, case.d, case.flip_mask, vote, stream)
            elif entry == "apply":
                B.ss_apply_vote(x, vote, case.lr, case.weight_decay, stream)
            elif entry == "fused":
                B.ss_fused_step(grads, moms, x, beta, case.lr, case.weight_decay, case.flip_mask,
                                vote, stream)
            elif entry == "fused_segments":
                B.ss_fused_step_segments(grads, moms, x, beta, seg_table, n_seg, case.flip_mask, vote, stream)
            elif entry == "vote_apply":
                B.ss_vote_apply(packed, x, case.lr, case.weight_decay, case.flip_mask, None, stream)
            elif entry == "chain_va":
                for k in range(case.M):
                    if mom:
                        B.ss_signum_update(grads[k], moms[k], beta, packed[k], stream)
                    else:
                        B.ss_sign_pack(grads[k], packed[k], stream)
                B.ss_vote_apply(packed, x, case.lr, case.weight_decay, case.flip_mask, None, stream)
            elif entry == "chain_va_graph":
                graph.replay()
            elif entry == "chain":
                for k in range(case.M):
                    if mom:
                        B.ss_signum_update(grads[k], moms[k], beta, packed[k], stream)
                    else:
                        B.ss_sign_pack(grads[k], packed[k], stream)
                B.ss_majority_vote(packed, case.d, case.flip_mask, vote, stream)
                B.ss_apply_vote(x, vote, case.lr, case.weight_decay, stream)

        # the unfused chain recorded once into a CUDA graph (one submission per iteration)
        graph = None
        if "chain_va_graph" in entries:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    cs = torch.cuda.current_stream()
                    for k in range(case.M):
                        if mom:
                            B.ss_signum_update(grads[k], moms[k], beta, packed[k], cs)
                        else:
                            B.ss_sign_pack(grads[k], packed[k], cs)
                    B.ss_vote_apply(packed, x, case.lr, case.weight_decay, case.flip_mask, None, cs)
            stream.wait_stream(side)

        for entry in entries:
            if entry in ("signum_update", "signum_update_push") and not mom:
                continue
            ms = time_launches(lambda: call(entry), args.steps, max(3, args.warmup), stream, flush)
            nbytes = entry_bytes(case, entry)
            med, best = statistics.median(ms), min(ms)
            row = {"table": args.table, "workload": case.name, "M": case.M, "d": case.d,
                   "dtype": dtype_name(case), "entry": entry, "launches": len(ms),
                   "ms_median": med, "ms_min": best, "algorithmic_bytes": nbytes,
                   "gbs_median": nbytes / (med * 1e-3) / 1e9, "gbs_best": nbytes / (best * 1e-3) / 1e9,
                   "frac_of_measured_copy": nbytes / (med * 1e-3) / 1e9 / peak,
                   "params_per_s": case.d / (med * 1e-3), "l2": "cold (512 MB written then read before every call)",
                   "peak": peak, "peak_source": peak_src}
            rows.append(row)
            print(json.dumps(row), flush=True)
        del grads, x, moms, packed, vote
        torch.cuda.empty_cache()
    print("| workload | entry | ms (median) | ms (min) | algorithmic MB | GB/s (median) | of measured copy |")
    print("|---|---|---|---|---|---|---|")
    for r in rows:
        print("| M=%d d=%d %s | %s | %.4f | %.4f | %.1f | %.0f | %.3f |" % (
            r["M"], r["d"], "bf16" if r["dtype"].startswith("bf16") else "f32", r["entry"],
            r["ms_median"], r["ms_min"], r["algorithmic_bytes"] / 1e6, r["gbs_median"],
            r["frac_of_measured_copy"]))


def smi_device_id(local_rank: int) -> str:
    """The id nvidia-smi knows this rank's GPU by: the rank's entry of CUDA_VISIBLE_DEVICES (an
    index or a GPU-/MIG- UUID, passed on as text) or, without that variable, the local rank."""
    vis = [v.strip() for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v.strip()]
    if local_rank < len(vis):
        return vis[local_rank]
    return str(local_rank)


def free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def launch_command(n_ranks: int, argv, port: int):
    """The command that runs this script as n_ranks processes on one node, one GPU each."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_ranks),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def spawn_ranks(n_ranks: int, argv, run=subprocess.call) -> int:
    """`bench.py --gpus N` started as a plain process: start the N ranks (the script itself under
    torch.distributed.run, which sets RANK / LOCAL_RANK / WORLD_SIZE) and pass on their exit code.
    --d is respelt --coords, the form torchrun's own parser leaves alone."""
    argv = ["--coords" if a == "--d" else a for a in argv]
    return run(launch_command(n_ranks, argv, free_port()))


def launch_check_mode(args) -> None:
    """--mode launch-check: every rank joins a gloo group on the CPU, the ranks are counted with an
    all-reduce and rank 0 prints one line. Exercises the launcher without a GPU."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    seen = world
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
        t = torch.ones(1, dtype=torch.int64)
        dist.all_reduce(t)
        seen = int(t.item())
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"mode": "launch-check", "n_gpus": world, "ranks_seen": seen,
                          "gpus_requested": args.gpus}), flush=True)


def timed_launches(step, steps: int, stream, barrier, per_launch: bool = False):
    """EXACTLY `steps` calls of step() between a barrier + synchronize on both sides, timed by one
    pair of CUDA events on the launching stream. With per_launch an event is also recorded after
    every call, which gives the duration of every single launch from the same region.
    Returns (total_ms, [per-launch ms] or None, host time at start, host time at end)."""
    import torch
    n_ev = steps + 1 if per_launch else 2
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_ev)]
    barrier()
    t0 = time.time()
    ev[0].record(stream)
    for i in range(steps):
        step()
        if per_launch:
            ev[i + 1].record(stream)
    if not per_launch:
        ev[1].record(stream)
    barrier()
    t1 = time.time()
    each = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)] if per_launch else None
    return ev[0].elapsed_time(ev[-1]), each, t0, t1


def keep_busy(step, seconds: float) -> None:
    """Runs step() back to back for about `seconds`, so that the clock samples taken around the
    timed region (itself too short for nvidia-smi to see) are samples of the GPU under this very load."""
    import torch
    t = time.time()
    while time.time() - t < seconds:
        for _ in range(50):
            step()
        torch.cuda.synchronize()


def spread(ms) -> dict:
    return {"ms_median": statistics.median(ms), "ms_min": min(ms), "ms_max": max(ms)}


def init_ranks():
    """(world, rank, local_rank, device) from the launcher's environment; NCCL group when world > 1."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    return world, rank, local_rank, dev


def fused_mode(args) -> None:
    """The default mode: one ss_fused_step per step on every rank's own coordinate shard."""
    import torch
    import torch.distributed as dist

    from paper_1810_05291_b200 import binding as B
    from paper_1810_05291_b200 import inputs, sharding

    world, rank, local_rank, dev = init_ranks()
    B.lib()  # fail here, loudly, if the CUDA library is missing
    if args.threads:
        B.ss_set_launch_option("threads", args.threads)
    if args.blocks_per_sm:
        B.ss_set_launch_option("blocks_per_sm", args.blocks_per_sm)

    case = make_case(args.workload, args.d)
    case.cfg = case.cfg * 100 + rank  # every rank holds its own shard of coordinates: distinct data
    grads = inputs.gradients(case, dev, 0)
    x = inputs.initial_params(case, dev)
    moms = inputs.zero_momenta(case, dev)
    vote = torch.zeros(B.ss_packed_words(case.d), dtype=torch.int32, device=dev)
    beta = case.beta if case.beta is not None else 0.0
    stream = torch.cuda.current_stream()

    def step():
        B.ss_fused_step(grads, moms, x, beta, case.lr, case.weight_decay, case.flip_mask, vote, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(smi_device_id(local_rank))
    busy = 0.0 if args.profile else 0.6
    if not args.profile:
        sampler.start()
        keep_busy(step, busy)          # the same kernel, back to back, before ...
    ms_total, _, t0, t1 = timed_launches(step, args.steps, stream, barrier)
    # the same K launches once more, straight after, now with an event after every launch: the
    # spread of single launches, and a second total to hold against the first
    ms_again, per_launch, _, t1 = timed_launches(step, args.steps, stream, barrier, per_launch=True)
    if not args.profile:
        keep_busy(step, busy)          # ... and after the timed launches
    clocks = (sampler.stop(t0 - 0.8 * busy, t1 + 0.8 * busy) if not args.profile
              else {"sm_mhz": None, "reasons": ["not sampled (--profile)"]})
    if not args.profile:
        clocks["window"] = ("samples every 50 ms while the same kernel runs back to back from %.1f s before "
                            "to %.1f s after the timed launches" % (busy, busy))

    ms_total = sharding.max_over_ranks(ms_total, dev)
    ms_step = ms_total / args.steps
    value = world * case.d / (ms_step * 1e-3)

    # ---- end to end: gradients start in pinned host memory, packed vote returns to the host ----
    e2e = None
    if not args.no_e2e:
        host = [g.cpu().pin_memory() for g in grads]
        hv = torch.zeros(vote.numel(), dtype=torch.int32).pin_memory()
        n_e2e = max(3, min(args.steps, 10))

        def step_host():
            B.ss_fused_step_host(host, grads, moms, x, beta, case.lr, case.weight_decay,
                                 case.flip_mask, vote, hv, stream)

        for _ in range(2):
            step_host()
        ms_e2e, per_e2e, _, _ = timed_launches(step_host, n_e2e, stream, barrier, per_launch=True)
        ms_e2e = sharding.max_over_ranks(ms_e2e, dev)
        e2e = {"value": world * case.d / (ms_e2e / n_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": sum(h.numel() * h.element_size() for h in host),
               "d2h_bytes_per_step": hv.numel() * 4, "steps": n_e2e,
               "ms_per_step": ms_e2e / n_e2e, "entry_point": "ss_fused_step_host",
               "result": "packed vote; x and v stay on the device"}
        e2e.update(spread(per_e2e))
        del host

    if rank == 0:
        abytes = algorithmic_bytes(case)
        peak, peak_src = measured_peak()
        achieved = abytes / (ms_step * 1e-3) / 1e9
        traffic, traffic_note = ncu_traffic(case)
        sm_mhz = clocks.get("sm_mhz")
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype_name(case), "data": "synthetic",
            "config": config_of(case, "inputs %.2f GB per step, far larger than the 126 MB L2; no flush"
                                % (abytes / 1e9)),
            "hbm_gbs": achieved, "pct_of_nominal_8tbs": 100.0 * achieved / NOMINAL_HBM_GBS,
            "gradient_elements_per_s": value * case.M,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": traffic, "traffic_source": traffic_note,
                         "peak_source": peak_src,
                         "frac_note": "the peak is a measured copy rate (1 read : 1 write), not a ceiling; "
                                      "a stream with a larger share of reads can exceed it",
                         "kernel": "%s<M=%d,%s,momentum=%s,apply>" % (
                             "step_vec_kernel" if case.dtype == torch.float32 else "step_oct_bf16_kernel",
                             case.M, "f32" if case.dtype == torch.float32 else "bf16",
                             "yes" if case.beta is not None else "no"),
                         "algorithmic_bytes_per_launch": abytes,
                         "launch_ms": ms_step},
            "gpu_launches": args.steps,
            "clocks": clocks,
            "ms_x_sm_mhz": ms_step * sm_mhz if sm_mhz else None,
        }
        line.update(spread(per_launch))   # rank 0's own launches, one event pair each
        line["per_launch"] = ("ms_median / ms_min / ms_max: a second pass of the same %d launches right after the "
                              "timed region, an event after every launch; its total / steps = %.6f ms"
                              % (args.steps, ms_again / args.steps))
        line["ms_per_step_second_pass"] = ms_again / args.steps
        if e2e is not None:
            line["e2e"] = e2e
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            cores = oracle.max_threads()
            v_all, d_s, used, _ = time_oracle(case, 3, 1, cores, budget_s=8.0)
            v_one, d_1, _, _ = time_oracle(case, 2, 1, 1, budget_s=8.0)
            line["cpu_baseline"] = {
                "value": v_all, "unit": UNIT, "cores": used, "kind": "oracle",
                "sample": "first %d of %d coordinates, all %d workers, 3 timed steps" % (d_s, case.d, case.M),
                "value_1_thread": v_one,
                "sample_1_thread": "first %d coordinates, 2 timed steps" % d_1}
        print(json.dumps(line), flush=True)

    if world > 1:
        dist.destroy_process_group()


def worker_per_gpu_mode(args) -> None:
    """--mode worker-per-gpu: Algorithm 1 with one worker per GPU (M = number of ranks). Every rank
    owns one gradient buffer, its momentum and a replica of x; a step is MajorityVoteWorker.step:
    momentum + sign packing of the local gradient, the exchange of packed signs in the chosen layout,
    vote and parameter update. Prints ms per step, params/s, the bytes each worker receives per step
    beside Appendix B's count, and the split of a step into kernel time and exchange time."""
    import torch
    import torch.distributed as dist

    from paper_1810_05291_b200 import binding as B
    from paper_1810_05291_b200 import inputs, sharding
    from paper_1810_05291_b200.distributed import MajorityVoteWorker

    world, rank, local_rank, dev = init_ranks()
    if world == 1 and not dist.is_initialized():      # one-rank NCCL group: the real collectives, alone
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(free_port()))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    B.lib()
    case = make_case(args.workload, args.d)
    if case.beta is None and args.layout == "push":
        raise SystemExit("the push layout carries the momentum kernel: use a workload with momentum")
    case.M = world
    stream = torch.cuda.current_stream()
    s = inputs.signal(case, dev, 0)
    grad = inputs.worker_gradient(case, rank, dev, 0, s)     # this worker's mini-batch gradient
    del s
    x = inputs.initial_params(case, dev)                     # same seed on every rank: one replica each
    marks = []

    def on_phase(label):
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        marks.append((label, e))

    worker = MajorityVoteWorker(x, case.beta, case.lr, case.weight_decay, args.layout, on_phase=on_phase)
    if args.layout == "push":
        worker.connect_push(barrier=args.push_barrier)

    def step():
        worker.step(grad, case.flip_mask & ((1 << world) - 1))

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    del marks[:]
    ms_total, per_step, _, _ = timed_launches(step, args.steps, stream, barrier, per_launch=True)
    # split: time between consecutive marks of a step goes to the phase that the later mark names
    kernel_ms = exchange_ms = 0.0
    phases = {}
    for (la, ea), (lb, eb) in zip(marks, marks[1:]):
        if lb == "start":
            continue
        dt = ea.elapsed_time(eb)
        phases[lb] = phases.get(lb, 0.0) + dt
        if lb.startswith("kernel:"):
            kernel_ms += dt
        else:
            exchange_ms += dt
    ours = ("kernel:", "exchange:signal", "exchange:wait")     # phases that are launches of this library's kernels
    launches_per_step = sum(1 for (l, _) in marks if l.startswith(ours)) // max(1, args.steps)
    worker.check()
    ms_total = sharding.max_over_ranks(ms_total, dev)
    kernel_ms = sharding.max_over_ranks(kernel_ms, dev)
    exchange_ms = sharding.max_over_ranks(exchange_ms, dev)
    ms_step = ms_total / args.steps
    # Algorithm 1 keeps one copy of x per worker and every worker applies the same vote: after any
    # number of steps all replicas must hold the same bits. Compare a digest of x across the ranks.
    digest = torch.stack([x.view(torch.int32).sum(dtype=torch.int64),
                          (x.view(torch.int32)[::97].to(torch.int64) * 31).sum()])
    digests = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(digests, digest)
    replicas_agree = all(bool(torch.equal(t, digests[0])) for t in digests)
    if rank == 0:
        W4 = ((case.d + 31) // 32) * 4
        paper_bits = 2 * world * case.d                      # Appendix B: 2 M d bits per iteration, whole system
        line = {
            "mode": "worker-per-gpu", "layout": args.layout, "metric": "majority-vote step params/s",
            "value": case.d / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong",
            "dtype": dtype_name(case), "data": "synthetic",
            "config": {"workload": case.name, "M": world, "d": case.d, "beta": case.beta, "lr": case.lr,
                       "layout": args.layout,
                       "push_barrier": args.push_barrier if args.layout == "push" else None},
            "kernel_ms_per_step": kernel_ms / args.steps, "exchange_ms_per_step": exchange_ms / args.steps,
            "phases_ms_per_step": {k: v / args.steps for k, v in sorted(phases.items())},
            "bytes_received_per_worker_per_step": worker.ex.bytes_received_per_step(),
            "bytes_received_allgather_formula": (world - 1) * W4,
            "bytes_received_sharded_formula": 2 * (world - 1) * W4 // world,
            "paper_bits_per_iteration_whole_system": paper_bits,
            "gpu_launches": launches_per_step * args.steps,
            "replicas_agree": replicas_agree,
            "note": ("M = number of ranks: every rank is one worker of Algorithm 1 with its own replica of x; "
                     "params/s counts the d parameters once"),
        }
        line.update(spread(per_step))
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()
    if not replicas_agree:
        raise SystemExit("worker-per-gpu: the workers' copies of x differ after %d steps" % (args.steps + args.warmup))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--d", "--coords", dest="d", type=int, default=None,
                    help="override the coordinate count (tests, profiling); --coords is the spelling to use "
                         "under torchrun, whose own parser finds --d ambiguous")
    ap.add_argument("--mode", default="fused", choices=["fused", "worker-per-gpu", "launch-check"],
                    help="fused: ss_fused_step on every rank's coordinate shard (the headline number); "
                         "worker-per-gpu: one worker of Algorithm 1 per GPU with the packed-sign exchange; "
                         "launch-check: CPU-only check of the multi-rank launcher")
    ap.add_argument("--layout", default="allgather", choices=["allgather", "sharded", "push"],
                    help="worker-per-gpu: how the packed signs are exchanged")
    ap.add_argument("--push-barrier", default="collective", choices=["collective", "signal", "flags"],
                    help="worker-per-gpu, push layout: what orders the push before the reads: a one-element "
                         "all-reduce (collective), the symmetric-memory signal barrier (signal), or the library's "
                         "own flags with a bounded wait and no collective at all (flags)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under a profiler: no clock sampling, no end-to-end and CPU legs")
    ap.add_argument("--table", default=None,
                    help="time every entry point: 'named' (cfg1-4), 'sweep' (the d x M sweep) or a "
                         "comma-separated list of workloads; one JSON line per row, then a table")
    ap.add_argument("--entries", default=None,
                    help="with --table: comma-separated entry points to time instead of the table's own list")
    ap.add_argument("--threads", type=int, default=0, help="launch-shape override: block size")
    ap.add_argument("--blocks-per-sm", type=int, default=0, help="launch-shape override")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = True

    if args.impl == "reference":
        reference_arm(args)
        return
    if args.table:
        table_mode(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: become N ranks, one GPU each
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.mode == "launch-check":
        launch_check_mode(args)
    elif args.mode == "worker-per-gpu":
        worker_per_gpu_mode(args)
    else:
        fused_mode(args)


if __name__ == "__main__":
    main()
