"""The benchmark's output contract: the reference arm (CPU oracle) on a small d without a GPU, the
byte accounting that the roofline figures rest on, and, on a GPU, the keys of the main line."""
import json
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def _run(args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True,
                         text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_prints_one_line_without_a_gpu():
    r = _run(["--impl", "reference", "--steps", "2", "--warmup", "1", "--d", "100000"])
    assert r["impl"] == "reference" and r["unit"] == "params/s" and r["higher_is_better"] is True
    assert r["value"] > 0 and r["gpu_launches"] == 0 and r["vs_baseline"] is None
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["cores"] >= 1
    assert r["cpu_baseline"]["value"] == r["value"] == r["e2e"]["value"]
    assert r["e2e"]["h2d_bytes_per_step"] == 0 and r["e2e"]["d2h_bytes_per_step"] == 0
    assert r["config"]["M"] == 15 and r["config"]["d"] == 100000


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_algorithmic_bytes_of_the_named_workloads():
    # per coordinate: M gradients read, M momenta read and written, x read and written
    assert bench.algorithmic_bytes(bench.make_case("cfg3")) == 188 * 25_557_032 == 4_804_722_016
    assert bench.algorithmic_bytes(bench.make_case("cfg2")) == 36 * 61_100_840
    assert bench.algorithmic_bytes(bench.make_case("cfg4")) == 158 * 25_557_032
    assert bench.algorithmic_bytes(bench.make_case("cfg4tie")) == 168 * 25_557_032
    assert bench.algorithmic_bytes(bench.make_case("cfg1")) == 20 * (1 << 20)
    c = bench.make_case("cfg3")
    W4 = ((c.d + 31) // 32) * 4
    assert bench.entry_bytes(c, "vote") == 16 * W4
    assert bench.entry_bytes(c, "signum_update") == 12 * c.d + W4
    assert bench.entry_bytes(c, "apply") == 8 * c.d + W4
    assert bench.entry_bytes(c, "chain") == 15 * (12 * c.d + W4) + 16 * W4 + 8 * c.d + W4


def test_gpus_n_as_a_plain_process_starts_n_ranks():
    """`bench.py --gpus 2` with no launcher in the environment must become two ranks by itself; the
    CPU-only launch-check mode lets that run here: both ranks join a gloo group and rank 0 reports."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--mode", "launch-check"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert lines == [{"mode": "launch-check", "n_gpus": 2, "ranks_seen": 2, "gpus_requested": 2}]


def test_launcher_command_and_stub_runner():
    seen = []
    rc = bench.spawn_ranks(4, ["--gpus", "4", "--steps", "7", "--d", "1000"], run=lambda cmd: seen.append(cmd) or 5)
    assert rc == 5 and len(seen) == 1
    cmd = seen[0]
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and cmd[cmd.index("--nproc-per-node") + 1] == "4"
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert 0 < int(cmd[cmd.index("--master-port") + 1]) < 65536
    tail = cmd[cmd.index(os.path.join(ROOT, "bench.py")) + 1:]
    assert tail == ["--gpus", "4", "--steps", "7", "--coords", "1000"]     # --d is ambiguous to torchrun


def test_under_a_launcher_no_second_launch_happens(monkeypatch):
    # WORLD_SIZE in the environment = already one of N ranks: main() must not spawn again
    calls = []
    monkeypatch.setattr(bench, "spawn_ranks", lambda *a, **k: calls.append(a) or 0)
    monkeypatch.setattr(bench, "launch_check_mode", lambda args: calls.append("ran"))
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--mode", "launch-check"])
    bench.main()
    assert calls == ["ran"]


def test_clock_sampler_takes_uuid_entries(monkeypatch):
    monkeypatch.setenv("CUDA_VISIBLE_DEVICES", "GPU-3b1c9f3e-aaaa-bbbb-cccc-0123456789ab, MIG-1f2e")
    assert bench.smi_device_id(0) == "GPU-3b1c9f3e-aaaa-bbbb-cccc-0123456789ab"
    assert bench.smi_device_id(1) == "MIG-1f2e"
    monkeypatch.setenv("CUDA_VISIBLE_DEVICES", "3,5")
    assert bench.smi_device_id(1) == "5"
    monkeypatch.delenv("CUDA_VISIBLE_DEVICES")
    assert bench.smi_device_id(2) == "2"


def test_traffic_is_null_once_the_kernel_sources_have_changed(monkeypatch):
    case = bench.make_case("cfg3")
    key = (15, 4, True)
    rec = dict(bench.NCU_DRAM_BYTES_PER_COORD[key])
    monkeypatch.setitem(bench.NCU_DRAM_BYTES_PER_COORD, key, dict(rec, source_hash=bench.kernel_source_hash("f32")))
    traffic, note = bench.ncu_traffic(case)
    assert traffic == pytest.approx(rec["bytes_per_coord"] * case.d) and "scaled by d" in note
    monkeypatch.setitem(bench.NCU_DRAM_BYTES_PER_COORD, key, dict(rec, source_hash="0123456789abcdef"))
    traffic, note = bench.ncu_traffic(case)
    assert traffic is None and "changed" in note
    no_capture = bench.make_case("cfg2")
    assert bench.ncu_traffic(no_capture)[0] is None


@pytest.mark.gpu
@pytest.mark.parametrize("layout", ["allgather", "sharded", "push", "push:flags"])
def test_worker_per_gpu_mode_runs_on_one_rank(layout):
    extra = []
    if ":" in layout:
        layout, barrier = layout.split(":")
        extra = ["--push-barrier", barrier]
    r = _run(["--mode", "worker-per-gpu", "--layout", layout, "--steps", "4", "--warmup", "3", "--d", "1000008"] + extra)
    assert r["mode"] == "worker-per-gpu" and r["layout"] == layout and r["n_gpus"] == 1
    assert r["config"]["M"] == 1 and r["value"] > 0 and r["ms_per_step"] > 0
    assert r["kernel_ms_per_step"] > 0 and r["exchange_ms_per_step"] >= 0
    assert r["kernel_ms_per_step"] + r["exchange_ms_per_step"] <= r["ms_per_step"] * 1.05
    assert r["replicas_agree"] is True
    assert r["bytes_received_per_worker_per_step"] == 0          # a lone worker receives nothing
    assert r["paper_bits_per_iteration_whole_system"] == 2 * 1000008
    per_step = 3 if extra else {"allgather": 2, "sharded": 3, "push": 2}[layout]
    assert r["gpu_launches"] == per_step * 4


@pytest.mark.gpu
def test_main_line_has_the_contract_keys():
    r = _run(["--steps", "5", "--warmup", "3", "--d", "4000008"])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e",
                "gpu_launches", "clocks"):
        assert key in r, key
    assert r["n_gpus"] == 1 and r["steps"] == 5 and r["gpu_launches"] == 5 and r["scaling"] == "weak"
    rf = r["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    assert rf["algorithmic_bytes_per_launch"] == 188 * 4000008
    assert r["e2e"]["h2d_bytes_per_step"] == 15 * 4 * 4000008 and r["e2e"]["value"] < r["value"]
    assert r["cpu_baseline"]["kind"] == "oracle"
    assert r["ms_min"] <= r["ms_median"] <= r["ms_max"] and r["ms_min"] <= r["ms_per_step_second_pass"] * 1.01
    assert abs(r["ms_per_step_second_pass"] - r["ms_per_step"]) < 0.2 * r["ms_per_step"]
    assert "traffic_source" in rf and "result" in r["e2e"]
    assert r["clocks"]["samples"] >= 5 and r["ms_x_sm_mhz"] > 0
