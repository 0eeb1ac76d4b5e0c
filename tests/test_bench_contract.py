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
