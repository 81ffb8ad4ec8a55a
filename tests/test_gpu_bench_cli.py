"""bench.py as the driver runs it: a subprocess with arbitrary ``--steps`` / ``--warmup`` (not
multiples of the log capacity, shorter than one cycle, longer than one graph) must exit 0 and print
ONE JSON line that carries every key of the contract with finite numbers."""
import json
import math
import subprocess
import sys
import time
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def run_bench(*args, timeout=1500):
    t0 = time.perf_counter()
    proc = subprocess.run([sys.executable, str(ROOT / "bench.py"), *args], capture_output=True, text=True,
                          timeout=timeout, cwd=str(ROOT))
    wall = time.perf_counter() - t0
    assert proc.returncode == 0, f"bench.py {' '.join(args)} exited {proc.returncode}:\n{proc.stderr[-3000:]}"
    lines = [ln for ln in proc.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, proc.stdout[-2000:]
    return json.loads(lines[0]), wall


def finite(x):
    return isinstance(x, (int, float)) and math.isfinite(x)


def check_line(line, steps, wall, cap=16, extras=True):
    assert line["metric"] == "state-update (seq*head)-steps/s" and line["unit"] == "(seq*head)-steps/s"
    assert line["config"]["workload"].startswith("configs[1]") and line["dtype"] == "f32"
    assert line["steps"] == steps and line["warmup"] >= 3 and line["n_gpus"] == 1
    assert line["higher_is_better"] is True and line["scaling"] == "weak" and line["vs_baseline"] is None
    assert finite(line["value"]) and line["value"] > 0 and finite(line["ms_per_step"]) and line["ms_per_step"] > 0
    assert line["ms_per_step"] * steps * 1e-3 < wall
    assert line["config"]["merges_in_timed_region"] == steps // cap
    assert line["gpu_launches"] == steps + steps // cap
    r = line["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s"
    for key in ("achieved", "peak", "frac", "algorithmic_bytes_per_launch", "avg_launch_ms",
                "achieved_algorithmic_incl_l2", "frac_algorithmic_incl_l2"):
        assert finite(r[key]) and r[key] > 0, key
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert 0.2 < r["frac"] < 1.15
    assert (r["traffic"] is None) == (r["traffic_unavailable"] is not None)
    if r["traffic"] is not None:   # DRAM bytes can only be fewer than the algorithmic ones (L2 serves the rest)
        assert 0.5 * r["algorithmic_bytes_per_launch"] < r["traffic"] < 1.1 * r["algorithmic_bytes_per_launch"]
    am = line["amortized"]
    for key in ("decode_ms_per_launch", "merge_ms_per_launch", "cycle_ms_per_step_from_kernel_times",
                "algorithmic_gbs_incl_l2", "write_reduction_vs_eager", "bytes_written_per_unit_step"):
        assert finite(am[key]) and am[key] > 0, key
    e = line["e2e"]
    assert finite(e["value"]) and e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] <= 1.05 * line["value"]            # copies can only cost time
    c = line["clocks"]
    assert c["samples"] > 0 and finite(c["sm_mhz"]) and c["sm_mhz"] > 0
    if extras:
        b = line["cpu_baseline"]
        assert b["kind"] == "oracle" and finite(b["value"]) and b["value"] > 0 and b["cores"] >= 1
        assert finite(line["eager_kernel"]["ms_per_step"]) and finite(line["paper_cycle"]["ms_per_step"])
        assert set(line["capacity_sweep"]) == {"4", "8", "16", "32"}
        for row in line["capacity_sweep"].values():
            assert finite(row["ms_per_step"]) and row["write_reduction_vs_eager"] > 1


def test_the_drivers_command_line():
    line, wall = run_bench("--gpus", "1", "--steps", "20", "--warmup", "5")
    check_line(line, 20, wall)


@pytest.mark.parametrize("steps,warmup", [(7, 3), (33, 4), (16, 0)])
def test_any_step_count(steps, warmup):
    line, wall = run_bench("--steps", str(steps), "--warmup", str(warmup), "--no-extras")
    check_line(line, steps, wall, extras=False)


def test_plain_launch_mode_and_another_capacity():
    line, wall = run_bench("--steps", "21", "--warmup", "3", "--no-extras", "--no-graph", "--cap", "8")
    check_line(line, 21, wall, cap=8, extras=False)
    assert line["config"]["launch"] == "plain launches"


def test_reference_arm_on_the_gpu_box():
    line, _ = run_bench("--impl", "reference", "--gpus", "1", "--steps", "20", "--warmup", "5")
    assert line["impl"] == "reference" and finite(line["value"]) and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"
