"""Host-side logic of bench.py that needs no GPU: how a region of K steps is cut into graph segments
and how many merges it holds for any K (the step count is the driver's choice, not a multiple of the
capacity), the parser that turns an ncu capture into the DRAM-traffic record, and the reference arm."""
import json
import subprocess
import sys
from pathlib import Path

import pytest

import bench
from paper_2608_15533_b200 import build, ncu_traffic

ROOT = Path(__file__).resolve().parent.parent


@pytest.mark.parametrize("cap", [1, 3, 4, 8, 16, 32, 64])
@pytest.mark.parametrize("steps", [1, 7, 16, 20, 33, 256, 2048])
def test_a_region_of_any_length_is_cut_into_whole_graphs_plus_a_tail(cap, steps):
    g = bench.graph_steps(cap)
    assert g % cap == 0 and g % bench.Rig.RING == 0          # whole cycles, back at the start of the token ring
    n_full, tail = bench.segments(steps, g)
    assert n_full * g + tail == steps and 0 <= tail < g
    # a region that starts on empty logs merges after every cap-th step: simulate the fill counter
    fill = merges = 0
    for t in range(steps):
        assert fill < cap                                     # never a decode on a full log
        fill += 1
        if (t + 1) % cap == 0:
            merges, fill = merges + 1, 0
    assert merges == bench.merges_in(steps, cap)
    # every segment starts at the beginning of a cycle, so the tail may be captured from step 0
    assert (n_full * g) % cap == 0


def test_ncu_capture_parser_scales_units_and_groups_kernel_families(tmp_path):
    launches = ncu_traffic.parse(ROOT / "tests" / "golden" / "ncu_two_counters_sample.csv")
    assert len(launches) == 4
    k = ncu_traffic.summarise(launches)
    assert set(k) == {"decode", "merge"}                      # torch's own kernels are ignored
    assert k["decode"]["launches"] == 2
    assert k["decode"]["dram_read_bytes_per_launch"] == pytest.approx(220e6)
    assert k["decode"]["dram_write_bytes_per_launch"] == pytest.approx(7e6)
    assert k["merge"]["dram_read_bytes_per_launch"] == pytest.approx(300e6)
    out = tmp_path / "t.json"
    ncu_traffic.main(["--csv", str(ROOT / "tests" / "golden" / "ncu_two_counters_sample.csv"), "--config", "1", "--cap", "16",
                      "--command", "ncu ...", "--out", str(out), "--build-id", "aaaaaaaaaaaa"])
    ncu_traffic.main(["--csv", str(ROOT / "tests" / "golden" / "ncu_two_counters_sample.csv"), "--config", "2", "--cap", "16",
                      "--command", "ncu ...", "--out", str(out), "--build-id", "aaaaaaaaaaaa"])
    doc = json.loads(out.read_text())
    assert set(doc["captures"]) == {"config1_cap16_fp32", "config2_cap16_fp32"}
    # a capture of another build replaces the file: figures of different builds are never mixed
    ncu_traffic.main(["--csv", str(ROOT / "tests" / "golden" / "ncu_two_counters_sample.csv"), "--config", "3", "--cap", "16",
                      "--command", "ncu ...", "--out", str(out), "--build-id", "bbbbbbbbbbbb"])
    doc = json.loads(out.read_text())
    assert doc["build_id"] == "bbbbbbbbbbbb" and set(doc["captures"]) == {"config3_cap16_fp32"}


def test_the_library_carries_the_identifier_of_its_sources():
    import paper_2608_15533_b200 as dl

    build.build_library()
    assert dl.build_id() == build.source_id(build.extra_flags())
    assert len(dl.build_id()) == 12


def test_stale_traffic_record_is_not_reported(monkeypatch, tmp_path):
    class FakeLib:
        @staticmethod
        def build_id():
            return "cccccccccccc"

    stale = tmp_path / "dram_traffic.json"
    stale.write_text(json.dumps({"build_id": "dddddddddddd", "captures": {"config1_cap16_fp32": {"kernels": {}}}}))
    monkeypatch.setattr(ncu_traffic, "DEFAULT_OUT", stale)
    monkeypatch.setattr(ncu_traffic.load, "__defaults__", (stale,))
    kernels, why = bench.dram_traffic(FakeLib, 1, 16, "fp32")
    assert kernels is None and "dddddddddddd" in why


@pytest.mark.parametrize("args", [["--steps", "20", "--warmup", "5"], ["--steps", "3", "--warmup", "0", "--config", "3"]])
def test_reference_arm_prints_one_json_line(args):
    proc = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", *args],
                          capture_output=True, text=True, timeout=600)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [ln for ln in proc.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["unit"] == bench.UNIT
    assert line["value"] > 0 and line["steps"] == int(args[1]) and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"] == {"value": line["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"].startswith("configs[")
