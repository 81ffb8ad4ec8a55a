"""bench_studies.py (the paper's kernel-level studies on this hardware) in its ``--small`` mode: every
study runs through, prints one JSON object with the rows and fields its summary under ``profiles/``
is written from, and all timings are finite."""
import json
import math
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

EXPECT = {
    "m_sweep": ("rows", ("cap", "split_us_per_step", "paper_us_per_step", "fused_step_us", "write_reduction_vs_eager")),
    "state_size": ("rows", ("batch", "state_mib", "split_us_per_step", "eager_us_per_step", "speedup_split_vs_eager")),
    "precision": ("rows", ("variant", "cap", "us_per_step", "bytes_per_unit_step")),
    "multi_token": ("rows", ("T", "us_per_token", "bytes_per_unit_token")),
}


def run(*args):
    proc = subprocess.run([sys.executable, str(ROOT / "bench_studies.py"), *args], capture_output=True, text=True,
                          timeout=1200, cwd=str(ROOT))
    assert proc.returncode == 0, proc.stderr[-3000:]
    return [json.loads(ln) for ln in proc.stdout.splitlines() if ln.startswith("{")]


@pytest.mark.parametrize("study", sorted(EXPECT))
def test_study_runs_small_and_prints_its_rows(study):
    (res,) = run("--study", study, "--small", "--steps", "64")
    key, fields = EXPECT[study]
    assert res["study"] == study and len(res[key]) >= 2
    for row in res[key]:
        for f in fields:
            assert f in row, (study, f)
            if isinstance(row[f], float):
                assert math.isfinite(row[f]) and row[f] > 0, (study, f, row[f])


def test_phase_costs_small():
    (res,) = run("--study", "phases", "--small", "--steps", "64")
    assert len(res["decode_us_by_fill"]) == 16 and all(math.isfinite(x) and x > 0 for x in res["decode_us_by_fill"])
    assert res["merge_us"] > 0 and res["fused_step_us"] > 0 and res["decode_bytes_by_fill"][15] > res["decode_bytes_by_fill"][0]


def test_pipeline_stage_ablation_runs_both_kernels():
    (res,) = run("--study", "ablation", "--steps", "48")
    assert len(res["rows"]) == 2 and all(r["us_per_step"] > 0 and r["decode_us"] > 0 for r in res["rows"])
