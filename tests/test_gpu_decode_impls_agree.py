"""The two decode kernels -- the persistent pipelined one and the one-CTA-per-unit one -- against each
other on ALL units of full-size configurations over one full cycle (log fills 0..15).

The kernel is chosen per process (``DELTALOG_DECODE_IMPL``, read once), so each side runs in a child
process that stores what it produced; the parent compares: the appended keys and the lengths are
bit-exact, outputs, value-side factors and decay snapshots agree to 1e-5 (the two kernels sum in
different orders).  This is the comparison that sees a fault tied to a unit's position in a
persistent CTA's walk -- every one of the 4 096 / 8 192 units is looked at."""
import subprocess
import sys
import textwrap
from pathlib import Path

import pytest
import torch

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

CHILD = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    import torch
    import bench, workloads
    config, path = int(sys.argv[1]), sys.argv[2]
    wl, cap = workloads.CONFIGS[config], 16
    rig = bench.Rig(wl, cap, torch.device("cuda", 0))
    rig.reset_logs()
    outs = []
    for t in range(cap):
        rig.out = torch.empty_like(rig.out)
        rig.step(t) if t < cap - 1 else rig.decode(t, 0, chained=True)      # stop before the merge: the log stays
        outs.append(rig.out)
    torch.cuda.synchronize()
    assert all(s == 0 for s in rig.status())
    st = rig.states[0]
    torch.save({{"out": torch.stack(outs).cpu(), "K": st.K_log.cpu(), "U": st.U_log.cpu(), "L": st.decay_log.cpu(),
                "len": st.log_len.cpu()}}, path)
""")


def rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).abs().max() / b.abs().max())


@pytest.mark.parametrize("config", [1, 2])
def test_pipelined_and_one_cta_per_unit_kernels_agree_on_every_unit(config, tmp_path):
    import os

    res = {}
    for impl in (1, 2):
        path = tmp_path / f"impl{impl}.pt"
        env = dict(os.environ, DELTALOG_DECODE_IMPL=str(impl))
        proc = subprocess.run([sys.executable, "-c", CHILD.format(root=str(ROOT)), str(config), str(path)],
                              capture_output=True, text=True, timeout=900, env=env)
        assert proc.returncode == 0, proc.stderr[-3000:]
        res[impl] = torch.load(path)
    a, b = res[1], res[2]
    assert torch.equal(a["len"], b["len"]) and int(a["len"].min()) == 16
    assert torch.equal(a["K"].view(torch.int16), b["K"].view(torch.int16))
    for name in ("out", "U", "L"):
        e = rel(a[name], b[name])
        assert e <= 1e-5 if name != "out" else e <= 8e-3, f"{name}: {e:.3e}"   # outputs are bf16: one ulp apart at most
    # outputs compared where it matters: in fp32 they agree to 1e-5, after rounding to bf16 they may differ by one ulp
    diff = (a["out"].float() - b["out"].float()).abs()
    ulp = b["out"].float().abs() * 2.0 ** -7 + 2e-5 * float(b["out"].float().abs().max())
    assert bool((diff <= ulp).all())
    assert float((diff > 0).float().mean()) < 0.02          # and they rarely differ at all


FUSED_CHILD = textwrap.dedent("""
    import sys
    sys.path.insert(0, {root!r})
    import torch
    import bench, workloads
    config, path = int(sys.argv[1]), sys.argv[2]
    wl, cap = workloads.CONFIGS[config], 16
    rig = bench.Rig(wl, cap, torch.device("cuda", 0))
    rig.reset_logs()
    for t in range(cap):
        rig.decode(t, 0)
    rig.out = torch.empty_like(rig.out)
    rig.fused(cap)                          # folds the full logs and consumes one more token
    torch.cuda.synchronize()
    assert all(s == 0 for s in rig.status())
    st = rig.states[0]
    torch.save({{"out": rig.out.cpu(), "S": st.S_base.cpu(), "len": st.log_len.cpu()}}, path)
""")


@pytest.mark.parametrize("config", [1, 2, 3])
def test_resident_and_one_unit_per_cta_fused_step_kernels_are_bit_identical_on_every_unit(config, tmp_path):
    """The fused merge step has two kernels (``DELTALOG_MAT_PREFETCH``, read once per process): a resident CTA
    with the next unit's operands in flight, and one unit per CTA.  Every element sees the same operations in
    the same order in both, so all units' outputs and folded states must be bit-identical."""
    import os

    res = {}
    for impl in (0, 1):
        path = tmp_path / f"fused{impl}.pt"
        env = dict(os.environ, DELTALOG_MAT_PREFETCH=str(impl))
        proc = subprocess.run([sys.executable, "-c", FUSED_CHILD.format(root=str(ROOT)), str(config), str(path)],
                              capture_output=True, text=True, timeout=900, env=env)
        assert proc.returncode == 0, proc.stderr[-3000:]
        res[impl] = torch.load(path)
    a, b = res[0], res[1]
    assert int(a["len"].abs().max()) == 0 and int(b["len"].abs().max()) == 0
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))
    assert torch.equal(a["S"].view(torch.int32), b["S"].view(torch.int32))
