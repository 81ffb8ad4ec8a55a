"""Parity at the full benchmark sizes over ALL (sequence, head) units, in the launch configuration
bench.py times: one CUDA graph per cycle (16 decode launches, chained, and the merge), replayed.

Compared with the fp64 oracle, 512 units at a time: every output of every unit and step, the final
state of every unit, and the state right after every merge for 32 sequences x all heads.  The
persistent decode kernel gives each CTA some 28 units through rings whose stage and phase
arithmetic depends on the unit's position in the CTA's walk; only an all-units comparison sees a
fault that depends on that position.  Both error metrics are checked: the global-max-normalised one
of the parity bar, and the worst case over units of the same metric taken per unit."""
import numpy as np
import pytest
import torch

import bench
import workloads
from harness import TOL_OUT_BF16, TOL_STATE, f64

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)
CHUNK = 512
SNAP_SEQS = 32


def per_unit_err(x, ref, axes):
    """max|x - ref| / max|ref| taken per unit (``axes``: every axis but the unit axis); worst unit."""
    num = np.max(np.abs(x - ref), axis=axes)
    den = np.max(np.abs(ref), axis=axes)
    return float(np.max(num / np.where(den > 0, den, 1.0)))


def global_err(x, ref):
    return float(np.max(np.abs(x - ref)) / np.max(np.abs(ref)))


@pytest.mark.parametrize("config", [1, 2, 3])
def test_every_unit_of_the_full_size_configuration(config):
    import oracle

    wl, cap, steps = workloads.CONFIGS[config], 16, 256
    rig = bench.Rig(wl, cap, DEV)
    N, d, H = wl.units, wl.d, wl.H
    S0 = rig.states[0].S_base.clone()
    outs = torch.empty(steps, wl.batch, H, d, dtype=wl.io_dtype, device=DEV)     # every output of every unit
    snaps = torch.empty(steps // cap, SNAP_SEQS, H, d, d, dtype=torch.float32, device=DEV)
    cycle_out = [torch.empty(wl.batch, H, d, dtype=wl.io_dtype, device=DEV) for _ in range(cap)]

    # one cycle as bench.py's region captures it, except that every step writes its own output buffer
    assert bench.graph_steps(cap) == cap
    rig.reset_logs()
    stream = torch.cuda.Stream(device=DEV)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for t in range(cap):
                rig.out = cycle_out[t]
                rig.step(t)
        for c in range(steps // cap):
            graph.replay()
            outs[c * cap:(c + 1) * cap].copy_(torch.stack(cycle_out))
            snaps[c].copy_(rig.states[0].S_base[:SNAP_SEQS])                  # the state right after the merge
    torch.cuda.synchronize()
    assert all(s == 0 for s in rig.status()) and int(rig.states[0].log_len.abs().sum()) == 0
    S_final = rig.states[0].S_base

    ring = rig.rings[0]
    bonus = rig.bonus[0]
    snap_at = list(range(cap, steps + 1, cap))
    t_idx = np.arange(steps) % rig.RING
    worst = dict(out=0.0, out_unit=0.0, state=0.0, state_unit=0.0, snap=0.0)
    for lo in range(0, N, CHUNK):
        hi = min(lo + CHUNK, N)
        n = hi - lo
        rows = lambda x: x.reshape(N, *x.shape[2:])[lo:hi]
        tok8 = {name: np.stack([f64(rows(tok[name])).reshape(n, -1) for tok in ring])
                for name in ("q", "k", "v", "g", "beta") if ring[0][name] is not None}
        with_snaps = hi <= SNAP_SEQS * H
        ref = oracle.eager_rollout(
            wl.op, f64(S0.reshape(N, d, d)[lo:hi]), tok8["q"][t_idx], tok8["k"][t_idx], tok8["v"][t_idx], tok8["g"][t_idx],
            beta=tok8["beta"][t_idx][..., 0] if "beta" in tok8 else None,
            bonus=np.tile(f64(bonus), (wl.batch, 1))[lo:hi] if bonus is not None else None,
            snapshot_at=snap_at if with_snaps else ())
        out = f64(outs.reshape(steps, N, d)[:, lo:hi])
        S = f64(S_final.reshape(N, d, d)[lo:hi])
        worst["out"] = max(worst["out"], global_err(out, ref["out"]))
        worst["out_unit"] = max(worst["out_unit"], per_unit_err(out, ref["out"], (0, 2)))
        worst["state"] = max(worst["state"], global_err(S, ref["S"]))
        worst["state_unit"] = max(worst["state_unit"], per_unit_err(S, ref["S"], (1, 2)))
        if with_snaps:
            got = f64(snaps.reshape(steps // cap, SNAP_SEQS * H, d, d)[:, lo:hi])
            for i in range(steps // cap):
                worst["snap"] = max(worst["snap"], global_err(got[i], ref["snapshots"][i]),
                                    per_unit_err(got[i], ref["snapshots"][i], (1, 2)))
    print(f"config {config}, all {N} units x {steps} steps: " + ", ".join(f"{k} {v:.2e}" for k, v in worst.items()))
    assert worst["out"] <= TOL_OUT_BF16 and worst["out_unit"] <= TOL_OUT_BF16
    assert worst["state"] <= TOL_STATE and worst["state_unit"] <= TOL_STATE and worst["snap"] <= TOL_STATE
    assert worst["snap"] > 0.0          # the snapshots were taken and compared
