"""Shapes whose per-unit log stage leaves little shared memory for the base ring of the persistent
decode kernel (per-key decay, head size 128, capacities towards 64).  Each chunk of a base tile has
its own producer warp, so the ring must hold at least one whole tile; where it cannot, the launch
falls back to one CTA per unit.  Either way the results must be those of the oracle: a wide batch
(many units per persistent CTA) over a full cycle at the capacity limit."""
import numpy as np
import pytest
import torch

from harness import oracle_for, out_tol, rel_err, run_deltalog, sample_units, TOL_STATE
from workloads import GDN, GLA, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("op,io,cap", [(KDA, torch.bfloat16, 64), (KDA, torch.bfloat16, 56), (KDA, torch.float32, 48),
                                       (KDA, torch.float32, 64), (GLA, torch.float32, 60), (RWKV6, torch.float32, 64),
                                       (GDN, torch.float32, 64), (KDA, torch.bfloat16, 40)])
def test_wide_batch_full_cycle_at_large_capacity(op, io, cap):
    wl = Workload(f"ring_{op}_{cap}", op, 80, 8, 128, cap + 9, (cap,), io_dtype=io)   # 640 units: > 4 per CTA
    units = sample_units(wl, 24)
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, generator_device="cuda")
    ref = oracle_for(wl, rec, S0u, bonus)
    out = np.stack(rec.out)
    assert rel_err(out, ref["out"]) <= out_tol(wl)
    assert rec.states and len(rec.states) == len(rec.state_at)
    for i, S in enumerate(rec.states):
        assert rel_err(S, ref["snapshots"][i]) <= TOL_STATE
    assert int(state.status.item()) == 0
