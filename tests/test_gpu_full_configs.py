"""Parity at the full benchmark sizes, in the launch configuration the benchmark times (one decode
call and one predicate-merge call per step over the whole batch).  The oracle follows a sample of
(sequence, head) units one by one; every output of those units and their state at every merge
boundary are compared.  Inputs are drawn on the device (the tensors are too large to draw on the
host in reasonable time); both sides receive the same bytes.
"""
import numpy as np
import pytest
import torch

import workloads
from harness import (TOL_STATE, Recorded, f64, make_desc, oracle_for, out_tol, rel_err, run_deltalog,
                     sample_units)
from test_gpu_parity import check_rollout
from workloads import CONFIGS

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("cap", CONFIGS[1].caps)
def test_config1_gdn_b128_h32_d128(cap):
    wl = CONFIGS[1]
    units = sample_units(wl, 16)
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, generator_device=DEV)
    assert len(rec.out) == 256 and len(rec.state_at) == 256 // cap
    e_out, e_state = check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))
    print(f"config1 cap={cap}: out {e_out:.2e} state {e_state:.2e}")
    assert int(state.status.item()) == 0


def test_config2_kda_b256_h32_d128():
    wl = CONFIGS[2]
    rec, state, S0u, bonus = run_deltalog(wl, 16, DEV, units=sample_units(wl, 16), generator_device=DEV)
    e_out, e_state = check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))
    print(f"config2: out {e_out:.2e} state {e_state:.2e}")
    assert int(state.status.item()) == 0


def test_config3_rwkv6_b256_h64_d64():
    wl = CONFIGS[3]
    rec, state, S0u, bonus = run_deltalog(wl, 16, DEV, units=sample_units(wl, 24), generator_device=DEV)
    e_out, e_state = check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))
    print(f"config3: out {e_out:.2e} state {e_state:.2e}")
    assert int(state.status.item()) == 0


def test_config4_serving_24_layers_slot_indexed_staggered():
    """24 layers resident at once (1 GiB of base state each), 512 rows addressed through a random
    slot permutation, every sequence at its own log fill so that about 1/16 of them merge at every
    step; 16 sampled slots x 2 heads per layer go through the oracle."""
    import paper_2608_15533_b200 as dl

    wl, cap = CONFIGS[4], 16
    free = torch.cuda.mem_get_info()[0]
    assert free > 40 * 2 ** 30, "needs the 24 GiB state pool plus logs resident"
    slot_idx = workloads.slot_permutation(wl).to(DEV)
    delay = ((cap - workloads.fill_offsets(wl, cap)) % cap).to(DEV)   # fill f_b at step cap <=> start at (cap-f_b)%cap
    all_steps = cap + wl.steps
    rows = sorted(np.random.default_rng(4).choice(wl.batch, 16, replace=False).tolist())
    units = [(b, h) for b in rows for h in (0, wl.H - 1)]
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    uslot = slot_idx[ub].long()
    desc = make_desc(wl, cap)
    layers = []
    for layer in range(wl.layers):
        src = workloads.TokenSource(wl, device=DEV, seed=layer)
        S0 = src.initial_state()
        rec = Recorded(units=units, start=[int(delay[b]) for b, _ in units])
        layers.append((src, dl.State(desc, S0), rec, f64(S0[uslot, uh])))
    fills_seen = set()
    for t in range(all_steps):
        step_slots = torch.where(delay <= t, slot_idx, torch.full_like(slot_idx, -1))
        for src, state, rec, _ in layers:
            dl.merge(desc, state, slot_idx=slot_idx, only_if_full=True)
            tok = src.token()
            out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                                 slot_idx=step_slots)
            rec.record_token(tok, out, wl)
        if t == cap:
            fills_seen = set(layers[0][1].log_len[slot_idx.long(), 0].cpu().tolist())
    assert len(fills_seen) == cap                                  # merges really are staggered over all phases
    worst_out = worst_state = 0.0
    for src, state, rec, S0u in layers:
        dl.merge(desc, state, slot_idx=slot_idx)
        rec.state_at, rec.states = [all_steps], [f64(state.S_base[uslot, uh])]
        ref = oracle_for(wl, rec, S0u, None)
        e_out, e_state = check_rollout(wl, rec, ref)
        worst_out, worst_state = max(worst_out, e_out), max(worst_state, e_state)
        assert int(state.status.item()) == 0
    print(f"config4: out {worst_out:.2e} state {worst_state:.2e}")
