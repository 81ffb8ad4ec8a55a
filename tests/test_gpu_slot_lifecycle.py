"""GPU tests of the slot hand-over (state-slot lifecycle of Section 4): a slot that is given to a new
request mid-cycle starts from the installed base with an empty log, and nothing else changes."""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, Recorded, f64, make_desc, oracle_for, out_tol, rel_err
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run(wl, cap, steps, reset_at=None, reset_rows=(), S_new=None, keep_base=False):
    """Split cycle over ``steps`` tokens; before step ``reset_at`` the rows in ``reset_rows`` are handed
    to new requests (``S_new`` installed, or the base kept when ``keep_base``)."""
    import paper_2608_15533_b200 as dl

    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    desc = make_desc(wl, cap, 1.0)
    state = dl.State(desc, S0.clone())
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    rec = Recorded(units=units)
    base_at_reset = None
    for t in range(steps):
        dl.merge(desc, state, only_if_full=True)
        if t == reset_at:
            idx = torch.tensor(list(reset_rows), dtype=torch.int32, device=DEV)
            base_at_reset = state.S_base[idx.long()].clone()
            dl.reset_slots(desc, state, slot_idx=idx, S_init=None if keep_base else S_new)
            assert int(state.log_len[idx.long()].abs().sum()) == 0
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
        rec.record_token(tok, out, wl)
    dl.merge(desc, state)
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    return rec, state, S0, bonus, base_at_reset


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("keep_base", [False, True])
def test_slot_handed_to_a_new_request_mid_cycle(op, keep_base):
    wl = Workload(f"lifecycle_op{op}", op, 6, 2, 128, 24, (4,))
    cap, steps, reset_at, rows = 4, 24, 7, (1, 4)          # step 7: three entries pending in every log
    S_new = torch.randn(len(rows), wl.H, wl.d, wl.d, generator=torch.Generator().manual_seed(5)).mul_(0.2).to(DEV)
    rec, state, S0, bonus, base_at = run(wl, cap, steps, reset_at, rows, S_new, keep_base)
    ref_plain, state_plain, _, _, _ = run(wl, cap, steps)
    out, out_plain = np.stack(rec.out), np.stack(ref_plain.out)
    units = rec.units
    other = [i for i, u in enumerate(units) if u[0] not in rows]
    moved = [i for i, u in enumerate(units) if u[0] in rows]
    # rows that were not handed over are bit-identical to a run without the hand-over
    assert np.array_equal(out[:, other], out_plain[:, other])
    for b in range(wl.batch):
        if b not in rows:
            assert torch.equal(state.S_base[b], state_plain.S_base[b])
    # before the hand-over the moved rows are the old requests
    assert np.array_equal(out[:reset_at, moved], out_plain[:reset_at, moved])
    # after it they are new requests starting from the installed base (or from the kept base alone)
    start_S = (base_at if keep_base else S_new)
    rec2 = Recorded(units=[units[i] for i in moved])
    for name in ("q", "k", "v", "g", "beta"):
        setattr(rec2, name, [x[moved] for x in getattr(rec, name)[reset_at:]])
    rec2.state_at = [steps - reset_at]
    S0u = np.stack([f64(start_S[rows.index(units[i][0]), units[i][1]]) for i in moved])
    bonus_u = np.stack([f64(bonus[units[i][1]]) for i in moved]) if bonus is not None else None
    ref = oracle_for(wl, rec2, S0u, bonus_u)
    assert rel_err(out[reset_at:, moved], ref["out"]) <= out_tol(wl)
    got = np.stack([f64(state.S_base[units[i][0], units[i][1]]) for i in moved])
    assert rel_err(got, ref["S"]) <= TOL_STATE


def test_reset_skips_padding_and_flags_bad_slots():
    import paper_2608_15533_b200 as dl

    wl = Workload("lifecycle_pad", GDN, 4, 2, 64, 4, (4,), num_slots=6)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4, 1.0)
    state = dl.State(desc, S0.clone())
    state.log_len.fill_(2)
    idx = torch.tensor([5, -1, 77, 0], dtype=torch.int32, device=DEV)
    S_new = torch.ones(4, wl.H, wl.d, wl.d, device=DEV)
    dl.reset_slots(desc, state, slot_idx=idx, S_init=S_new)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_BAD_SLOT
    assert state.log_len[:, 0].tolist() == [0, 2, 2, 2, 2, 0]
    for s in range(6):
        assert torch.equal(state.S_base[s], S_new[0] if s in (0, 5) else S0[s])
