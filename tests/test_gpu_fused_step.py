"""GPU parity of the fused merge step (Algorithm 1, else-branch; Eq. 5 with the current-token term),
called through the C ABI, against the fp64 CPU oracle on the same seeded inputs.  Bars as in
test_gpu_parity.py: fp32 state 1e-4, bf16 outputs 2e-2, fp32 outputs 1e-4."""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, f64, make_desc, materialize_units, oracle_for, out_tol, rel_err, run_deltalog
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small(op, d, io, batch=3, H=2, steps=40, **kw) -> Workload:
    return Workload(f"small_op{op}_d{d}", op, batch, H, d, steps, (1,), io_dtype=io, **kw)


def all_units(wl):
    return [(b, h) for b in range(wl.batch) for h in range(wl.H)]


def check(wl, rec, ref):
    out = np.stack(rec.out)
    mask = ~np.isnan(ref["out"])
    assert mask.any()
    e_out = rel_err(np.where(mask, out, 0.0), np.where(mask, ref["out"], 0.0))
    assert e_out <= out_tol(wl), f"output error {e_out:.3e}"
    assert rec.states and len(rec.states) == len(rec.state_at)
    worst = max(rel_err(S, ref["snapshots"][i]) for i, S in enumerate(rec.states))
    assert worst <= TOL_STATE, f"state error {worst:.3e}"


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("io", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("cap", [1, 3, 8])
def test_paper_cycle_invariant_every_step(op, d, io, cap):
    """cap appends, then one step that consumes a token and materialises; the state represented
    by base + log equals the eager recurrence after every token, and the cycle has the paper's
    period cap + 1."""
    wl = small(op, d, io, steps=28)
    units = all_units(wl)
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    mats, lens = [], []

    def hook(t, state, tok, out):
        mats.append(materialize_units(state, wl, ub, uh))
        lens.append(state.log_len[ub, uh].cpu().numpy().copy())

    scale = 0.5 if op != RWKV6 else 1.0
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, scale=scale, every_step_hook=hook,
                                          cycle="paper")
    for t, L in enumerate(lens):
        assert (L == (t + 1) % (cap + 1)).all()
    rec.state_at = list(range(1, wl.steps + 1))
    rec.states = mats
    check(wl, rec, oracle_for(wl, rec, S0u, bonus, scale=scale))
    assert int(state.status.item()) == 0


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_paper_cycle_cap64(op):
    wl = small(op, 128, torch.bfloat16, batch=2, H=3, steps=140)
    rec, state, S0u, bonus = run_deltalog(wl, 64, DEV, units=all_units(wl), cycle="paper")
    assert 65 in rec.state_at and 130 in rec.state_at      # base alone is the state after each fused step
    check(wl, rec, oracle_for(wl, rec, S0u, bonus))


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("d", [64, 128])
def test_fused_step_at_every_live_length(op, d):
    """The fused step is defined for any live length 0..cap, not only for a full log."""
    import paper_2608_15533_b200 as dl

    cap = 5
    for n_append in range(cap + 1):
        wl = small(op, d, torch.float32, batch=2, H=2, steps=n_append + 1)
        src = workloads.TokenSource(wl, device="cpu")
        S0 = src.initial_state().to(DEV)
        bonus = src.bonus()
        bonus = bonus.to(DEV) if bonus is not None else None
        desc = make_desc(wl, cap, 0.7)
        state = dl.State(desc, S0.clone())
        units = all_units(wl)
        ub = torch.tensor([u[0] for u in units], device=DEV)
        uh = torch.tensor([u[1] for u in units], device=DEV)
        from harness import Recorded

        rec = Recorded(units=units)
        for t in range(n_append + 1):
            tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
            fn = dl.decode_step if t < n_append else dl.decode_merge_step
            out = fn(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
            rec.record_token(tok, out, wl)
        assert int(state.log_len.abs().sum()) == 0 and int(state.status.item()) == 0
        rec.state_at = [n_append + 1]
        rec.states = [f64(state.S_base[ub, uh])]
        check(wl, rec, oracle_for(wl, rec, f64(S0[ub, uh]), f64(bonus[uh]) if bonus is not None else None,
                                  scale=0.7))


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_fused_step_on_empty_log_is_the_eager_step(op):
    import paper_2608_15533_b200 as dl

    wl = small(op, 128, torch.bfloat16, batch=4, H=3, steps=6)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    desc = make_desc(wl, 4, 1.0)
    state = dl.State(desc, S0.clone())
    S_eager = S0.clone()
    for _ in range(wl.steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        args = (tok["q"], tok["k"], tok["v"], tok["g"])
        out_f = dl.decode_merge_step(desc, state, *args, beta=tok["beta"], u_bonus=bonus)
        out_e = dl.eager_step(desc, S_eager, *args, beta=tok["beta"], u_bonus=bonus)
        # same arithmetic up to the summation order of the two readouts
        assert rel_err(f64(out_f), f64(out_e)) <= 8e-3
        assert rel_err(f64(state.S_base), f64(S_eager)) <= 1e-5
    assert int(state.log_len.abs().sum()) == 0


def test_phase_split_batches_with_staggered_fills():
    """Rows that joined at different steps reach their merge boundary at different steps: each step is
    an append call over the rows with room and a fused-step call over the rows whose log is full."""
    wl = small(KDA, 128, torch.bfloat16, batch=8, H=2, steps=44)
    cap = 4
    delay = torch.tensor([0, 1, 2, 3, 4, 0, 2, 9])
    units = all_units(wl)
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, start_delay=delay, cycle="paper")
    ref = oracle_for(wl, rec, S0u, bonus)
    out = np.stack(rec.out)
    mask = ~np.isnan(ref["out"])
    assert rel_err(np.where(mask, out, 0.0), np.where(mask, ref["out"], 0.0)) <= out_tol(wl)
    assert rel_err(rec.states[-1], ref["S"]) <= TOL_STATE
    assert int(state.status.item()) == 0


def test_fused_step_padding_bad_slots_and_slot_indirection():
    import paper_2608_15533_b200 as dl

    wl = small(GDN, 64, torch.bfloat16, batch=6, H=2, steps=1, num_slots=9)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4, 1.0)
    state = dl.State(desc, S0.clone())
    tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
    slot_idx = torch.tensor([7, -1, 2, 99, 0, -1], dtype=torch.int32, device=DEV)
    out = torch.full((wl.batch, wl.H, wl.d), 3.0, dtype=wl.io_dtype, device=DEV)
    dl.decode_merge_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                         slot_idx=slot_idx, out=out)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_BAD_SLOT          # slot 99; -1 is silent padding
    for b in (1, 3, 5):
        assert bool((out[b] == 3.0).all())
    touched = {7, 2, 0}
    for s in range(wl.slots):
        same = torch.equal(state.S_base[s], S0[s])
        assert same != (s in touched)
    # the rows that ran agree with the eager kernel on a copy of the pool
    S_e = S0.clone()
    out_e = dl.eager_step(desc, S_e, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], slot_idx=slot_idx)
    for b in (0, 2, 4):
        assert rel_err(f64(out[b]), f64(out_e[b])) <= 8e-3
    assert rel_err(f64(state.S_base), f64(S_e)) <= 1e-5


@pytest.mark.parametrize("op,d", [(GDN, 128), (KDA, 128), (RWKV6, 64)])
def test_fused_step_walk_over_many_units_with_padding_and_indirection(op, d):
    """A batch large enough that every resident CTA of the fused-step kernel walks over several units, with a
    permuted slot list, padding rows and one slot outside the pool in the walk: after a few appends, the fused
    step's outputs and folded states agree with the eager kernel run on a materialised copy of the pool, rows
    that were skipped are untouched, and their units keep their logs."""
    import paper_2608_15533_b200 as dl

    batch, H, cap, appends = 150, 8, 8, 3                      # 1200 (row, head) pairs: 2-4 per resident CTA
    wl = small(op, d, torch.bfloat16, batch=batch, H=H, steps=appends + 1, num_slots=batch + 10)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus().to(DEV) if op == RWKV6 else None
    desc = make_desc(wl, cap, 1.0)
    state = dl.State(desc, S0.clone())
    g = torch.Generator().manual_seed(5)
    slots = torch.randperm(wl.slots, generator=g)[:batch].to(torch.int32)
    pad_rows = [3, 77, 78, 149]
    bad_row = 40
    slots[pad_rows] = -1
    slots[bad_row] = wl.slots + 5
    slot_idx = slots.to(DEV)
    S_e = S0.clone()                                            # the eager kernel's pool
    tok = None
    for t in range(appends + 1):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        if t < appends:
            dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                           slot_idx=slot_idx)
            dl.eager_step(desc, S_e, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                          slot_idx=slot_idx)
    torch.cuda.synchronize()
    state.status.zero_()                                        # (the appends flagged the bad slot as well)
    out = torch.full((batch, H, d), 3.0, dtype=wl.io_dtype, device=DEV)
    dl.decode_merge_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                         slot_idx=slot_idx, out=out)
    out_e = dl.eager_step(desc, S_e, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                          slot_idx=slot_idx)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_BAD_SLOT
    ran = [b for b in range(batch) if b not in pad_rows and b != bad_row]
    for b in pad_rows + [bad_row]:
        assert bool((out[b] == 3.0).all())
    assert rel_err(f64(out[ran]), f64(out_e[ran])) <= 1.6e-2    # two bf16 roundings of nearly equal fp32 values
    used = slots[ran].long()
    assert rel_err(f64(state.S_base[used]), f64(S_e[used])) <= 1e-5
    assert int(state.log_len[used].abs().max()) == 0            # folded
    unused = torch.tensor(sorted(set(range(wl.slots)) - set(used.tolist())))
    assert torch.equal(state.S_base[unused], S0[unused])        # never touched
    assert int(state.log_len[unused].abs().max()) == 0


def test_mixing_fused_steps_and_token_less_merges():
    """The two ways of materialising can be mixed freely on one state."""
    import paper_2608_15533_b200 as dl

    wl = small(RWKV6, 64, torch.bfloat16, batch=3, H=2, steps=30)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus().to(DEV)
    cap = 3
    desc = make_desc(wl, cap, 1.0)
    state = dl.State(desc, S0.clone())
    units = all_units(wl)
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    from harness import Recorded

    rec = Recorded(units=units)
    for t in range(wl.steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        full = bool((state.log_len == cap).all())
        if full and t % 2 == 0:
            dl.merge(desc, state)
            full = False
        fn = dl.decode_merge_step if full else dl.decode_step
        out = fn(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], u_bonus=bonus)
        rec.record_token(tok, out, wl)
    dl.merge(desc, state)
    rec.state_at = [wl.steps]
    rec.states = [f64(state.S_base[ub, uh])]
    check(wl, rec, oracle_for(wl, rec, f64(S0[ub, uh]), f64(bonus[uh])))
