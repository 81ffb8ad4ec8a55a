"""GPU parity: the CUDA decode / append / merge / eager kernels, called through the C ABI, against
the fp64 CPU oracle on the same seeded inputs.

Bars (max|x - ref| / max|ref| over the compared tensor): fp32 state 1e-4, bf16 outputs 2e-2,
fp32 outputs 1e-4; log entries K bit-exact, U 1e-5, Lambda 1e-6; integer metadata exact.
"""
import numpy as np
import pytest
import torch

import workloads
from harness import (TOL_STATE, f64, make_desc, materialize_units, oracle_for, out_tol, rel_err, run_deltalog,
                     sample_units)
from workloads import CONFIGS, GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small(op, d, io, batch=3, H=2, steps=40, **kw) -> Workload:
    return Workload(f"small_op{op}_d{d}", op, batch, H, d, steps, (1,), io_dtype=io, **kw)


def check_rollout(wl, rec, ref, state_tol=TOL_STATE):
    out = np.stack(rec.out)
    mask = ~np.isnan(ref["out"])
    assert mask.any()
    e_out = rel_err(np.where(mask, out, 0.0), np.where(mask, ref["out"], 0.0))
    assert e_out <= out_tol(wl), f"output error {e_out:.3e}"
    assert len(rec.states) == len(rec.state_at) and rec.states
    worst = 0.0
    for i, S in enumerate(rec.states):
        worst = max(worst, rel_err(S, ref["snapshots"][i]))
    assert worst <= state_tol, f"state error {worst:.3e}"
    return e_out, worst


# ------------------------------------------------------------------------------------------------
# configuration 0: all-fp32 GDN, every output, every merge boundary, every log entry
# ------------------------------------------------------------------------------------------------
def test_config0_gdn_fp32_outputs_states_and_log_contents():
    import paper_2608_15533_b200 as dl

    wl, cap = CONFIGS[0], CONFIGS[0].caps[0]
    units = [(0, 0), (0, 1)]
    seen = {"U": [], "K": [], "Lam": [], "len": []}

    def hook(t, state, tok, out):
        L = int(state.log_len[0, 0])
        seen["len"].append(L)
        seen["U"].append(f64(state.U_log[0, :, L - 1]))
        seen["K"].append(state.K_log[0, :, L - 1].cpu())
        seen["Lam"].append(f64(state.decay_log[0, :, L - 1, 0]))
        assert torch.equal(state.K_log[0, :, L - 1], tok["k"][0])          # K entry is k_t, bit for bit

    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, every_step_hook=hook)
    ref = oracle_for(wl, rec, S0u, bonus)
    e_out, e_state = check_rollout(wl, rec, ref)
    assert len(rec.state_at) == wl.steps // cap                              # every merge boundary was compared
    assert seen["len"] == [(t % cap) + 1 for t in range(wl.steps)]
    U = np.stack(seen["U"])
    assert rel_err(U, ref["b"]) <= 1e-5                                       # U entry is b_t
    g = np.stack(rec.g)[:, :, 0]
    for t in range(wl.steps):
        first = t - (t % cap)
        np.testing.assert_allclose(seen["Lam"][t], g[first:t + 1].sum(axis=0), rtol=1e-6, atol=1e-6)
    assert int(state.status.item()) == 0
    assert int(state.log_len.abs().sum()) == 0


# ------------------------------------------------------------------------------------------------
# every operator x head size x dtype: Eq. 6 after every step, several capacities incl. ragged ones
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("io", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("cap", [1, 3, 8])
def test_small_rollout_invariant_every_step(op, d, io, cap):
    wl = small(op, d, io, steps=26)
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    mats = []

    def hook(t, state, tok, out):
        mats.append(materialize_units(state, wl, ub, uh))

    scale = 0.5 if op != RWKV6 else 1.0
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, scale=scale, every_step_hook=hook)
    rec.state_at = list(range(1, wl.steps + 1))                 # compare the materialised state after every token
    rec.states = mats
    ref = oracle_for(wl, rec, S0u, bonus, scale=scale)
    check_rollout(wl, rec, ref)
    assert int(state.status.item()) == 0


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_cap64_and_long_rollout(op):
    wl = small(op, 64, torch.bfloat16, batch=2, H=3, steps=150)
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    rec, state, S0u, bonus = run_deltalog(wl, 64, DEV, units=units)
    check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))


# ------------------------------------------------------------------------------------------------
# eager comparator and representation independence
# ------------------------------------------------------------------------------------------------
def run_eager(wl, steps, scale=1.0, S_init=None, src=None, bonus=None, slot_idx=None):
    import paper_2608_15533_b200 as dl

    if src is None:
        src = workloads.TokenSource(wl, device="cpu")
        S_init = src.initial_state().to(DEV)
        bonus = src.bonus()
        bonus = bonus.to(DEV) if bonus is not None else None
    S = S_init.clone()
    desc = make_desc(wl, 1, scale)
    outs, toks = [], []
    for _ in range(steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        outs.append(dl.eager_step(desc, S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                                  u_bonus=bonus, slot_idx=slot_idx))
        toks.append(tok)
    return S_init, S, outs, toks, bonus


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("d,io", [(64, torch.float32), (128, torch.bfloat16)])
def test_eager_kernel_matches_oracle(op, d, io):
    import oracle

    wl = small(op, d, io, steps=48)
    scale = 0.25 if op != RWKV6 else 1.0
    S0, S, outs, toks, bonus = run_eager(wl, wl.steps, scale)
    N = wl.batch * wl.H
    flat = lambda key: np.stack([f64(t[key]).reshape(N, -1) for t in toks])
    ref = oracle.eager_rollout(op, f64(S0).reshape(N, d, d), flat("q"), flat("k"), flat("v"), flat("g"),
                               beta=flat("beta")[..., 0] if op != RWKV6 else None,
                               bonus=np.tile(f64(bonus), (wl.batch, 1)) if bonus is not None else None, scale=scale)
    assert rel_err(f64(S).reshape(N, d, d), ref["S"]) <= TOL_STATE
    assert rel_err(np.stack([f64(o).reshape(N, d) for o in outs]), ref["out"]) <= out_tol(wl)


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_cap1_equals_eager_kernel_and_outputs_do_not_depend_on_cap(op):
    wl = small(op, 128, torch.float32, steps=36)
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    _, S_eager, outs_eager, _, _ = run_eager(wl, wl.steps)
    eager_out = np.stack([f64(o).reshape(len(units), -1) for o in outs_eager])
    for cap in (1, 4, 8, 16, 32):
        rec, state, _, _ = run_deltalog(wl, cap, DEV, units=units)
        assert rel_err(np.stack(rec.out), eager_out) <= 2e-5, f"cap={cap}"
        assert rel_err(f64(state.S_base), f64(S_eager)) <= 2e-5, f"cap={cap}"


def test_switching_between_log_schedule_and_eager_kernel():
    """Merged base == dense state: decode with the log, merge, continue with the eager kernel."""
    import oracle
    import paper_2608_15533_b200 as dl

    wl = small(GDN, 64, torch.float32, steps=30)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 8)
    state = dl.State(desc, S0.clone())
    toks, outs = [], []
    for t in range(wl.steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        toks.append(tok)
        if t < 13:
            outs.append(dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"]))
            if int(state.log_len[0, 0]) == 8:
                dl.merge(desc, state)
        else:
            if t == 13:
                dl.merge(desc, state)  # partial log (5 entries) folded
                assert int(state.log_len.sum()) == 0
            outs.append(dl.eager_step(desc, state.S_base, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"]))
    N = wl.batch * wl.H
    flat = lambda key: np.stack([f64(t[key]).reshape(N, -1) for t in toks])
    ref = oracle.eager_rollout(GDN, f64(S0).reshape(N, 64, 64), flat("q"), flat("k"), flat("v"), flat("g"),
                               beta=flat("beta")[..., 0])
    assert rel_err(f64(state.S_base).reshape(N, 64, 64), ref["S"]) <= TOL_STATE
    assert rel_err(np.stack([f64(o).reshape(N, 64) for o in outs]), ref["out"]) <= 1e-4


# ------------------------------------------------------------------------------------------------
# slot addressing, padding, device-detected conditions, untouched memory
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [GDN, RWKV6])
def test_slot_indirection_padding_and_pool_larger_than_batch(op):
    wl = small(op, 64, torch.bfloat16, batch=6, H=2, steps=20, num_slots=11)
    slot_idx = workloads.slot_permutation(wl, pad_every=4)       # rows 0 and 4 are padding
    live = [b for b in range(wl.batch) if slot_idx[b] >= 0]
    units = [(b, h) for b in live for h in range(wl.H)]
    rec, state, S0u, bonus = run_deltalog(wl, 4, DEV, units=units, slot_idx=slot_idx)
    check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))
    used = set(int(s) for s in slot_idx if s >= 0)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state()
    for s in range(wl.slots):
        if s not in used:   # slots outside the batch keep their initial bits
            assert torch.equal(state.S_base[s].cpu(), S0[s])
            assert int(state.log_len[s].sum()) == 0


def test_padded_rows_leave_out_untouched_and_bad_slots_set_status():
    import paper_2608_15533_b200 as dl

    wl = small(GDN, 64, torch.float32, batch=4, H=2)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4)
    state = dl.State(desc, S0.clone())
    tok = {k_: v_.to(DEV) for k_, v_ in src.token().items()}
    out = torch.full((4, 2, 64), 777.0, device=DEV)
    slot_idx = torch.tensor([2, -1, 99, 0], dtype=torch.int32, device=DEV)
    dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], slot_idx=slot_idx, out=out)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_BAD_SLOT
    assert bool((out[1] == 777.0).all()) and bool((out[2] == 777.0).all())
    assert not bool((out[0] == 777.0).any()) and not bool((out[3] == 777.0).any())
    assert state.log_len.cpu().tolist() == [[1, 1], [0, 0], [1, 1], [0, 0]]
    assert torch.equal(state.S_base, S0)                          # decode never writes the base
    state.status.zero_()
    dl.merge(desc, state, slot_idx=slot_idx)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_BAD_SLOT
    assert int(state.log_len.sum()) == 0
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    S = S0.clone()
    dl.eager_step(desc, S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], slot_idx=slot_idx, status=st)
    assert int(st.item()) == dl.STATUS_BAD_SLOT
    assert torch.equal(S[1], S0[1]) and torch.equal(S[3], S0[3]) and not torch.equal(S[2], S0[2])


def test_decode_on_full_log_sets_status_and_changes_nothing():
    import paper_2608_15533_b200 as dl

    wl = small(KDA, 64, torch.bfloat16, batch=2, H=2)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 2)
    state = dl.State(desc, S0.clone())
    toks = [{k_: v_.to(DEV) for k_, v_ in src.token().items()} for _ in range(3)]
    for tok in toks[:2]:
        dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"])
    snap = [t.clone() for t in (state.K_log, state.U_log, state.decay_log, state.log_len, state.S_base)]
    out = torch.full((2, 2, 64), 5.0, dtype=torch.bfloat16, device=DEV)
    tok = toks[2]
    dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], out=out)
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_LOG_FULL
    for a, b in zip(snap, (state.K_log, state.U_log, state.decay_log, state.log_len, state.S_base)):
        assert torch.equal(a, b)
    assert bool((out == 5.0).all())


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_unused_log_entries_are_never_read_and_merge_of_empty_log_writes_nothing(op):
    import paper_2608_15533_b200 as dl

    wl = small(op, 64, torch.float32, batch=2, H=2, steps=5)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    desc = make_desc(wl, 8)
    state = dl.State(desc, S0.clone())
    for t_ in (state.K_log, state.U_log, state.decay_log):
        t_.fill_(float("nan"))                                   # poison: reading a dead entry shows up as NaN
    dl.merge(desc, state)                                        # empty logs: must not touch the base
    dl.merge(desc, state, only_if_full=True)
    assert torch.equal(state.S_base, S0)
    for _ in range(wl.steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
        assert bool(torch.isfinite(out).all())
    dl.merge(desc, state, only_if_full=True)                     # 5 of 8 entries: skipped
    assert torch.equal(state.S_base, S0) and int(state.log_len[0, 0]) == 5
    dl.merge(desc, state)
    assert bool(torch.isfinite(state.S_base).all()) and int(state.log_len.sum()) == 0
    assert bool(torch.isnan(state.K_log[:, :, 5:]).all())        # dead entries were never written either


def test_staggered_batch_is_bit_identical_to_rows_run_on_their_own():
    """Results of a row do not depend on what the other rows of the call are doing."""
    wl = small(GDN, 128, torch.bfloat16, batch=8, H=2, steps=40)
    cap = 4
    delay = torch.tensor([0, 1, 2, 3, 0, 1, 2, 3])
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    rec_all, state_all, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, start_delay=delay)
    out_all = np.stack(rec_all.out)
    ref = oracle_for(wl, rec_all, S0u, bonus)
    mask = ~np.isnan(ref["out"])
    assert rel_err(np.where(mask, out_all, 0.0), np.where(mask, ref["out"], 0.0)) <= out_tol(wl)
    assert rel_err(rec_all.states[-1], ref["S"]) <= TOL_STATE
    for dly in range(4):   # the same rows, alone in their call: all other rows are padding for the whole run
        solo_delay = torch.where(delay == dly, delay, torch.full_like(delay, 10 ** 6))
        rec, state, _, _ = run_deltalog(wl, cap, DEV, units=units, start_delay=solo_delay)
        rows = [i for i, u in enumerate(units) if int(delay[u[0]]) == dly]
        solo = np.stack(rec.out)[dly:, rows]
        assert np.array_equal(solo, out_all[dly:, rows])
        for b in range(wl.batch):
            if int(delay[b]) == dly:
                assert torch.equal(state.S_base[b], state_all.S_base[b])


def test_rerun_is_bit_identical():
    wl = small(KDA, 128, torch.bfloat16, steps=24)
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    a = run_deltalog(wl, 8, DEV, units=units)
    b = run_deltalog(wl, 8, DEV, units=units)
    assert np.array_equal(np.stack(a[0].out), np.stack(b[0].out))
    assert torch.equal(a[1].S_base, b[1].S_base)


def test_host_buffer_entry_point_matches_device_entry_point():
    import paper_2608_15533_b200 as dl

    wl = small(GDN, 128, torch.bfloat16, batch=4, H=2)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4)
    s_dev, s_host = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    staging = dl.HostStaging(desc, wl.batch, DEV)
    for _ in range(3):
        tok = src.token()
        pinned = {k_: v_.pin_memory() for k_, v_ in tok.items()}
        host_out = torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory()
        dl.decode_step_host(desc, s_host, staging, pinned["q"], pinned["k"], pinned["v"], pinned["g"],
                            pinned["beta"], host_out)
        dev = {k_: v_.to(DEV) for k_, v_ in tok.items()}
        out = dl.decode_step(desc, s_dev, dev["q"], dev["k"], dev["v"], dev["g"], beta=dev["beta"])
        torch.cuda.synchronize()
        assert torch.equal(out.cpu(), host_out)
    assert torch.equal(s_dev.U_log, s_host.U_log)


def test_overlapped_host_entry_point_matches_device_entry_point_over_a_cycle():
    """Three streams, two staging sets, merges on the compute stream: same bits as the plain path."""
    import paper_2608_15533_b200 as dl

    wl = small(KDA, 128, torch.bfloat16, batch=4, H=2)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4)
    s_dev, s_host = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    streams = [torch.cuda.Stream() for _ in range(3)]
    sets = [(dl.HostStaging(desc, wl.batch, DEV), dl.HostLane(*streams)) for _ in range(2)]
    toks = [src.token() for _ in range(10)]
    pinned = [{k_: v_.pin_memory() for k_, v_ in tok.items()} for tok in toks]
    host_outs = [torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory() for _ in toks]
    torch.cuda.synchronize()
    with torch.cuda.stream(streams[1]):
        for t, p in enumerate(pinned):
            staging, lane = sets[t % 2]
            dl.decode_step_host_overlapped(desc, s_host, staging, lane, p["q"], p["k"], p["v"], p["g"], p["beta"],
                                           host_outs[t])
            if (t + 1) % 4 == 0:
                dl.merge(desc, s_host, only_if_full=True)
    for st in streams:
        st.synchronize()
    for t, tok in enumerate(toks):
        dev = {k_: v_.to(DEV) for k_, v_ in tok.items()}
        out = dl.decode_step(desc, s_dev, dev["q"], dev["k"], dev["v"], dev["g"], beta=dev["beta"])
        if (t + 1) % 4 == 0:
            dl.merge(desc, s_dev, only_if_full=True)
        assert torch.equal(out.cpu(), host_outs[t]), f"step {t}"
    torch.cuda.synchronize()
    assert torch.equal(s_dev.S_base, s_host.S_base) and torch.equal(s_dev.U_log, s_host.U_log)
    assert torch.equal(s_dev.log_len, s_host.log_len)


@pytest.mark.parametrize("op", [GDN, KDA])
def test_predicate_merge_at_capacity_64_head_size_128(op):
    """The packed predicate merge needs more than 48 KiB of dynamic shared memory here, beside its
    static arrays."""
    wl = small(op, 128, torch.bfloat16, batch=5, H=3, steps=140)
    rec, state, S0u, bonus = run_deltalog(wl, 64, DEV, units=[(0, 0), (2, 1), (4, 2)])
    assert 64 in rec.state_at and 128 in rec.state_at
    check_rollout(wl, rec, oracle_for(wl, rec, S0u, bonus))


@pytest.mark.parametrize("op,d", [(GDN, 128), (KDA, 128), (RWKV6, 64)])
def test_chained_launches_are_bit_identical(op, d):
    """Decode steps that follow a decode step of the same state may be launched ahead of its completion
    (the caller's hint): lengths and log entries are still read only after it has finished."""
    import paper_2608_15533_b200 as dl

    wl = small(op, d, torch.bfloat16, batch=40, H=8, steps=48)
    cap = 16
    results = []
    for chained in (False, True):
        src = workloads.TokenSource(wl, device="cpu")
        S0 = src.initial_state().to(DEV)
        bonus = src.bonus()
        bonus = bonus.to(DEV) if bonus is not None else None
        toks = [{k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()} for _ in range(wl.steps)]
        desc = make_desc(wl, cap)
        desc_c = make_desc(wl, cap)
        desc_c.hints = dl.HINT_BASE_UNTOUCHED if chained else 0
        state = dl.State(desc, S0.clone())
        outs = [torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype, device=DEV) for _ in range(wl.steps)]
        torch.cuda.synchronize()
        for t, tok in enumerate(toks):     # launched back to back, nothing in between
            first = t % cap == 0
            if first and t:
                dl.merge(desc, state)
            dl.decode_step(desc if first else desc_c, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                           u_bonus=bonus, out=outs[t])
        dl.merge(desc, state)
        torch.cuda.synchronize()
        assert int(state.status.item()) == 0
        results.append((torch.stack(outs), state.S_base.clone()))
    assert torch.equal(results[0][0], results[1][0]) and torch.equal(results[0][1], results[1][1])


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_packed_host_buffers_travel_in_one_copy_and_give_the_same_result(op):
    """Host tokens and staging buffers laid out back to back (256-byte aligned) are copied as one
    block; the result is that of the device entry point."""
    import paper_2608_15533_b200 as dl

    wl = small(op, 64, torch.bfloat16, batch=5, H=3, steps=3)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    desc = make_desc(wl, 4)
    st_h, st_d = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    staging = dl.HostStaging(desc, wl.batch, DEV)
    staging.packed = True
    host = dl.packed_host_tokens(desc, wl.batch)
    assert host["k"].data_ptr() - host["q"].data_ptr() == staging.k.data_ptr() - staging.q.data_ptr()
    host_out = torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory()
    for _ in range(wl.steps):
        tok = src.token()
        for name in ("q", "k", "v", "g", "beta"):
            if tok[name] is not None:
                host[name].copy_(tok[name])
        dl.decode_step_host(desc, st_h, staging, host["q"], host["k"], host["v"], host["g"],
                            host["beta"] if tok["beta"] is not None else None, host_out, u_bonus=bonus)
        ref = dl.decode_step(desc, st_d, *(tok[n].to(DEV) for n in ("q", "k", "v", "g")),
                             beta=tok["beta"].to(DEV) if tok["beta"] is not None else None, u_bonus=bonus)
        torch.cuda.synchronize()
        assert torch.equal(host_out.to(DEV), ref)
    assert torch.equal(st_h.U_log, st_d.U_log) and torch.equal(st_h.log_len, st_d.log_len)
