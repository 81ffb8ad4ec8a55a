"""Key and value head dimensions that differ (d_k != d_v: 128 x 64 and 64 x 128), as real checkpoints of
the gated-delta and per-channel-gated operators have them.  Every entry point that takes a shape:
single-token decode with the token-less merge (Eq. 6 materialised from the downloaded physical state
after every token), the paper's cycle with the fused merge step, blocks of tokens, the eager kernel,
slot hand-over with a prefill state, and the host-buffer entry points -- all against the fp64 oracle,
on narrow and on wide batches."""
import numpy as np
import pytest
import torch

import workloads
from harness import (TOL_STATE, f64, make_desc, materialize_units, oracle_for, out_tol, rel_err, run_deltalog)
from workloads import GDN, GLA, KDA, RETNET, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"
SHAPES = [(128, 64), (64, 128)]


def wl_for(op, dk, dv, io, batch=3, H=2, steps=22, **kw):
    return Workload(f"mixed_{op}_{dk}x{dv}", op, batch, H, dk, steps, (1,), io_dtype=io, d_v=dv, **kw)


def all_units(wl):
    return [(b, h) for b in range(wl.batch) for h in range(wl.H)]


@pytest.mark.parametrize("dk,dv", SHAPES)
@pytest.mark.parametrize("op", [GDN, KDA, RWKV6, GLA, RETNET])
@pytest.mark.parametrize("io,cap,cycle", [(torch.bfloat16, 8, "split"), (torch.float32, 3, "split"), (torch.bfloat16, 4, "paper")])
def test_invariant_after_every_token(op, dk, dv, io, cap, cycle):
    wl = wl_for(op, dk, dv, io)
    units = all_units(wl)
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    mats = []
    scale = 0.5 if op != RWKV6 else 1.0
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, scale=scale, cycle=cycle,
                                          every_step_hook=lambda t, st, tok, out: mats.append(materialize_units(st, wl, ub, uh)))
    assert state.S_base.shape[-2:] == (dk, dv) and state.K_log.shape[-1] == dk and state.U_log.shape[-1] == dv
    rec.state_at, rec.states = list(range(1, wl.steps + 1)), mats
    ref = oracle_for(wl, rec, S0u, bonus, scale=scale)
    assert rel_err(np.stack(rec.out), ref["out"]) <= out_tol(wl)
    for i, S in enumerate(mats):
        assert rel_err(S, ref["snapshots"][i]) <= TOL_STATE, f"after token {i + 1}"
    assert int(state.status.item()) == 0


@pytest.mark.parametrize("dk,dv", SHAPES)
@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_wide_batch_capacity_16_and_64(op, dk, dv):
    for cap in (16, 64):
        wl = wl_for(op, dk, dv, torch.bfloat16, batch=48, H=8, steps=cap + 7)
        units = [(0, 0), (47, 7), (13, 5), (31, 2), (20, 0), (5, 7)]
        rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, generator_device="cuda")
        ref = oracle_for(wl, rec, S0u, bonus)
        assert rel_err(np.stack(rec.out), ref["out"]) <= out_tol(wl)
        for i, S in enumerate(rec.states):
            assert rel_err(S, ref["snapshots"][i]) <= TOL_STATE
        assert int(state.status.item()) == 0


@pytest.mark.parametrize("dk,dv", SHAPES)
@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_blocks_of_tokens_eager_kernel_and_slot_hand_over(op, dk, dv):
    import oracle
    import paper_2608_15533_b200 as dl

    wl = wl_for(op, dk, dv, torch.bfloat16, batch=4, H=3, steps=16)
    cap, T = 8, 4
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    toks = [{k: (v.to(DEV) if v is not None else None) for k, v in src.token().items()} for _ in range(wl.steps)]
    desc = make_desc(wl, cap)
    N = wl.batch * wl.H
    flat = lambda name: np.stack([f64(t[name]).reshape(N, -1) for t in toks])
    ref = oracle.eager_rollout(op, f64(S0).reshape(N, dk, dv), flat("q"), flat("k"), flat("v"), flat("g"),
                               beta=flat("beta")[..., 0] if toks[0]["beta"] is not None else None,
                               bonus=np.tile(f64(bonus), (wl.batch, 1)) if bonus is not None else None)
    # blocks of T tokens
    st = dl.State(desc, S0.clone())
    outs = []
    for i in range(0, wl.steps, T):
        if i and i % cap == 0:
            dl.merge(desc, st)
        cat = lambda n: torch.stack([t[n] for t in toks[i:i + T]], dim=1).contiguous()
        o = dl.decode_steps(desc, st, cat("q"), cat("k"), cat("v"), cat("g"),
                            beta=cat("beta") if toks[0]["beta"] is not None else None, u_bonus=bonus)
        outs.extend(o.unbind(1))
    dl.merge(desc, st)
    assert rel_err(np.stack([f64(o).reshape(N, dv) for o in outs]), ref["out"]) <= 2e-2
    assert rel_err(f64(st.S_base).reshape(N, dk, dv), ref["S"]) <= TOL_STATE
    # eager kernel
    S = S0.clone()
    outs = [dl.eager_step(desc, S, t["q"], t["k"], t["v"], t["g"], beta=t["beta"], u_bonus=bonus) for t in toks]
    assert rel_err(np.stack([f64(o).reshape(N, dv) for o in outs]), ref["out"]) <= 2e-2
    assert rel_err(f64(S).reshape(N, dk, dv), ref["S"]) <= TOL_STATE
    # slot hand-over: two slots get a prefill state, their logs are emptied, the others keep theirs
    st = dl.State(desc, S0.clone())
    for t in toks[:3]:
        dl.decode_step(desc, st, t["q"], t["k"], t["v"], t["g"], beta=t["beta"], u_bonus=bonus)
    fresh = torch.randn(2, wl.H, dk, dv, device=DEV)
    dl.reset_slots(desc, st, slot_idx=torch.tensor([2, 0], dtype=torch.int32, device=DEV), S_init=fresh)
    torch.cuda.synchronize()
    assert torch.equal(st.S_base[2], fresh[0]) and torch.equal(st.S_base[0], fresh[1]) and torch.equal(st.S_base[1], S0[1])
    assert st.log_len[:, 0].tolist() == [0, 3, 0, 3] and int(st.status.item()) == 0


@pytest.mark.parametrize("dk,dv", SHAPES)
def test_host_buffer_entry_points(dk, dv):
    import paper_2608_15533_b200 as dl

    wl = wl_for(KDA, dk, dv, torch.bfloat16, batch=5, H=3, steps=2)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 4)
    ref, host, static = (dl.State(desc, S0.clone()) for _ in range(3))
    staging = dl.HostStaging(desc, wl.batch, DEV)
    for _ in range(wl.steps):
        tok = src.token()
        dev_tok = {k: v.to(DEV) for k, v in tok.items()}
        pin = {k: v.pin_memory() for k, v in tok.items()}
        want = dl.decode_step(desc, ref, dev_tok["q"], dev_tok["k"], dev_tok["v"], dev_tok["g"], beta=dev_tok["beta"])
        o1 = torch.empty(wl.batch, wl.H, dv, dtype=wl.io_dtype).pin_memory()
        o2 = torch.empty_like(o1).pin_memory()
        dl.decode_step_host(desc, host, staging, pin["q"], pin["k"], pin["v"], pin["g"], pin["beta"], o1)
        dl.decode_step_host_static(desc, static, pin["q"], pin["k"], pin["v"], pin["g"], pin["beta"], o2)
        torch.cuda.synchronize()
        assert torch.equal(o1, want.cpu()) and torch.equal(o2, want.cpu())
    assert torch.equal(ref.U_log, host.U_log) and torch.equal(ref.U_log, static.U_log)
