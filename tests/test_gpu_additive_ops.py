"""GPU parity of the additive operator family of Table 1 (plain linear attention, RetNet, GLA:
b_t = v_t, output read from the updated state) through the same entry points, against the fp64 CPU
oracle on the same seeded inputs.  Bars as in test_gpu_parity.py."""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, f64, make_desc, materialize_units, oracle_for, out_tol, rel_err, run_deltalog
from workloads import GLA, LINATTN, RETNET, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"
OPS = [LINATTN, RETNET, GLA]


def small(op, d, io, batch=3, H=2, steps=40, **kw) -> Workload:
    return Workload(f"small_op{op}_d{d}", op, batch, H, d, steps, (1,), io_dtype=io, **kw)


def all_units(wl):
    return [(b, h) for b in range(wl.batch) for h in range(wl.H)]


def check(wl, rec, ref):
    e_out = rel_err(np.stack(rec.out), ref["out"])
    assert e_out <= out_tol(wl), f"output error {e_out:.3e}"
    assert rec.states and len(rec.states) == len(rec.state_at)
    worst = max(rel_err(S, ref["snapshots"][i]) for i, S in enumerate(rec.states))
    assert worst <= TOL_STATE, f"state error {worst:.3e}"


@pytest.mark.parametrize("cycle", ["split", "paper"])
@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("io", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("cap", [1, 3, 8])
def test_rollout_invariant_every_step(op, d, io, cap, cycle):
    """Eq. 6 materialised from the downloaded base + log equals the eager recurrence after every token,
    for the split cycle (appends + token-less merge) and for the paper's cycle (appends + fused step)."""
    wl = small(op, d, io, steps=26)
    units = all_units(wl)
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    mats = []

    def hook(t, state, tok, out):
        mats.append(materialize_units(state, wl, ub, uh))

    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units, scale=0.5, every_step_hook=hook, cycle=cycle)
    rec.state_at = list(range(1, wl.steps + 1))
    rec.states = mats
    check(wl, rec, oracle_for(wl, rec, S0u, bonus, scale=0.5))
    assert int(state.status.item()) == 0


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("cap", [16, 64])
def test_wide_batch_long_rollout(op, cap):
    """Enough units for the persistent decode kernel to walk several units per CTA, 150 tokens."""
    wl = small(op, 128, torch.bfloat16, batch=40, H=8, steps=150)
    units = [(0, 0), (7, 3), (19, 7), (39, 7), (23, 1)]
    rec, state, S0u, bonus = run_deltalog(wl, cap, DEV, units=units)
    check(wl, rec, oracle_for(wl, rec, S0u, bonus))
    assert int(state.status.item()) == 0


@pytest.mark.parametrize("op", OPS)
@pytest.mark.parametrize("d,io", [(64, torch.float32), (128, torch.bfloat16)])
def test_eager_kernel_and_log_entries(op, d, io):
    import paper_2608_15533_b200 as dl

    wl = small(op, d, io, batch=3, H=2, steps=12)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    desc = make_desc(wl, 16, 0.9)
    state = dl.State(desc, S0.clone())
    S = S0.clone()
    units = all_units(wl)
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    from harness import Recorded

    rec, rec_log = Recorded(units=units), Recorded(units=units)
    for t in range(wl.steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        out_e = dl.eager_step(desc, S, tok["q"], tok["k"], tok["v"], tok["g"])
        out_l = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"])
        rec.record_token(tok, out_e, wl)
        rec_log.record_token(tok, out_l, wl)
        # the appended entry: a_t = k_t and b_t = v_t bit-exact (the U log keeps the I/O dtype)
        assert torch.equal(state.K_log[:, :, t], tok["k"]) and torch.equal(state.U_log[:, :, t], tok["v"])
    rec.state_at, rec.states = [wl.steps], [f64(S[ub, uh])]
    ref = oracle_for(wl, rec, f64(S0[ub, uh]), None, scale=0.9)
    check(wl, rec, ref)
    assert rel_err(np.stack(rec_log.out), ref["out"]) <= out_tol(wl)
    assert bool((state.log_len == wl.steps).all())
    assert torch.equal(state.S_base, S0)                           # appends never write the base
    lam = np.cumsum(np.stack(rec.g), axis=0)                       # running log-decay [T, N, d_lambda]
    got = f64(state.decay_log[ub, uh])[:, : wl.steps]
    np.testing.assert_allclose(got, np.transpose(lam, (1, 0, 2)), rtol=1e-6, atol=1e-6)
