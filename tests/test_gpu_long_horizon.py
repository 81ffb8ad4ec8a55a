"""Long horizon: 1 500 tokens through a schedule that mixes everything the serving loop uses -- split
cycles (appends + token-less merge) and the paper's cycles (appends + fused merge step) in turn, decode
launches chained where the promise holds, walking directions alternating from launch to launch -- on
batches where every persistent CTA walks over several units.

The parity bar is stated for 256 steps; this follows a sample of units for six times that, across some
ninety materialisations of both kinds, against the fp64 oracle (every output, the final state), and
checks that a second run of the same schedule reproduces outputs, state and log bit for bit."""
import dataclasses

import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, Recorded, f64, make_desc, oracle_for, out_tol, rel_err, sample_units
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"
STEPS, CAP = 1500, 16


def run_schedule(wl, record):
    import paper_2608_15533_b200 as dl

    src = workloads.TokenSource(wl, device=DEV)
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    base = make_desc(wl, CAP, 1.0)
    state = dl.State(base, S0.clone())
    rec = Recorded(units=sample_units(wl, 12)) if record else None
    outs_last = None
    period = 2 * CAP + 1                     # CAP appends, merge, CAP appends, fused step
    for t in range(STEPS):
        tok = src.token()
        place = t % period
        fused = place == period - 1
        fill = place if place < CAP else place - CAP
        if fused:
            out = dl.decode_merge_step(base, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                                       u_bonus=bonus)
        else:
            hints = (dl.HINT_WALK_DOWN if fill & 1 else 0) | \
                    (dl.HINT_BASE_UNTOUCHED | dl.HINT_SLOTS_STABLE if fill else 0)
            out = dl.decode_step(dataclasses.replace(base, hints=hints), state, tok["q"], tok["k"], tok["v"], tok["g"],
                                 beta=tok["beta"], u_bonus=bonus)
            if place == CAP - 1:
                dl.merge(base, state)
        if rec is not None:
            rec.record_token(tok, out, wl)
        outs_last = out
    dl.merge(base, state)                    # whatever is live at the end
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    return rec, state, S0, bonus, outs_last


@pytest.mark.parametrize("op,d,batch,H", [(GDN, 128, 40, 16), (KDA, 128, 40, 8), (RWKV6, 64, 80, 16)])
def test_fifteen_hundred_tokens_through_both_cycles(op, d, batch, H):
    wl = Workload(f"long_op{op}", op, batch, H, d, STEPS, (CAP,), io_dtype=torch.bfloat16)
    rec, state, S0, bonus, out_a = run_schedule(wl, record=True)
    ub = torch.tensor([u[0] for u in rec.units], device=DEV)
    uh = torch.tensor([u[1] for u in rec.units], device=DEV)
    ref = oracle_for(wl, rec, f64(S0[ub, uh]), f64(bonus[uh]) if bonus is not None else None)
    out = np.stack(rec.out)
    e_out = rel_err(out, ref["out"])
    assert e_out <= out_tol(wl), f"output error over {STEPS} steps {e_out:.3e}"
    # the last quarter on its own (an error that grows with the horizon would show here first)
    e_tail = rel_err(out[-STEPS // 4:], ref["out"][-STEPS // 4:])
    assert e_tail <= out_tol(wl), f"output error over the last quarter {e_tail:.3e}"
    e_state = rel_err(f64(state.S_base[ub, uh]), ref["S"])
    assert e_state <= TOL_STATE, f"state error after {STEPS} steps {e_state:.3e}"
    assert int(state.log_len.abs().max()) == 0

    # the same schedule again: bit-identical
    _, state_b, _, _, out_b = run_schedule(wl, record=False)
    assert torch.equal(out_a.view(torch.int16), out_b.view(torch.int16))
    assert torch.equal(state.S_base, state_b.S_base)
    assert torch.equal(state.K_log.view(torch.int16), state_b.K_log.view(torch.int16))
