"""Reduced-precision value-side log for the delta rule (a 16-bit U log instead of fp32).

The paper keeps b_t in fp32 "to mitigate cancellation error along the correction path".  The CPU test
quantifies that on the oracle alone: the exact log schedule with every stored b_t rounded to bf16
leaves a state error two orders of magnitude above the 1e-4 parity bar, while rounding to fp32 stays
far below it.  The GPU test checks that the library's 16-bit variant computes exactly this reduced-
precision schedule (and no worse), which is why it is an opt-in variant and not the default."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from harness import Recorded, f64, oracle_for, out_tol, rel_err
from oracle import logical
from workloads import GDN, KDA, Workload


def to_bf16(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float64)).to(torch.bfloat16).to(torch.float64).numpy()


def to_f32(x):
    return np.asarray(x, dtype=np.float32).astype(np.float64)


def tokens_of(wl, steps):
    src = workloads.TokenSource(wl, device="cpu")
    S0 = f64(src.initial_state()).reshape(-1, wl.d, wl.d)
    toks = [src.token() for _ in range(steps)]
    flat = lambda t: f64(t).reshape(wl.batch * wl.H, -1)
    return S0, [{k: (flat(v) if v is not None else None) for k, v in tok.items()} for tok in toks]


@pytest.mark.parametrize("op", [GDN, KDA])
def test_error_study_on_the_oracle(op):
    wl = Workload("ulog_cpu", op, 1, 2, 32, 96, (16,))
    cap, steps = 16, 96
    S0, toks = tokens_of(wl, steps)
    stack = lambda name: np.stack([t[name] for t in toks])
    ref = oracle.eager_rollout(op, S0, stack("q"), stack("k"), stack("v"), stack("g"), beta=stack("beta")[..., 0])
    errs = {}
    for name, rounding in (("bf16", to_bf16), ("fp32", to_f32)):
        st = logical.LogState(op, S0, cap, store_u=rounding)
        for t, tok in enumerate(toks):
            if (st.length == cap).all():
                logical.merge(st)
            logical.decode_step(st, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"][:, 0])
        errs[name] = rel_err(logical.materialize(st), ref["S"])
    assert errs["fp32"] < 1e-6
    assert 1e-4 < errs["bf16"] < 2e-2, errs     # breaks the state bar: the default keeps b_t in fp32


@pytest.mark.gpu
@pytest.mark.parametrize("op", [GDN, KDA])
@pytest.mark.parametrize("d,cap", [(64, 8), (128, 16)])
def test_16_bit_u_log_variant_on_the_gpu(op, d, cap):
    import paper_2608_15533_b200 as dl

    DEV = "cuda"
    wl = Workload("ulog_gpu", op, 6, 4, d, 64, (cap,))
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    desc = dl.Desc(op=op, num_slots=wl.batch, H=wl.H, d_k=d, d_v=d, cap=cap, io_dtype=dl.BF16, ulog_dtype=dl.BF16)
    desc32 = dl.Desc(op=op, num_slots=wl.batch, H=wl.H, d_k=d, d_v=d, cap=cap, io_dtype=dl.BF16)
    state, state32 = dl.State(desc, S0.clone()), dl.State(desc32, S0.clone())
    assert state.U_log.dtype == torch.bfloat16 and state32.U_log.dtype == torch.float32
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    rec = Recorded(units=units)
    for t in range(wl.steps):
        if t and t % cap == 0:
            dl.merge(desc, state)
            dl.merge(desc32, state32)
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"])
        dl.decode_step(desc32, state32, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"])
        rec.record_token(tok, out, wl)
        if t == 0:   # both variants have seen identical states so far: the entry is the rounded fp32 entry
            assert torch.equal(state.U_log[:, :, 0], state32.U_log[:, :, 0].to(torch.bfloat16))
    dl.merge(desc, state)
    dl.merge(desc32, state32)
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    rec.state_at, rec.states = [wl.steps], [f64(state.S_base[ub, uh])]
    ref = oracle_for(wl, rec, f64(S0[ub, uh]), None)
    assert rel_err(np.stack(rec.out), ref["out"]) <= out_tol(wl)          # outputs still meet the bf16 bar
    e16 = rel_err(rec.states[0], ref["S"])
    e32 = rel_err(f64(state32.S_base[ub, uh]), ref["S"])
    assert e32 <= 1e-4 and e32 < e16 <= 2e-2, (e16, e32)                  # the state does not meet 1e-4
