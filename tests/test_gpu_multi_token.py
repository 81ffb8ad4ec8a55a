"""GPU parity of the multi-token decode entry point: T tokens per row in one call must give what T
single-token calls give (and what the oracle gives), for every operator, with grouped heads, slot
indirection, and rows that have no room for all T entries."""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, Recorded, f64, oracle_for, out_tol, rel_err
from workloads import GDN, GLA, KDA, LINATTN, RETNET, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


def stack_tokens(toks):
    """List of T token dicts ([B,H,..] each) -> one dict with a token axis after the batch axis."""
    return {k: (torch.stack([t[k] for t in toks], dim=1).contiguous() if toks[0][k] is not None else None)
            for k in toks[0]}


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6, LINATTN, RETNET, GLA])
@pytest.mark.parametrize("d,io", [(64, torch.float32), (128, torch.bfloat16)])
@pytest.mark.parametrize("T", [1, 3, 4])
def test_block_of_tokens_equals_single_steps_and_the_oracle(op, d, io, T):
    import paper_2608_15533_b200 as dl

    cap, blocks = 8, 5
    wl = Workload(f"multi_op{op}", op, 3, 2, d, T * blocks, (cap,), io_dtype=io)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    dt = dl.F32 if io == torch.float32 else dl.BF16
    desc = dl.Desc(op=op, num_slots=wl.batch, H=wl.H, d_k=d, d_v=d, cap=cap, io_dtype=dt, scale=0.9)
    st_m, st_s = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    rec = Recorded(units=units)
    for blk in range(blocks):
        if int(st_m.log_len.max()) + T > cap:
            dl.merge(desc, st_m)
            dl.merge(desc, st_s)
        toks = [{k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()} for _ in range(T)]
        blk_tok = stack_tokens(toks)
        out_m = dl.decode_steps(desc, st_m, blk_tok["q"], blk_tok["k"], blk_tok["v"], blk_tok["g"],
                                beta=blk_tok["beta"], u_bonus=bonus)
        for t, tok in enumerate(toks):
            out_s = dl.decode_step(desc, st_s, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
            assert rel_err(f64(out_m[:, t]), f64(out_s)) <= (1e-6 if io == torch.float32 else 8e-3)
            rec.record_token(tok, out_m[:, t], wl)
        assert torch.equal(st_m.log_len, st_s.log_len) and torch.equal(st_m.K_log, st_s.K_log)
        assert rel_err(f64(st_m.decay_log), f64(st_s.decay_log)) <= 1e-6
        assert rel_err(f64(st_m.U_log), f64(st_s.U_log)) <= 1e-5
    assert rel_err(f64(st_m.S_base), f64(st_s.S_base)) <= 1e-5   # same merges of (almost) the same logs
    dl.merge(desc, st_m)
    torch.cuda.synchronize()
    assert int(st_m.status.item()) == 0
    rec.state_at, rec.states = [wl.steps], [f64(st_m.S_base[ub, uh])]
    ref = oracle_for(wl, rec, f64(S0[ub, uh]), f64(bonus[uh]) if bonus is not None else None, scale=0.9)
    assert rel_err(np.stack(rec.out), ref["out"]) <= out_tol(wl)
    assert rel_err(rec.states[0], ref["S"]) <= TOL_STATE


def test_rows_without_room_are_skipped_whole_and_grouped_heads_with_slot_indirection():
    import paper_2608_15533_b200 as dl

    cap, T, H, H_qk, d = 4, 3, 4, 2, 128
    wl = Workload("multi_edges", GDN, 4, H, d, 8, (cap,), num_slots=6)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    desc = dl.Desc(op=GDN, num_slots=6, H=H, d_k=d, d_v=d, cap=cap, io_dtype=dl.BF16, H_qk=H_qk)
    st_m, st_s = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    slot_idx = torch.tensor([5, -1, 0, 3], dtype=torch.int32, device=DEV)
    for st in (st_m, st_s):          # slot 3 already holds two entries: no room for three more
        st.log_len[3] = 2
    toks = [{k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()} for _ in range(T)]
    for tok in toks:
        tok["q"], tok["k"] = tok["q"][:, ::2].contiguous(), tok["k"][:, ::2].contiguous()
    blk = stack_tokens(toks)
    out = torch.full((4, T, H, d), 7.0, dtype=torch.bfloat16, device=DEV)
    dl.decode_steps(desc, st_m, blk["q"], blk["k"], blk["v"], blk["g"], beta=blk["beta"], slot_idx=slot_idx, out=out)
    torch.cuda.synchronize()
    assert int(st_m.status.item()) == dl.STATUS_LOG_FULL
    assert bool((out[1] == 7.0).all()) and bool((out[3] == 7.0).all())         # padding row, row without room
    assert st_m.log_len[:, 0].tolist() == [3, 0, 0, 2, 0, 3]
    ok = torch.tensor([5, -1, 0, -1], dtype=torch.int32, device=DEV)
    for t, tok in enumerate(toks):
        o = dl.decode_step(desc, st_s, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], slot_idx=ok)
        for b in (0, 2):
            assert rel_err(f64(out[b, t]), f64(o[b])) <= 8e-3
    assert torch.equal(st_m.K_log, st_s.K_log) and rel_err(f64(st_m.U_log), f64(st_s.U_log)) <= 1e-5


def test_block_length_outside_the_capacity_is_rejected():
    import paper_2608_15533_b200 as dl

    desc = dl.Desc(op=GDN, num_slots=2, H=2, d_k=64, d_v=64, cap=4, io_dtype=dl.F32)
    state = dl.State(desc, torch.zeros(2, 2, 64, 64, device=DEV))
    z = lambda *s: torch.zeros(*s, device=DEV)
    with pytest.raises(dl.DeltalogError) as e:
        dl.decode_steps(desc, state, z(2, 5, 2, 64), z(2, 5, 2, 64), z(2, 5, 2, 64), z(2, 5, 2), beta=z(2, 5, 2))
    assert e.value.code == dl.binding.ERR_CAP_RANGE
