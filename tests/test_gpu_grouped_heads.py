"""Grouped query/key heads (several value heads share one query/key head, as in the GDN and KDA
layers of released checkpoints): q and k are [B, H_qk, d]; the result must be bit-identical to the
same run with q and k expanded to one copy per state head, which the oracle then checks."""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, Recorded, f64, oracle_for, out_tol, rel_err
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run(wl, cap, H_qk, cycle, steps):
    import paper_2608_15533_b200 as dl

    G = wl.H // H_qk
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    io = dl.F32 if wl.io_dtype == torch.float32 else dl.BF16
    mk = lambda hqk: dl.Desc(op=wl.op, num_slots=wl.slots, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=io,
                             scale=0.8, H_qk=hqk)
    desc_g, desc_x = mk(H_qk), mk(0)
    st_g, st_x = dl.State(desc_g, S0.clone()), dl.State(desc_x, S0.clone())
    Se_g, Se_x = S0.clone(), S0.clone()
    units = [(b, h) for b in range(wl.batch) for h in range(wl.H)]
    rec = Recorded(units=units)
    for t in range(steps):
        tok = {k_: (v_.to(DEV) if v_ is not None else None) for k_, v_ in src.token().items()}
        qg, kg = tok["q"][:, ::G].contiguous(), tok["k"][:, ::G].contiguous()          # [B, H_qk, d]
        qx, kx = qg.repeat_interleave(G, dim=1), kg.repeat_interleave(G, dim=1)          # one copy per state head
        kw = dict(beta=tok["beta"], u_bonus=bonus)
        full = bool((st_g.log_len == cap).all())
        if cycle == "split" and full:
            dl.merge(desc_g, st_g)
            dl.merge(desc_x, st_x)
        fn = dl.decode_merge_step if (cycle == "paper" and full) else dl.decode_step
        out_g = fn(desc_g, st_g, qg, kg, tok["v"], tok["g"], **kw)
        out_x = fn(desc_x, st_x, qx, kx, tok["v"], tok["g"], **kw)
        assert torch.equal(out_g, out_x)
        oe_g = dl.eager_step(desc_g, Se_g, qg, kg, tok["v"], tok["g"], **kw)
        oe_x = dl.eager_step(desc_x, Se_x, qx, kx, tok["v"], tok["g"], **kw)
        assert torch.equal(oe_g, oe_x)
        rec.record_token(dict(tok, q=qx, k=kx), out_g, wl)
    dl.merge(desc_g, st_g)
    dl.merge(desc_x, st_x)
    torch.cuda.synchronize()
    assert torch.equal(st_g.S_base, st_x.S_base) and torch.equal(Se_g, Se_x)
    assert torch.equal(st_g.K_log, st_x.K_log) and int(st_g.status.item()) == 0
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    rec.state_at, rec.states = [steps], [f64(st_g.S_base[ub, uh])]
    ref = oracle_for(wl, rec, f64(S0[ub, uh]), f64(bonus[uh]) if bonus is not None else None, scale=0.8)
    assert rel_err(np.stack(rec.out), ref["out"]) <= out_tol(wl)
    assert rel_err(rec.states[0], ref["S"]) <= TOL_STATE


@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("H,H_qk", [(4, 2), (6, 1)])
@pytest.mark.parametrize("cycle", ["split", "paper"])
def test_grouped_heads_equal_expanded_heads(op, d, H, H_qk, cycle):
    wl = Workload(f"gqa_op{op}", op, 3, H, d, 20, (4,))
    run(wl, 4, H_qk, cycle, 20)


def test_grouped_heads_through_the_persistent_kernel_and_the_host_entry_point():
    import paper_2608_15533_b200 as dl

    wl = Workload("gqa_wide", GDN, 48, 8, 128, 20, (16,))
    run(wl, 16, 2, "split", 20)
    # host-buffer entry point: q and k are copied with their own (smaller) size
    desc = dl.Desc(op=GDN, num_slots=4, H=4, d_k=128, d_v=128, cap=4, io_dtype=dl.BF16, H_qk=2)
    src = workloads.TokenSource(Workload("gqa_host", GDN, 4, 4, 128, 1, (4,)), device="cpu")
    S0 = src.initial_state().to(DEV)
    st_a, st_b = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    tok = src.token()
    q, k = tok["q"][:, ::2].contiguous(), tok["k"][:, ::2].contiguous()
    staging = dl.HostStaging(desc, 4, DEV)
    host = [t.pin_memory() for t in (q, k, tok["v"], tok["g"], tok["beta"])]
    host_out = torch.empty(4, 4, 128, dtype=torch.bfloat16).pin_memory()
    dl.decode_step_host(desc, st_a, staging, *host, host_out)
    ref = dl.decode_step(desc, st_b, q.to(DEV), k.to(DEV), tok["v"].to(DEV), tok["g"].to(DEV), beta=tok["beta"].to(DEV))
    torch.cuda.synchronize()
    assert torch.equal(host_out.to(DEV), ref)


def test_descriptor_rejects_head_counts_that_do_not_divide():
    import paper_2608_15533_b200 as dl

    desc = dl.Desc(op=GDN, num_slots=2, H=4, d_k=64, d_v=64, cap=4, io_dtype=dl.F32, H_qk=3)
    S0 = torch.zeros(2, 4, 64, 64, device=DEV)
    state = dl.State(desc, S0)
    z = torch.zeros(2, 3, 64, device=DEV)
    with pytest.raises(dl.DeltalogError):
        dl.decode_step(desc, state, z, z, torch.zeros(2, 4, 64, device=DEV), torch.zeros(2, 4, device=DEV),
                       beta=torch.zeros(2, 4, device=DEV))
