"""DELTALOG_HINT_WALK_DOWN: the persistent decode kernels take the call's units from the last to the first.

It is an ordering request, not a promise: a unit's arithmetic does not depend on its place in a CTA's walk, so
outputs, appended log entries and lengths must be bit-identical to the default order -- on batches large enough
that every persistent CTA walks over several units, with a slot list that has padding rows, and when the bit
alternates from step to step (the way the benchmark uses it)."""
import dataclasses

import pytest
import torch

import workloads
from harness import make_desc
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("op,d,batch,H", [(GDN, 128, 40, 16), (KDA, 128, 21, 16), (RWKV6, 64, 90, 16)])
def test_walking_downwards_changes_no_bit(op, d, batch, H):
    import paper_2608_15533_b200 as dl

    cap, steps = 8, 8
    wl = Workload(f"walk_op{op}", op, batch, H, d, steps, (cap,), io_dtype=torch.bfloat16, num_slots=batch + 7)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus().to(DEV) if op == RWKV6 else None
    toks = [{k: (v.to(DEV) if v is not None else None) for k, v in src.token().items()} for _ in range(steps)]
    g = torch.Generator().manual_seed(11)
    slots = torch.randperm(wl.slots, generator=g)[:batch].to(torch.int32)
    slots[[2, batch // 2, batch - 1]] = -1                       # padding rows, also at the ends of the walk
    slot_idx = slots.to(DEV)
    base = make_desc(wl, cap, 1.0)

    def rollout(pattern):
        """pattern(t) -> hint bits of step t."""
        state = dl.State(base, S0.clone())
        outs = []
        for t, tok in enumerate(toks):
            desc = dataclasses.replace(base, hints=pattern(t))
            out = torch.full((batch, H, d), 7.0, dtype=wl.io_dtype, device=DEV)
            dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                           slot_idx=slot_idx, out=out)
            outs.append(out)
        torch.cuda.synchronize()
        assert int(state.status.item()) == 0
        return torch.stack(outs), state

    ref_out, ref = rollout(lambda t: 0)
    for name, pattern in (("always down", lambda t: dl.HINT_WALK_DOWN),
                          ("alternating", lambda t: dl.HINT_WALK_DOWN if t & 1 else 0),
                          ("alternating, chained", lambda t: (dl.HINT_WALK_DOWN if t & 1 else 0) |
                           (dl.HINT_BASE_UNTOUCHED | dl.HINT_SLOTS_STABLE if t else 0))):
        out, st = rollout(pattern)
        assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16)), name
        assert torch.equal(st.log_len, ref.log_len), name
        assert torch.equal(st.K_log.view(torch.int16), ref.K_log.view(torch.int16)), name
        assert torch.equal(st.U_log.contiguous().view(torch.uint8), ref.U_log.contiguous().view(torch.uint8)), name
        assert torch.equal(st.decay_log.view(torch.int32), ref.decay_log.view(torch.int32)), name
        assert torch.equal(st.S_base, S0), name                  # a decode step never writes the base
    live = slots[slots >= 0].long()
    assert int(ref.log_len[live].min()) == steps and int(ref.log_len.sum()) == steps * live.numel() * H


@pytest.mark.parametrize("op,d", [(GDN, 128), (RWKV6, 64)])
def test_eager_step_walking_downwards_changes_no_bit(op, d):
    import paper_2608_15533_b200 as dl

    batch, H = 24, 8
    wl = Workload(f"walk_eager_op{op}", op, batch, H, d, 4, (1,), io_dtype=torch.bfloat16)
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus().to(DEV) if op == RWKV6 else None
    toks = [{k: (v.to(DEV) if v is not None else None) for k, v in src.token().items()} for _ in range(4)]
    base = make_desc(wl, 1, 1.0)
    res = []
    for pattern in (lambda t: 0, lambda t: dl.HINT_WALK_DOWN if t & 1 else 0):
        S, outs = S0.clone(), []
        for t, tok in enumerate(toks):
            outs.append(dl.eager_step(dataclasses.replace(base, hints=pattern(t)), S, tok["q"], tok["k"], tok["v"], tok["g"],
                                      beta=tok["beta"], u_bonus=bonus))
        torch.cuda.synchronize()
        res.append((torch.stack(outs), S))
    assert torch.equal(res[0][0].view(torch.int16), res[1][0].view(torch.int16))
    assert torch.equal(res[0][1], res[1][1])
