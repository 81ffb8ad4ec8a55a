"""Memory discipline and schedule switches.

* Guard bands: every tensor the library writes (base, the three log tensors, lengths, status, the
  output) is carved out of one allocation with sentinel-filled bands before and after it; after
  rollouts through every entry point that writes (decode, blocks of tokens, merge, fused merge step,
  slot hand-over, eager kernel) every band still holds the sentinel -- no kernel writes outside the
  tensors it was given, at any capacity or shape, including the ragged tail of the batch.
* The reverse switch: a state advanced by the eager kernel is handed to the log schedule (its dense
  state becomes the base, logs empty) and continues there; the result is the oracle's.
"""
import numpy as np
import pytest
import torch

import workloads
from harness import TOL_STATE, f64, make_desc, rel_err
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"
BAND = 4096          # bytes of sentinel on either side of every tensor
SENTINEL = 0x5A


class Guarded:
    """Tensors carved out of one byte buffer with sentinel bands between them."""

    def __init__(self):
        self.specs, self.total = [], BAND

    def add(self, name, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.specs.append((name, self.total, n, shape, dtype))
        self.total += (n + 255) // 256 * 256 + BAND

    def build(self):
        self.buf = torch.full((self.total,), SENTINEL, dtype=torch.uint8, device=DEV)
        self.mask = torch.ones(self.total, dtype=torch.bool, device=DEV)
        out = {}
        for name, off, n, shape, dtype in self.specs:
            out[name] = self.buf[off:off + n].view(dtype).view(*shape)
            self.mask[off:off + n] = False
        return out

    def intact(self):
        return bool((self.buf[self.mask] == SENTINEL).all())


@pytest.mark.parametrize("op,dk,dv,io,cap", [(GDN, 128, 128, torch.bfloat16, 16), (KDA, 128, 128, torch.bfloat16, 8),
                                             (RWKV6, 64, 64, torch.bfloat16, 16), (GDN, 64, 64, torch.float32, 5),
                                             (KDA, 128, 64, torch.bfloat16, 4), (RWKV6, 64, 128, torch.float32, 8)])
def test_no_kernel_writes_outside_the_tensors_it_was_given(op, dk, dv, io, cap):
    import paper_2608_15533_b200 as dl

    wl = Workload("guard", op, 37, 5, dk, 2 * cap + 3, (cap,), io_dtype=io, d_v=dv, num_slots=41)   # 185 units: a ragged tail
    desc = make_desc(wl, cap)
    src = workloads.TokenSource(wl, device=DEV)
    S0 = src.initial_state()
    bonus = src.bonus()
    g = Guarded()
    ulog = torch.float32 if op in (GDN, KDA) else io
    g.add("S_base", (wl.slots, wl.H, dk, dv), torch.float32)
    g.add("K_log", (wl.slots, wl.H, cap, dk), io)
    g.add("U_log", (wl.slots, wl.H, cap, dv), ulog)
    g.add("decay_log", (wl.slots, wl.H, cap, desc.d_lambda), torch.float32)
    g.add("log_len", (wl.slots, wl.H), torch.int32)
    g.add("status", (1,), torch.int32)
    g.add("out", (wl.batch, wl.H, dv), io)
    g.add("out_T", (wl.batch, 2, wl.H, dv), io)
    g.add("S_eager", (wl.slots, wl.H, dk, dv), torch.float32)
    t = g.build()
    state = dl.State(desc, S0.clone())
    for name in ("S_base", "K_log", "U_log", "decay_log", "log_len", "status"):
        t[name].copy_(getattr(state, name))
        setattr(state, name, t[name])
    t["S_eager"].copy_(S0)
    slots = workloads.slot_permutation(wl, pad_every=7).to(DEV)
    kw = lambda tok: dict(beta=tok["beta"], u_bonus=bonus, slot_idx=slots)
    for i in range(wl.steps):
        tok = src.token()
        if i % (cap + 1) == cap:
            dl.decode_merge_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], out=t["out"], **kw(tok))
        else:
            dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], out=t["out"], **kw(tok))
        dl.eager_step(desc, t["S_eager"], tok["q"], tok["k"], tok["v"], tok["g"], out=t["out"], status=t["status"], **kw(tok))
    dl.merge(desc, state, slot_idx=slots, n=wl.batch)
    if cap >= 2:   # a block of two tokens, then the predicate merge and a slot hand-over
        a, b = src.token(), src.token()
        cat = lambda n: torch.stack([a[n], b[n]], dim=1).contiguous() if a[n] is not None else None
        dl.decode_steps(desc, state, cat("q"), cat("k"), cat("v"), cat("g"), beta=cat("beta"), u_bonus=bonus, slot_idx=slots,
                        out=t["out_T"])
    dl.merge(desc, state, slot_idx=slots, n=wl.batch, only_if_full=True)
    dl.reset_slots(desc, state, slot_idx=slots[:3].contiguous(), S_init=torch.randn(3, wl.H, dk, dv, device=DEV))
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    assert g.intact()


@pytest.mark.parametrize("op,d", [(GDN, 128), (KDA, 64), (RWKV6, 64)])
def test_switch_from_the_eager_kernel_to_the_log_schedule(op, d):
    import oracle
    import paper_2608_15533_b200 as dl

    wl = Workload("reverse_switch", op, 6, 4, d, 30, (8,))
    cap, n_eager = 8, 11
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    toks = [{k: (v.to(DEV) if v is not None else None) for k, v in src.token().items()} for _ in range(wl.steps)]
    desc = make_desc(wl, cap)
    S = S0.clone()
    outs = [dl.eager_step(desc, S, t["q"], t["k"], t["v"], t["g"], beta=t["beta"], u_bonus=bonus) for t in toks[:n_eager]]
    state = dl.State(desc, S)            # the eager state is the base of an empty log
    for i, t in enumerate(toks[n_eager:]):
        if i and i % cap == 0:
            dl.merge(desc, state)
        outs.append(dl.decode_step(desc, state, t["q"], t["k"], t["v"], t["g"], beta=t["beta"], u_bonus=bonus))
    dl.merge(desc, state)
    torch.cuda.synchronize()
    N = wl.batch * wl.H
    flat = lambda name: np.stack([f64(t[name]).reshape(N, -1) for t in toks])
    ref = oracle.eager_rollout(op, f64(S0).reshape(N, d, d), flat("q"), flat("k"), flat("v"), flat("g"),
                               beta=flat("beta")[..., 0] if toks[0]["beta"] is not None else None,
                               bonus=np.tile(f64(bonus), (wl.batch, 1)) if bonus is not None else None)
    assert rel_err(np.stack([f64(o).reshape(N, d) for o in outs]), ref["out"]) <= 2e-2
    assert rel_err(f64(state.S_base).reshape(N, d, d), ref["S"]) <= TOL_STATE
    assert int(state.status.item()) == 0
