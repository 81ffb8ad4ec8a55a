"""The 16-bit (bfloat16) dense state -- the variant the roofline discussion of Section 2.2 mentions.

All arithmetic stays fp32; only what is *stored* in the dense state is bf16.  With the log schedule the
dense base is stored once per materialisation (Eq. 5), with the eager recurrence once per token, so the
log schedule rounds the state `cap` times less often.  The oracle side of every comparison rounds at
exactly the same points (fp64 -> fp32 -> bf16, nearest even): `oracle.eager_rollout(state_bf16=True)`
for the eager kernel, and the exact recurrence over one cycle followed by `logical.round_bf16` for the
log schedule (tests/test_oracle_pins.py shows that this is what `LogState(store_base=round_bf16)` does).

Tolerances.  A stored element can differ from the oracle's by one bf16 ulp (2^-8 relative) when the
fp32 and the fp64 value fall on different sides of a rounding boundary, and such a flip feeds the
next cycle; so the state is compared at 2^-7 of max|ref| over a long rollout (two ulps of the largest
element), and exactly -- all elements equal except a small fraction one ulp apart -- after the first
store, where both sides start from identical states.  Outputs keep the 2e-2 bar of bf16 outputs.
"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from harness import Recorded, f64, rel_err
from oracle import logical
from workloads import GDN, GLA, KDA, LINATTN, RETNET, RWKV6, Workload

TOL_STATE_BF16 = 2.0 ** -7
TOL_OUT = 2e-2
ALL_OPS = [GDN, KDA, RWKV6, LINATTN, RETNET, GLA]


def _kw(op, beta, bonus):
    kw = {}
    if op in (GDN, KDA):
        kw["beta"] = beta
    if op == RWKV6:
        kw["bonus"] = bonus
    return kw


def schedule_oracle(op, S0, q, k, v, g, beta, bonus, boundaries):
    """Exact recurrence between the listed token counts, the state rounded to bf16 at each of them (the
    points where the log schedule stores its dense base); tokens after the last boundary stay in the log,
    unrounded.  Returns (out [T,N,d], stored states after each boundary, logical state after all T tokens)."""
    S = logical.round_bf16(S0)
    outs, states, t0 = [], [], 0
    for t1 in list(boundaries) + [q.shape[0]]:
        if t1 > t0:
            r = oracle.eager_rollout(op, S, q[t0:t1], k[t0:t1], v[t0:t1], g[t0:t1],
                                     **_kw(op, beta[t0:t1] if beta is not None else None, bonus))
            outs.append(r["out"])
            S = r["S"]
        if len(states) < len(boundaries):
            S = logical.round_bf16(S)
            states.append(S.copy())
        t0 = t1
    return np.concatenate(outs), states, S


def ulp_bf16(x):
    """Spacing of bfloat16 at |x| (normal range)."""
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(x), 2.0 ** -120))) - 7)


def assert_same_rounding(got, want, max_flip_fraction=0.01):
    """Equal except for a small fraction of elements that sit one ulp apart (plus, for elements far
    below the tile's magnitude, the fp32 accumulation error of the value that was rounded)."""
    diff = np.abs(got - want)
    flips = diff > 0
    assert flips.mean() <= max_flip_fraction, flips.mean()
    slack = 4e-6 * np.max(np.abs(want))
    assert np.all(diff[flips] <= 1.0001 * np.maximum(ulp_bf16(got[flips]), ulp_bf16(want[flips])) + slack)


# ---------------------------------------------------------------------------------------------
# CPU: what the variant costs in accuracy, on the oracle alone
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("op", [GDN, KDA, RWKV6])
def test_error_study_on_the_oracle(op):
    wl = Workload("b16_cpu", op, 1, 2, 32, 120, (16,))
    cap, T = 16, 120      # ends in the middle of a cycle: the state the next token would see
    src = workloads.TokenSource(wl, device="cpu")
    S0 = logical.round_bf16(f64(src.initial_state()).reshape(-1, wl.d, wl.d))
    bonus = src.bonus()
    bonus = np.tile(f64(bonus), (wl.batch, 1)) if bonus is not None else None
    toks = [src.token() for _ in range(T)]
    flat = lambda name: np.stack([f64(t[name]).reshape(wl.batch * wl.H, -1) for t in toks])
    q, k, v, g = flat("q"), flat("k"), flat("v"), flat("g")
    beta = flat("beta")[..., 0] if op != RWKV6 else None
    last = T // cap * cap   # the last materialisation
    exact = oracle.eager_rollout(op, S0, q, k, v, g, snapshot_at=[last], **_kw(op, beta, bonus))
    eager16 = oracle.eager_rollout(op, S0, q, k, v, g, state_bf16=True, **_kw(op, beta, bonus))
    out_log, stored, S_log = schedule_oracle(op, S0, q, k, v, g, beta, bonus, list(range(cap, T + 1, cap)))
    e_eager = rel_err(eager16["S"], exact["S"])
    e_stored = rel_err(stored[-1], exact["snapshots"][0])
    e_log = rel_err(S_log, exact["S"])
    # A state that has just been stored in 16 bits is half an ulp off, far above the 1e-4 bar of the fp32
    # state (which is why fp32 is the default) -- with the eager recurrence that is every token's state,
    # with the log schedule only the base right after a materialisation; the tokens that follow are
    # appended exactly while the operator's decay shrinks the base's rounding error, so the state a token
    # sees is on average much closer to the exact one, and so are the outputs.
    assert 1e-4 < e_eager < 5e-2 and 1e-4 < e_stored < 5e-2, (e_eager, e_stored)
    assert e_log < 0.5 * e_eager, (e_log, e_eager)
    rms = lambda x, r: float(np.sqrt(np.mean((x - r) ** 2)) / np.sqrt(np.mean(r ** 2)))
    assert rms(out_log, exact["out"]) < 0.7 * rms(eager16["out"], exact["out"]) < 5e-2


def test_abi_rejects_16_bit_state_with_fp32_io():
    import paper_2608_15533_b200 as dl

    lib = dl.load_library()
    import ctypes

    d = dl.Desc(op=dl.GDN, num_slots=1, H=1, d_k=64, d_v=64, cap=4, io_dtype=dl.F32, base_dtype=dl.BF16).c_struct()
    st = dl.binding._State(256, 256, 256, 256, 256, 0)
    rc = lib.deltalog_merge(ctypes.byref(d), ctypes.byref(st), None, 1, 0, None)
    assert rc == 2   # DELTALOG_ERR_UNSUPPORTED_SHAPE, nothing launched
    d = dl.Desc(op=dl.GDN, num_slots=1, H=1, d_k=64, d_v=64, cap=4, io_dtype=dl.BF16, base_dtype=7).c_struct()
    assert lib.deltalog_merge(ctypes.byref(d), ctypes.byref(st), None, 1, 0, None) == 1


# ---------------------------------------------------------------------------------------------
# GPU
# ---------------------------------------------------------------------------------------------
def _setup(op, d, cap, batch, H, steps, seed_name="b16_gpu"):
    import paper_2608_15533_b200 as dl

    wl = Workload(seed_name, op, batch, H, d, steps, (cap,))
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to("cuda").to(torch.bfloat16)
    bonus = src.bonus()
    bonus = bonus.to("cuda") if bonus is not None else None
    desc = dl.Desc(op=op, num_slots=batch, H=H, d_k=d, d_v=d, cap=cap, io_dtype=dl.BF16, base_dtype=dl.BF16)
    return dl, wl, src, S0, bonus, desc


def _arrays(rec, op):
    q, k, v, g = (np.stack(x) for x in (rec.q, rec.k, rec.v, rec.g))
    beta = np.stack(rec.beta) if rec.beta else None
    return q, k, v, g, beta


@pytest.mark.gpu
@pytest.mark.parametrize("op", ALL_OPS)
@pytest.mark.parametrize("d,cap,batch,H", [(128, 16, 40, 8), (64, 8, 24, 6), (128, 4, 3, 2)])
def test_log_schedule_with_16_bit_base(op, d, cap, batch, H):
    """Decode + append + merge over several cycles (enough units for the persistent kernel to take
    more than one unit per CTA at d = 128), the paper's fused merge step at every other boundary."""
    steps = 4 * cap + 3
    dl, wl, src, S0, bonus, desc = _setup(op, d, cap, batch, H, steps)
    state = dl.State(desc, S0.clone())
    assert state.S_base.dtype == torch.bfloat16
    units = [(b, h) for b in range(batch) for h in range(H)][:: max(1, batch * H // 48)]
    ub = torch.tensor([u[0] for u in units], device="cuda")
    uh = torch.tensor([u[1] for u in units], device="cuda")
    rec = Recorded(units=units)
    boundaries, got_states = [], []
    fused_next = False
    for t in range(steps):
        tok = {k_: (v_.to("cuda") if v_ is not None else None) for k_, v_ in src.token().items()}
        full = int(state.log_len[0, 0].item()) == cap
        if full and fused_next:
            out = dl.decode_merge_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
            boundaries.append(t + 1)
            got_states.append(f64(state.S_base[ub, uh]))
            fused_next = False
        else:
            if full:
                base_before = state.S_base.clone()
                dl.merge(desc, state)
                assert not torch.equal(base_before, state.S_base)
                boundaries.append(t)
                got_states.append(f64(state.S_base[ub, uh]))
                fused_next = True
            base_before = state.S_base.clone() if t < 3 else None
            out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
            if base_before is not None:
                assert torch.equal(base_before, state.S_base)     # the append never writes the base
        rec.record_token(tok, out, wl)
    dl.merge(desc, state)
    boundaries.append(steps)
    got_states.append(f64(state.S_base[ub, uh]))
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0 and int(state.log_len.abs().sum().item()) == 0

    q, k, v, g, beta = _arrays(rec, op)
    bonus_u = f64(bonus[uh]) if bonus is not None else None
    want_out, want_states, _ = schedule_oracle(op, f64(S0[ub, uh]), q, k, v, g, beta, bonus_u, boundaries)
    assert rel_err(np.stack(rec.out), want_out) <= TOL_OUT
    assert_same_rounding(got_states[0], want_states[0])           # first store: identical inputs on both sides
    for got, want in zip(got_states, want_states):
        assert rel_err(got, want) <= TOL_STATE_BF16
    # against the exact recurrence (no rounding anywhere) the variant drifts, but stays bounded
    exact = oracle.eager_rollout(op, f64(S0[ub, uh]), q, k, v, g, **_kw(op, beta, bonus_u))
    assert rel_err(got_states[-1], exact["S"]) <= 3e-2
    assert rel_err(np.stack(rec.out), exact["out"]) <= 3e-2


@pytest.mark.gpu
@pytest.mark.parametrize("op", ALL_OPS)
@pytest.mark.parametrize("d", [64, 128])
def test_eager_kernel_with_16_bit_state(op, d):
    steps, batch, H = 24, 5, 4
    dl, wl, src, S0, bonus, desc = _setup(op, d, 4, batch, H, steps, "b16_eager")
    S = S0.clone()
    units = [(b, h) for b in range(batch) for h in range(H)]
    ub = torch.tensor([u[0] for u in units], device="cuda")
    uh = torch.tensor([u[1] for u in units], device="cuda")
    rec = Recorded(units=units)
    first = None
    for t in range(steps):
        tok = {k_: (v_.to("cuda") if v_ is not None else None) for k_, v_ in src.token().items()}
        out = dl.eager_step(desc, S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus)
        rec.record_token(tok, out, wl)
        if t == 0:
            first = f64(S[ub, uh])
    torch.cuda.synchronize()
    q, k, v, g, beta = _arrays(rec, op)
    bonus_u = f64(bonus[uh]) if bonus is not None else None
    ref = oracle.eager_rollout(op, f64(S0[ub, uh]), q, k, v, g, state_bf16=True, snapshot_at=[1],
                               **_kw(op, beta, bonus_u))
    assert_same_rounding(first, ref["snapshots"][0])
    assert rel_err(f64(S[ub, uh]), ref["S"]) <= TOL_STATE_BF16
    assert rel_err(np.stack(rec.out), ref["out"]) <= TOL_OUT


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_16_bit_base_with_slots_blocks_of_tokens_and_reset(d):
    """The other entry points on a 16-bit base: slot indirection with padding rows, blocks of tokens in
    one launch (same results as single steps), predicate merges, slot reset with a new fp32 state."""
    op, cap, batch, H, T = GDN, 8, 6, 4, 4
    dl, wl, src, S0, bonus, desc = _setup(op, d, cap, batch, H, 2 * cap, "b16_misc")
    pool = 9
    desc = dl.Desc(op=op, num_slots=pool, H=H, d_k=d, d_v=d, cap=cap, io_dtype=dl.BF16, base_dtype=dl.BF16)
    Spool = torch.zeros(pool, H, d, d, dtype=torch.bfloat16, device="cuda")
    slots = torch.tensor([7, 2, -1, 5, 0, 8], dtype=torch.int32, device="cuda")
    live = slots >= 0
    Spool[slots[live].long()] = S0[live]
    a, b = dl.State(desc, Spool.clone()), dl.State(desc, Spool.clone())
    toks = [{k_: (v_.to("cuda") if v_ is not None else None) for k_, v_ in src.token().items()} for _ in range(2 * cap)]
    outs_a = []
    for t, tok in enumerate(toks):
        dl.merge(desc, a, slot_idx=slots, n=batch, only_if_full=True)
        outs_a.append(dl.decode_step(desc, a, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], slot_idx=slots))
    outs_b = []
    for t0 in range(0, 2 * cap, T):
        dl.merge(desc, b, slot_idx=slots, n=batch, only_if_full=True)
        blk = {k_: torch.stack([toks[t0 + i][k_] for i in range(T)], dim=1).contiguous() for k_ in ("q", "k", "v", "g", "beta")}
        o = dl.decode_steps(desc, b, blk["q"], blk["k"], blk["v"], blk["g"], beta=blk["beta"], slot_idx=slots)
        outs_b += [o[:, i] for i in range(T)]
    torch.cuda.synchronize()
    assert int(a.status.item()) == 0 and int(b.status.item()) == 0
    for oa, ob in zip(outs_a, outs_b):
        assert rel_err(f64(ob[live]), f64(oa[live])) <= 2e-2
    dl.merge(desc, a, slot_idx=slots, n=batch)
    dl.merge(desc, b, slot_idx=slots, n=batch)
    assert rel_err(f64(b.S_base), f64(a.S_base)) <= TOL_STATE_BF16
    untouched = [s for s in range(pool) if s not in slots.tolist()]
    assert torch.equal(a.S_base[untouched], Spool[untouched])
    # slot reset installs the rounded fp32 state and empties the log
    S_new = torch.randn(2, H, d, d, device="cuda") * 0.1
    dl.decode_step(desc, a, toks[0]["q"], toks[0]["k"], toks[0]["v"], toks[0]["g"], beta=toks[0]["beta"], slot_idx=slots)
    which = torch.tensor([5, 1], dtype=torch.int32, device="cuda")
    dl.reset_slots(desc, a, slot_idx=which, S_init=S_new)
    torch.cuda.synchronize()
    assert torch.equal(a.S_base[which.long()], S_new.to(torch.bfloat16))
    assert int(a.log_len[which.long()].abs().sum().item()) == 0 and int(a.log_len[7, 0].item()) == 1


@pytest.mark.gpu
def test_16_bit_base_at_the_full_size_of_configuration_1():
    """Configuration 1's shape (128 x 32 heads, d = 128, cap 16) with the 16-bit base, launched the way the
    benchmark launches it (a merge after every 16th step, decode steps behind a decode step chained);
    a sample of units goes through the oracle that rounds at the same points."""
    import paper_2608_15533_b200 as dl

    base = workloads.CONFIGS[1]
    cap, steps = 16, 3 * 16 + 5
    wl = Workload("b16_full", base.op, base.batch, base.H, base.d, steps, (cap,))
    src = workloads.TokenSource(wl, device="cuda")
    S0 = src.initial_state().to(torch.bfloat16)
    desc = dl.Desc(op=wl.op, num_slots=wl.batch, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=dl.BF16,
                   base_dtype=dl.BF16)
    desc_c = dl.Desc(op=wl.op, num_slots=wl.batch, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=dl.BF16,
                     base_dtype=dl.BF16, hints=dl.HINT_BASE_UNTOUCHED)
    state = dl.State(desc, S0.clone())
    rng = np.random.default_rng(7)
    picks = sorted({0, wl.batch * wl.H - 1, *rng.choice(wl.batch * wl.H, 14, replace=False).tolist()})
    units = [(p // wl.H, p % wl.H) for p in picks]
    ub = torch.tensor([u[0] for u in units], device="cuda")
    uh = torch.tensor([u[1] for u in units], device="cuda")
    rec = Recorded(units=units)
    boundaries, got_states = [], []
    for t in range(steps):
        tok = src.token()
        if t and t % cap == 0:
            dl.merge(desc, state)
            boundaries.append(t)
            got_states.append(f64(state.S_base[ub, uh]))
        out = dl.decode_step(desc if t % cap == 0 else desc_c, state, tok["q"], tok["k"], tok["v"], tok["g"],
                             beta=tok["beta"])
        rec.record_token(tok, out, wl)
    dl.merge(desc, state)
    boundaries.append(steps)
    got_states.append(f64(state.S_base[ub, uh]))
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    q, k, v, g, beta = _arrays(rec, wl.op)
    want_out, want_states, _ = schedule_oracle(wl.op, f64(S0[ub, uh]), q, k, v, g, beta, None, boundaries)
    assert rel_err(np.stack(rec.out), want_out) <= TOL_OUT
    assert_same_rounding(got_states[0], want_states[0])
    for got, want in zip(got_states, want_states):
        assert rel_err(got, want) <= TOL_STATE_BF16
