"""Numeric edge cases on every CUDA path -- the decode kernels (persistent pipelined at head size 128,
one CTA per unit at head size 64, blocks of tokens), the merge, the fused merge step and the eager
kernel -- against the fp64 oracle and against what the mathematics fixes:

* ``g = 0`` with ``beta = 0``: the state never changes; the merged base is BIT-identical to the initial
  one, every stored value-side factor is exactly zero, ``out = scale * S0^T q``;
* ``beta = 1`` with unit keys and ``q = k``: the delta rule recalls the value, ``out = v``, whatever
  the decay;
* strong decay (``g = -30`` per step over a capacity-64 cycle): ``exp`` of the accumulated decay
  underflows to zero -- that must give zeros, never NaN or infinity;
* a zero initial state; zero keys; a capacity-64 cycle with per-key decay accumulating to |Lambda| ~ 100
  (the fp32 difference ``lbar - Lambda[i]`` then carries an absolute error of ~ 1e-5).
"""
import numpy as np
import pytest
import torch

from harness import TOL_OUT_BF16, TOL_OUT_F32, TOL_STATE, f64, rel_err
from workloads import GDN, KDA, RWKV6

pytestmark = pytest.mark.gpu
DEV = "cuda"
VEC = (KDA, RWKV6)


def make_tokens(op, B, H, d, io, steps, seed, g_value=None, beta_value=None, unit_keys=False, zero_key_every=0,
                g_vec_mean=None):
    gen = torch.Generator().manual_seed(seed)
    rn = lambda *s: torch.randn(*s, generator=gen)
    toks = []
    for t in range(steps):
        q, k, v = rn(B, H, d), rn(B, H, d), rn(B, H, d)
        if op != RWKV6:
            q, k = q / q.norm(dim=-1, keepdim=True), k / k.norm(dim=-1, keepdim=True)
        if unit_keys:       # one-hot keys: norm exactly 1 in every dtype; the query asks for the value just written
            idx = torch.randint(0, d, (B, H, 1), generator=gen)
            k = torch.zeros(B, H, d).scatter_(-1, idx, 1.0)
            q = k.clone()
        if zero_key_every and t % zero_key_every == 1:
            k = torch.zeros(B, H, d)
        gshape = (B, H, d) if op in VEC else (B, H)
        if g_value is not None:
            g = torch.full(gshape, float(g_value))
        elif g_vec_mean is not None:
            g = g_vec_mean + 0.1 * rn(*gshape).clamp(-2, 2)
        elif op == RWKV6:
            g = -torch.exp(rn(*gshape) * 0.5 - 0.5)
        else:
            g = -torch.nn.functional.softplus(rn(*gshape))
        beta = None
        if op != RWKV6:
            beta = torch.full((B, H), float(beta_value)) if beta_value is not None else torch.sigmoid(rn(B, H))
        toks.append({"q": q.to(io).to(DEV), "k": k.to(io).to(DEV), "v": v.to(io).to(DEV),
                     "g": g.contiguous().to(DEV), "beta": beta.to(DEV) if beta is not None else None})
    return toks


def run_paths(op, d, io, cap, S0, toks, bonus, scale=1.0, block=4):
    """Every CUDA path over the same tokens -> {path: (outs [T,B,H,d], final dense state [B,H,d,d], status)}."""
    import paper_2608_15533_b200 as dl

    B, H = S0.shape[0], S0.shape[1]
    desc = dl.Desc(op=op, num_slots=B, H=H, d_k=d, d_v=d, cap=cap, io_dtype=dl.F32 if io == torch.float32 else dl.BF16,
                   scale=scale)
    kw = lambda t: dict(beta=t["beta"], u_bonus=bonus)
    res = {}
    # split cycle: append until the log is full, token-less merge, ...
    st = dl.State(desc, S0.clone())
    outs = []
    for i, t in enumerate(toks):
        if i and i % cap == 0:
            dl.merge(desc, st)
        outs.append(dl.decode_step(desc, st, t["q"], t["k"], t["v"], t["g"], **kw(t)))
    logs = (st.U_log.clone(), st.log_len.clone())
    dl.merge(desc, st)
    res["split"] = (torch.stack(outs), st.S_base.clone(), int(st.status.item()), logs)
    # the paper's cycle: cap appends, then the fused merge step
    st = dl.State(desc, S0.clone())
    outs = [(dl.decode_merge_step if i % (cap + 1) == cap else dl.decode_step)(desc, st, t["q"], t["k"], t["v"], t["g"], **kw(t))
            for i, t in enumerate(toks)]
    dl.merge(desc, st)
    res["paper"] = (torch.stack(outs), st.S_base.clone(), int(st.status.item()), None)
    # blocks of `block` tokens per call
    if cap % block == 0 and len(toks) % block == 0:
        st = dl.State(desc, S0.clone())
        outs = []
        for i in range(0, len(toks), block):
            if i and i % cap == 0:
                dl.merge(desc, st)
            blk = toks[i:i + block]
            cat = lambda n: torch.stack([t[n] for t in blk], dim=1).contiguous()
            o = dl.decode_steps(desc, st, cat("q"), cat("k"), cat("v"), cat("g"),
                                beta=cat("beta") if blk[0]["beta"] is not None else None, u_bonus=bonus)
            outs.extend(o.unbind(1))
        dl.merge(desc, st)
        res["blocks"] = (torch.stack(outs), st.S_base.clone(), int(st.status.item()), None)
    # eager dense kernel
    S = S0.clone()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    outs = [dl.eager_step(desc, S, t["q"], t["k"], t["v"], t["g"], status=status, **kw(t)) for t in toks]
    res["eager"] = (torch.stack(outs), S, int(status.item()), None)
    torch.cuda.synchronize()
    return res


def reference(op, S0, toks, bonus, scale=1.0):
    import oracle

    B, H, d = S0.shape[0], S0.shape[1], S0.shape[2]
    N = B * H
    flat = lambda n: np.stack([f64(t[n]).reshape(N, -1) for t in toks])
    return oracle.eager_rollout(op, f64(S0).reshape(N, d, d), flat("q"), flat("k"), flat("v"), flat("g"),
                                beta=flat("beta")[..., 0] if toks[0]["beta"] is not None else None,
                                bonus=np.tile(f64(bonus), (B, 1)) if bonus is not None else None, scale=scale)


def check_against_oracle(op, d, io, res, ref, S0):
    N = S0.shape[0] * S0.shape[1]
    tol_out = TOL_OUT_F32 if io == torch.float32 else TOL_OUT_BF16
    for path, (outs, S, status, _) in res.items():
        assert status == 0, path
        assert torch.isfinite(outs.float()).all() and torch.isfinite(S).all(), f"{path}: NaN or infinity"
        o = f64(outs).reshape(len(outs), N, d)
        den_out = max(np.max(np.abs(ref["out"])), 1e-30)
        assert np.max(np.abs(o - ref["out"])) / den_out <= tol_out, path
        den_S = max(np.max(np.abs(ref["S"])), 1e-30)
        assert np.max(np.abs(f64(S).reshape(N, d, d) - ref["S"])) / den_S <= TOL_STATE, path


def shapes(d):
    """Wide enough at head size 128 for several units per persistent CTA."""
    return (40, 8) if d == 128 else (5, 3)


def state0(B, H, d, seed=0, zero=False):
    if zero:
        return torch.zeros(B, H, d, d, device=DEV)
    return (0.1 * torch.randn(B, H, d, d, generator=torch.Generator().manual_seed(seed))).to(DEV)


def bonus_for(op, H, d):
    return (0.1 * torch.randn(H, d, generator=torch.Generator().manual_seed(5))).to(DEV) if op == RWKV6 else None


@pytest.mark.parametrize("op", [GDN, KDA])
@pytest.mark.parametrize("d,io,cap", [(128, torch.bfloat16, 8), (64, torch.float32, 8), (64, torch.bfloat16, 5)])
def test_unit_decay_and_zero_beta_leave_the_state_bit_identical(op, d, io, cap):
    B, H = shapes(d)
    S0 = state0(B, H, d)
    toks = make_tokens(op, B, H, d, io, 24 if cap % 4 == 0 else 16, 11, g_value=0.0, beta_value=0.0)
    res = run_paths(op, d, io, cap, S0, toks, None, scale=0.5)
    for path, (outs, S, status, logs) in res.items():
        assert status == 0
        assert torch.equal(S, S0), f"{path}: the base changed"
        if logs is not None:
            assert bool((logs[0] == 0).all()) and int(logs[1].max()) > 0      # every stored b is exactly zero
        want = 0.5 * torch.einsum("bhkv,tbhk->tbhv", S0.double(), torch.stack([t["q"] for t in toks]).double())
        tol = TOL_OUT_F32 if io == torch.float32 else TOL_OUT_BF16
        assert rel_err(f64(outs), want.cpu().numpy()) <= tol, path


@pytest.mark.parametrize("op", [GDN, KDA])
@pytest.mark.parametrize("d,io", [(128, torch.bfloat16), (64, torch.float32)])
def test_delta_rule_recalls_the_value_for_unit_keys(op, d, io):
    B, H = shapes(d)
    cap = 8
    S0 = state0(B, H, d)
    toks = make_tokens(op, B, H, d, io, 20, 12, beta_value=1.0, unit_keys=True)
    res = run_paths(op, d, io, cap, S0, toks, None)
    v = torch.stack([t["v"] for t in toks]).double()
    for path, (outs, S, status, _) in res.items():
        assert status == 0
        # fp32 arithmetic: (v - y) + y returns v up to one rounding of values of the state's size
        tol = 2e-6 if io == torch.float32 else 2.0 ** -8
        assert float((outs.double() - v).abs().max() / v.abs().max()) <= tol, path
    check_against_oracle(op, d, io, res, reference(op, S0, toks, None), S0)


@pytest.mark.parametrize("op,d,io", [(GDN, 128, torch.bfloat16), (KDA, 128, torch.bfloat16), (GDN, 64, torch.float32),
                                     (KDA, 64, torch.bfloat16), (RWKV6, 64, torch.bfloat16), (RWKV6, 128, torch.bfloat16)])
def test_strong_decay_underflows_to_zero_without_nan(op, d, io):
    B, H = shapes(d)
    cap = 64
    S0 = state0(B, H, d)
    bonus = bonus_for(op, H, d)
    toks = make_tokens(op, B, H, d, io, 72, 13, g_value=-30.0)     # accumulated decay reaches -1920: exp underflows
    res = run_paths(op, d, io, cap, S0, toks, bonus)
    check_against_oracle(op, d, io, res, reference(op, S0, toks, bonus), S0)
    # nothing of S0 is left after the first token (e^-30 ~ 1e-13): the run from a zero state ends in the same state
    res0 = run_paths(op, d, io, cap, torch.zeros_like(S0), toks, bonus)
    assert float((res["split"][1] - res0["split"][1]).abs().max()) <= 1e-10


@pytest.mark.parametrize("op,d,io", [(GDN, 128, torch.bfloat16), (KDA, 64, torch.float32), (RWKV6, 64, torch.bfloat16),
                                     (KDA, 128, torch.bfloat16), (RWKV6, 128, torch.bfloat16)])
def test_zero_initial_state_and_zero_keys(op, d, io):
    B, H = shapes(d)
    cap = 8
    S0 = state0(B, H, d, zero=True)
    bonus = bonus_for(op, H, d)
    toks = make_tokens(op, B, H, d, io, 20, 14, zero_key_every=3)
    res = run_paths(op, d, io, cap, S0, toks, bonus)
    ref = reference(op, S0, toks, bonus)
    check_against_oracle(op, d, io, res, ref, S0)
    # first token from a zero state: GDN / KDA out = beta (q.k) v (closed form), RWKV6 out = (r.(u*k)) v
    t0 = toks[0]
    qk = (t0["q"].double() * t0["k"].double() * (bonus.double() if bonus is not None else 1.0)).sum(-1, keepdim=True)
    want = qk * t0["v"].double() * (t0["beta"].double().unsqueeze(-1) if t0["beta"] is not None else 1.0)
    tol = TOL_OUT_F32 if io == torch.float32 else TOL_OUT_BF16
    for path, (outs, _, _, _) in res.items():
        assert float((outs[0].double() - want).abs().max() / want.abs().max()) <= tol, path


@pytest.mark.parametrize("op,d,io", [(KDA, 128, torch.bfloat16), (KDA, 64, torch.float32), (RWKV6, 64, torch.bfloat16),
                                     (KDA, 128, torch.float32)])
def test_capacity_64_with_large_accumulated_per_key_decay(op, d, io):
    B, H = shapes(d)
    cap = 64
    S0 = state0(B, H, d)
    bonus = bonus_for(op, H, d)
    toks = make_tokens(op, B, H, d, io, 132, 15, g_vec_mean=-1.55)   # |Lambda| reaches ~ 100 at the end of a cycle
    res = run_paths(op, d, io, cap, S0, toks, bonus)
    check_against_oracle(op, d, io, res, reference(op, S0, toks, bonus), S0)
