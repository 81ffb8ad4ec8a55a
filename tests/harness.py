"""Shared test harness: drives the CUDA library over a seeded token stream, records what a sample of
(sequence, head) units saw and produced, and runs the fp64 oracle on exactly those units."""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

import workloads
from workloads import GDN, RWKV6, Workload

# tolerances of the parity bar: max|x - ref| / max|ref| over the compared tensor
TOL_STATE = 1e-4       # fp32 state vs fp64 oracle
TOL_OUT_BF16 = 2e-2    # bf16 outputs
TOL_OUT_F32 = 1e-4     # fp32 outputs (all-fp32 configuration)


def rel_err(x, ref) -> float:
    """Global-max-normalised error: max|x - ref| / max|ref|."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.max(np.abs(ref))
    return float(np.max(np.abs(x - ref)) / (denom if denom > 0 else 1.0))


def out_tol(wl: Workload) -> float:
    return TOL_OUT_F32 if wl.io_dtype == torch.float32 else TOL_OUT_BF16


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def make_desc(wl: Workload, cap: int, scale: float = 1.0):
    import paper_2608_15533_b200 as dl

    io = dl.F32 if wl.io_dtype == torch.float32 else dl.BF16
    return dl.Desc(op=wl.op, num_slots=wl.slots, H=wl.H, d_k=wl.d, d_v=wl.dv, cap=cap, io_dtype=io, scale=scale)


@dataclass
class Recorded:
    """Per-token inputs and outputs of the sampled units, gathered to the host."""

    units: List[Tuple[int, int]]                      # (batch row, head)
    q: List[np.ndarray] = field(default_factory=list)
    k: List[np.ndarray] = field(default_factory=list)
    v: List[np.ndarray] = field(default_factory=list)
    g: List[np.ndarray] = field(default_factory=list)
    beta: List[np.ndarray] = field(default_factory=list)
    out: List[np.ndarray] = field(default_factory=list)
    start: List[int] = field(default_factory=list)         # first global step each unit takes part in
    state_at: List[int] = field(default_factory=list)      # global step counts after which the state was recorded
    states: List[np.ndarray] = field(default_factory=list)  # [N, d, d] each

    def record_token(self, tok: Dict[str, torch.Tensor], out: torch.Tensor, wl: Workload):
        b = torch.tensor([u[0] for u in self.units], device=out.device)
        h = torch.tensor([u[1] for u in self.units], device=out.device)
        self.q.append(f64(tok["q"][b, h]))
        self.k.append(f64(tok["k"][b, h]))
        self.v.append(f64(tok["v"][b, h]))
        if tok["g"] is not None:
            self.g.append(f64(tok["g"][b, h]).reshape(len(self.units), -1))
        else:  # plain linear attention has no gate
            self.g.append(np.zeros((len(self.units), 1)))
        if tok["beta"] is not None:
            self.beta.append(f64(tok["beta"][b, h]))
        self.out.append(f64(out[b, h]))


def sample_units(wl: Workload, n: int, seed: int = 1) -> List[Tuple[int, int]]:
    """``n`` distinct (batch row, head) pairs, always including the first and the last unit."""
    total = wl.batch * wl.H
    rng = np.random.default_rng(seed)
    picks = {0, total - 1}
    while len(picks) < min(n, total):
        picks.add(int(rng.integers(total)))
    return [(p // wl.H, p % wl.H) for p in sorted(picks)]


def oracle_for(wl: Workload, rec: Recorded, S0_units: np.ndarray, bonus_units: Optional[np.ndarray],
               scale: float = 1.0):
    """Run the fp64 eager oracle on the recorded units.

    Units that joined late (``rec.start``) consume only the tokens from their first step on.  Returns
    ``dict(out [T,N,d] (NaN before a unit's start), b [T,N,d], S [N,d,d], snapshots [n_snap,N,d,d])``
    with snapshots taken after the global step counts in ``rec.state_at``.
    """
    import oracle

    q, k, v, g = (np.stack(x) for x in (rec.q, rec.k, rec.v, rec.g))
    beta = np.stack(rec.beta) if rec.beta else None
    T, N, d = v.shape
    start = rec.start if rec.start else [0] * N
    res = {"out": np.full((T, N, d), np.nan), "b": np.full((T, N, d), np.nan), "S": np.empty_like(S0_units),
           "snapshots": np.full((len(rec.state_at), N, S0_units.shape[1], d), np.nan)}
    for s0 in sorted(set(start)):
        idx = [n for n in range(N) if start[n] == s0]
        snaps = [(i, a - s0) for i, a in enumerate(rec.state_at) if a - s0 >= 1]
        r = oracle.eager_rollout(
            wl.op, S0_units[idx], q[s0:, idx], k[s0:, idx], v[s0:, idx], g[s0:, idx],
            beta=beta[s0:, idx] if beta is not None else None,
            bonus=bonus_units[idx] if bonus_units is not None else None, scale=scale,
            snapshot_at=[a for _, a in snaps])
        res["out"][s0:, idx] = r["out"]
        res["b"][s0:, idx] = r["b"]
        res["S"][idx] = r["S"]
        for j, (i, _) in enumerate(snaps):
            res["snapshots"][i, idx] = r["snapshots"][j]
    return res


def run_deltalog(wl: Workload, cap: int, device, *, units: Sequence[Tuple[int, int]], scale: float = 1.0,
                 slot_idx: Optional[torch.Tensor] = None, start_delay: Optional[torch.Tensor] = None,
                 generator_device: str = "cpu", steps: Optional[int] = None, final_merge: bool = True,
                 every_step_hook=None, cycle: str = "split"):
    """Decode ``steps`` tokens with the log schedule: merge (only full logs) before every step, one
    call over the whole batch, which is the launch configuration the benchmark times.

    ``cycle="paper"`` runs the paper's own cycle instead (Algorithm 1): no token-less merge; rows
    whose log is full take the fused merge step, the others append -- two calls over phase-split
    batches (a row sits out of a call with slot index -1).

    ``start_delay``: optional int ``[batch]``; row b sits out (slot index -1) until global step
    ``start_delay[b]``, so merge boundaries are staggered across the batch by real decode steps
    rather than by fabricated log contents.  Mid-run state snapshots are then skipped.
    Returns ``(rec, state, S0, bonus)`` with everything recorded for ``units``.
    """
    import paper_2608_15533_b200 as dl

    steps = wl.steps if steps is None else steps
    src = workloads.TokenSource(wl, device=generator_device)
    S0 = src.initial_state().to(device)
    bonus = src.bonus()
    bonus = bonus.to(device) if bonus is not None else None
    desc = make_desc(wl, cap, scale)
    state = dl.State(desc, S0.clone())
    sidx = slot_idx.to(device) if slot_idx is not None else None
    rec = Recorded(units=list(units))
    ub = torch.tensor([u[0] for u in rec.units], device=device)
    uh = torch.tensor([u[1] for u in rec.units], device=device)
    uslot = sidx[ub].long() if sidx is not None else ub

    all_slots = sidx if sidx is not None else torch.arange(wl.batch, dtype=torch.int32, device=device)
    delay = start_delay.to(device) if start_delay is not None else None
    if delay is not None:
        rec.start = [int(delay[u[0]]) for u in rec.units]

    for t in range(steps):
        step_slots = sidx
        if delay is not None:
            step_slots = torch.where(delay <= t, all_slots, torch.full_like(all_slots, -1))
        if cycle == "split":
            dl.merge(desc, state, slot_idx=sidx, n=wl.batch, only_if_full=True)
        if delay is None and t > 0 and bool((state.log_len[uslot, uh] == 0).all()):
            rec.state_at.append(t)
            rec.states.append(f64(state.S_base[uslot, uh]))
        tok = {k_: (v_.to(device) if v_ is not None else None) for k_, v_ in src.token().items()}
        if cycle == "split":
            out = dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                                 u_bonus=bonus, slot_idx=step_slots)
        else:
            rows = step_slots if step_slots is not None else all_slots
            full = state.log_len[all_slots.long(), 0] == cap  # heads of a row fill in lockstep
            skip = torch.full_like(all_slots, -1)
            out = torch.zeros(wl.batch, wl.H, wl.dv, dtype=wl.io_dtype, device=device)
            for fn, sel in ((dl.decode_step, ~full), (dl.decode_merge_step, full)):
                if bool(sel.any()):
                    fn(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"], u_bonus=bonus,
                       slot_idx=torch.where(sel, rows, skip), out=out)
        rec.record_token(tok, out, wl)
        if every_step_hook is not None:
            every_step_hook(t, state, tok, out)
    if final_merge:
        dl.merge(desc, state, slot_idx=sidx, n=wl.batch, only_if_full=False)
        if not rec.state_at or rec.state_at[-1] != steps:
            rec.state_at.append(steps)
            rec.states.append(f64(state.S_base[uslot, uh]))
    torch.cuda.synchronize()
    S0_units = f64(S0[uslot, uh])
    bonus_units = f64(bonus[uh]) if bonus is not None else None
    return rec, state, S0_units, bonus_units


def materialize_units(state, wl: Workload, slots: torch.Tensor, heads: torch.Tensor) -> np.ndarray:
    """Eq. 6 in fp64 on the host from the downloaded physical state of the given (slot, head) pairs."""
    from oracle import logical

    Sb = f64(state.S_base[slots, heads])
    K = f64(state.K_log[slots, heads])
    U = f64(state.U_log[slots, heads])
    Lam = f64(state.decay_log[slots, heads])
    L = state.log_len[slots, heads].cpu().numpy()
    res = []
    for n in range(Sb.shape[0]):
        lbar = Lam[n, L[n] - 1] if L[n] > 0 else np.zeros(Lam.shape[-1])
        res.append(logical.materialize_unit(Sb[n], lbar, K[n], U[n], Lam[n], L[n]))
    return np.stack(res)
