"""More compact log-decay snapshots for the per-key operators (the snapshot Lambda is half of an
RWKV6 log entry at head size 64 and 40 % of a KDA entry): an error study on the oracle alone.

The replay weight of entry i is exp(lbar - Lambda[i]); a snapshot stored with absolute error eps turns
into a relative error eps of that weight, and hence of the entry's whole contribution to the state.
The accumulated log-decay reaches 10 .. 20 within a capacity-16 cycle of the benchmark recipes, so a
16-bit snapshot (bfloat16: eps ~ 3e-2, float16: eps ~ 4e-3 at that magnitude) misses the 1e-4 state
bar by one to two orders of magnitude, and even a 24-bit float (fp32 with its low mantissa byte
dropped) only just reaches it (1e-4) while saving no more than one byte in four of the snapshot,
12.5 % of an RWKV6 entry.  This is why the library stores the snapshots in fp32, as the paper does;
the test pins the numbers behind that decision.  (The running log-decay itself stays exact in every variant; only the stored snapshots are
rounded.)"""
import numpy as np
import pytest
import torch

import oracle
import workloads
from harness import f64, rel_err
from oracle import logical
from workloads import KDA, RWKV6, Workload


def to_bf16(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float64)).to(torch.bfloat16).to(torch.float64).numpy()


def to_f16(x):
    return np.asarray(x, dtype=np.float16).astype(np.float64)


def to_f24(x):
    """fp32 with the low 8 mantissa bits dropped (round to nearest even on the kept 15 bits)."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32)).view(np.uint32).astype(np.uint64)
    u = (u + 0x7F + ((u >> 8) & 1)) & 0xFFFFFF00
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


@pytest.mark.parametrize("op", [KDA, RWKV6])
def test_snapshot_precision_study_on_the_oracle(op):
    wl = Workload("lam_cpu", op, 1, 2, 32, 64, (16,))
    cap, steps = 16, 64
    src = workloads.TokenSource(wl, device="cpu")
    S0 = f64(src.initial_state()).reshape(-1, wl.d, wl.d)
    bonus = src.bonus()
    N = wl.batch * wl.H
    bon = np.tile(f64(bonus), (wl.batch, 1)) if bonus is not None else None
    toks = []
    for _ in range(steps):
        tok = src.token()
        toks.append({k: (f64(v).reshape(N, -1) if v is not None else None) for k, v in tok.items()})
    stack = lambda name: np.stack([t[name] for t in toks])
    ref = oracle.eager_rollout(op, S0, stack("q"), stack("k"), stack("v"), stack("g"),
                               beta=stack("beta")[..., 0] if toks[0]["beta"] is not None else None, bonus=bon)
    errs, largest = {}, 0.0
    for name, rounding in (("fp32", lambda x: np.asarray(x, dtype=np.float32).astype(np.float64)), ("f24", to_f24),
                           ("f16", to_f16), ("bf16", to_bf16)):
        st = logical.LogState(op, S0, cap, store_lam=rounding)
        worst = 0.0
        for t, tok in enumerate(toks):
            if (st.length == cap).all():
                logical.merge(st)
            logical.decode_step(st, tok["q"], tok["k"], tok["v"], tok["g"],
                                beta=tok["beta"][:, 0] if tok["beta"] is not None else None, bonus=bon)
            largest = max(largest, float(np.abs(st.lbar).max()))
            if (st.length == cap).all():   # right before a merge: every snapshot of the cycle is in use
                r = oracle.eager_rollout(op, S0, stack("q")[:t + 1], stack("k")[:t + 1], stack("v")[:t + 1], stack("g")[:t + 1],
                                         beta=stack("beta")[:t + 1, :, 0] if tok["beta"] is not None else None, bonus=bon)
                worst = max(worst, rel_err(logical.materialize(st), r["S"]))
        errs[name] = worst
    print(f"op {op}: largest accumulated |log-decay| {largest:.1f}; state error by snapshot format: "
          + ", ".join(f"{k} {v:.1e}" for k, v in errs.items()))
    assert largest > 8.0                      # the snapshots do reach the magnitudes the argument is about
    assert errs["fp32"] < 2e-6                # what the library stores
    assert 2e-5 < errs["f24"] < 5e-4          # right at the bar, for one byte in four of the snapshot
    assert errs["f16"] > 1e-4 and errs["bf16"] > 1e-3   # 16-bit snapshots break the 1e-4 state bar
