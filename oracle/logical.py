"""TEST INFRASTRUCTURE -- the base-plus-log schedule in fp64 numpy. Not part of the product path.

The physical state of the deferred representation (Section 3.1): a dense base ``S_base``, a
cumulative log-decay ``lbar`` since the last materialisation, a bounded log of compact factors
``K_log[i] = a``, ``U_log[i] = b``, one log-decay snapshot ``Lam_log[i]`` per entry, and the live
length ``length``.  The functions below follow Algorithm 1 with the cycle split the way this
library splits it: the decode step always appends (Eq. 4), and materialisation (Eq. 5 without the
current-token term) is a separate, token-less merge.

Everything is written for clarity, not speed: every readout first materialises the logical state
with Eq. 6 as a dense matrix and then applies the operator's definition to it.  Python loops run
over units; use small N, T.

Pins (tests/test_oracle_pins.py): after every append and every merge the state materialised by
Eq. 6 equals the eager recurrence of ``eager_oracle.c`` to ~1e-13, for every capacity, which is
the closure property the paper proves below Eq. 6; the eager recurrence itself is pinned against
closed forms there.
"""
from __future__ import annotations

import numpy as np

GDN, KDA, RWKV6, LINATTN, RETNET, GLA = 0, 1, 2, 3, 4, 5


def round_bf16(x) -> np.ndarray:
    """The value a bfloat16 storage element holds after a store of ``x``: fp64 -> fp32 -> bfloat16,
    both round-to-nearest-even, returned as fp64 (finite inputs).  Pass it as ``store_base`` for the
    16-bit base state (the 16-bit-state variant of Section 2.2's roofline remark) or as ``store_u``."""
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(np.shape(x))
ADDITIVE = (LINATTN, RETNET, GLA)  # b = v, readout from the updated state; LINATTN: lambda == 0


class LogState:
    """Base + bounded log for ``N`` independent (sequence, head) units (Section 3.1)."""

    def __init__(self, op: int, S0: np.ndarray, cap: int, store_u=None, store_base=None, store_lam=None):
        """``store_u``: optional function applied to a value-side factor when it is written into the
        log (e.g. rounding to a 16-bit format), for studies of reduced-precision logs; None = exact.
        ``store_base``: the same for every write of the dense base (the initial state, Eq. 5) -- the
        base is then only re-rounded once per materialisation, not once per token.
        ``store_lam``: the same for every log-decay snapshot written into the log (the running
        cumulative log-decay ``lbar`` itself stays exact), for studies of more compact snapshots."""
        S0 = np.asarray(S0, dtype=np.float64)
        self.store_u = store_u
        self.store_base = store_base
        self.store_lam = store_lam
        self.op = int(op)
        self.N, self.d_k, self.d_v = S0.shape
        self.cap = int(cap)
        self.d_lambda = 1 if self.op in (GDN, RETNET, LINATTN) else self.d_k
        self.S_base = S0.copy() if store_base is None else np.asarray(store_base(S0), dtype=np.float64).copy()
        self.lbar = np.zeros((self.N, self.d_lambda))
        self.K_log = np.zeros((self.N, self.cap, self.d_k))
        self.U_log = np.zeros((self.N, self.cap, self.d_v))
        self.Lam_log = np.zeros((self.N, self.cap, self.d_lambda))
        self.length = np.zeros(self.N, dtype=np.int64)


def _row_scale(ell: np.ndarray, d_k: int) -> np.ndarray:
    """exp(ell) as a length-d_k vector (a scalar decay is shared by all key coordinates)."""
    ell = np.asarray(ell, dtype=np.float64).reshape(-1)
    return np.exp(np.broadcast_to(ell, (d_k,)) if ell.size == 1 else ell)


def materialize_unit(S_base, lbar, K_log, U_log, Lam_log, length) -> np.ndarray:
    """Eq. 6 for one unit: S = D(lbar) S_base + sum_{i<length} D(lbar - Lam[i]) K[i] U[i]^T."""
    d_k = S_base.shape[0]
    S = _row_scale(lbar, d_k)[:, None] * S_base
    for i in range(int(length)):
        w = _row_scale(np.asarray(lbar) - np.asarray(Lam_log[i]), d_k)
        S = S + np.outer(w * K_log[i], U_log[i])
    return S


def materialize(st: LogState) -> np.ndarray:
    """Eq. 6 for every unit -> [N, d_k, d_v]."""
    return np.stack([
        materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], st.length[n])
        for n in range(st.N)
    ])


def _lam(st: LogState, lam) -> np.ndarray:
    """The token's log-decay as [N, d_lambda]; plain linear attention has none (zeros)."""
    if st.op == LINATTN:
        return np.zeros((st.N, st.d_lambda))
    return np.asarray(lam, dtype=np.float64).reshape(st.N, st.d_lambda)


def decode_step(st: LogState, q, k, v, lam, beta=None, bonus=None, scale: float = 1.0) -> np.ndarray:
    """One token through Algorithm 1's append branch for every unit; returns ``out [N, d_v]``.

    ``q,k [N,d_k]``, ``v [N,d_v]``, ``lam [N,d_lambda]``, ``beta [N]`` (GDN/KDA), ``bonus [N,d_k]`` (RWKV6).
    Raises if a unit's log is already full (the caller merges first).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    lam = _lam(st, lam)
    out = np.empty((st.N, st.d_v))
    for n in range(st.N):
        L = int(st.length[n])
        if L >= st.cap:
            raise RuntimeError(f"unit {n}: log full (length {L} == capacity); merge first")
        # line 1: readouts defined on the pre-update logical state
        S_prev = materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], L)
        # line 2: fold the token's log-decay into the cumulative log-decay
        st.lbar[n] = st.lbar[n] + lam[n]
        S_decayed = _row_scale(lam[n], st.d_k)[:, None] * S_prev
        # line 3: update factors (a, b) and the output of the original recurrence
        a = k[n]
        if st.op == RWKV6:
            b = v[n]
            out[n] = S_prev.T @ q[n] + float(np.sum(q[n] * bonus[n] * k[n])) * v[n]
        elif st.op in ADDITIVE:
            b = v[n]
        else:
            b = float(beta[n]) * (v[n] - S_decayed.T @ k[n])
        # lines 4-5 / Eq. 4: append (a, b, lbar) into slot L; the base is untouched
        st.K_log[n, L] = a
        st.U_log[n, L] = b if st.store_u is None else st.store_u(b)
        st.Lam_log[n, L] = st.lbar[n] if st.store_lam is None else st.store_lam(st.lbar[n])
        st.length[n] = L + 1
        if st.op != RWKV6:
            S_new = materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], L + 1)
            out[n] = scale * (S_new.T @ q[n])
    return out


def decode_merge_step(st: LogState, q, k, v, lam, beta=None, bonus=None, scale: float = 1.0) -> np.ndarray:
    """One token through Algorithm 1's else-branch for every unit (whatever its live length):
    readouts from the pre-update logical state, ``lbar += lambda_t``, factors (a, b), then Eq. 5 --
    the represented state *plus the current update* is written into the base -- and the log is
    cleared (``lbar = 0``, ``length = 0``).  Returns ``out [N, d_v]``."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    lam = _lam(st, lam)
    out = np.empty((st.N, st.d_v))
    for n in range(st.N):
        L = int(st.length[n])
        # line 1: readouts defined on the pre-update logical state
        S_prev = materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], L)
        # line 2
        st.lbar[n] = st.lbar[n] + lam[n]
        S_decayed = _row_scale(lam[n], st.d_k)[:, None] * S_prev
        # line 3
        a = k[n]
        if st.op == RWKV6:
            b = v[n]
            out[n] = S_prev.T @ q[n] + float(np.sum(q[n] * bonus[n] * k[n])) * v[n]
        elif st.op in ADDITIVE:
            b = v[n]
        else:
            b = float(beta[n]) * (v[n] - S_decayed.T @ k[n])
        # lines 7-8 / Eq. 5: D(lbar) S_base + sum_i D(lbar - Lam[i]) K[i] U[i]^T + a b^T, then reset
        S_new = materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], L) + np.outer(a, b)
        if st.op != RWKV6:
            out[n] = scale * (S_new.T @ q[n])
        st.S_base[n] = S_new if st.store_base is None else st.store_base(S_new)
        st.lbar[n] = 0.0
        st.length[n] = 0
    return out


def merge(st: LogState, only_if_full: bool = False) -> None:
    """Eq. 5 without the current-token term: fold the log into the base, reset lbar and length."""
    for n in range(st.N):
        L = int(st.length[n])
        if L == 0 or (only_if_full and L < st.cap):
            continue
        S_new = materialize_unit(st.S_base[n], st.lbar[n], st.K_log[n], st.U_log[n], st.Lam_log[n], L)
        st.S_base[n] = S_new if st.store_base is None else st.store_base(S_new)
        st.lbar[n] = 0.0
        st.length[n] = 0
