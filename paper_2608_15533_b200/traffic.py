"""Algorithmic bytes of the decode path: what the method itself must move through HBM.

Per (sequence, head) unit, following the paper's traffic model (Eq. 7-9) adapted to this
library's cycle: ``cap`` decode+append steps at log fill 0..cap-1, then one token-less merge of
``cap`` entries.  Differences from Eq. 9: the cumulative log-decay is not a separate buffer here
(it is the newest snapshot in the log, already counted in the replay read), so the ``2 C_decay``
term is absent; token I/O and the 4-byte length word are counted.

All functions are plain host arithmetic used by the benchmark's roofline lines and checked in the
CPU tests against the figures the paper prints for its own profile.
"""
from __future__ import annotations

from dataclasses import dataclass

GDN, KDA, RWKV6 = 0, 1, 2


@dataclass(frozen=True)
class UnitShape:
    op: int
    d_k: int
    d_v: int
    io_bytes: int = 2      # q, k, v, out element size
    klog_bytes: int = 2
    ulog_bytes: int = 4
    state_bytes: int = 4   # p_S

    @property
    def d_lambda(self) -> int:
        return 1 if self.op == GDN else self.d_k

    @property
    def state(self) -> int:
        """C_state per unit: p_S d_k d_v."""
        return self.state_bytes * self.d_k * self.d_v

    @property
    def entry(self) -> int:
        """C_entry per unit: p_K d_k + p_U d_v + 4 d_lambda."""
        return self.klog_bytes * self.d_k + self.ulog_bytes * self.d_v + 4 * self.d_lambda

    @property
    def token_in(self) -> int:
        """q, k, v, the log-decay gate, and beta (delta rule) -- T_common's input half."""
        gate = 4 * self.d_lambda
        beta = 0 if self.op == RWKV6 else 4
        return self.io_bytes * (2 * self.d_k + self.d_v) + gate + beta

    @property
    def token_out(self) -> int:
        return self.io_bytes * self.d_v


LEN_WORD = 4  # the live-length word is read and written by every decode step


def decode_read(u: UnitShape, fill: int) -> int:
    """Bytes one decode step reads with ``fill`` live entries: base + live log + token + length."""
    return u.state + fill * u.entry + u.token_in + LEN_WORD


def decode_write(u: UnitShape) -> int:
    """Bytes one decode step writes: the appended entry, the output, the length."""
    return u.entry + u.token_out + LEN_WORD


def merge_read(u: UnitShape, fill: int) -> int:
    return u.state + fill * u.entry + LEN_WORD


def merge_write(u: UnitShape) -> int:
    return u.state + LEN_WORD


def fused_read(u: UnitShape, fill: int) -> int:
    """Bytes the fused merge step reads with ``fill`` live entries: base + live log + token + length."""
    return u.state + fill * u.entry + u.token_in + LEN_WORD


def fused_write(u: UnitShape) -> int:
    """Bytes the fused merge step writes: the base, the output, the length."""
    return u.state + u.token_out + LEN_WORD


def eager_read(u: UnitShape) -> int:
    return u.state + u.token_in


def eager_write(u: UnitShape) -> int:
    return u.state + u.token_out


def cycle_bytes(u: UnitShape, cap: int) -> dict:
    """Amortised per-step bytes of a full cycle (cap decode steps + one merge), per unit."""
    rd = sum(decode_read(u, f) for f in range(cap)) + merge_read(u, cap)
    wr = cap * decode_write(u) + merge_write(u)
    eager = eager_read(u) + eager_write(u)
    return {
        "read": rd / cap,
        "write": wr / cap,
        "total": (rd + wr) / cap,
        "eager_total": eager,
        "eager_write": eager_write(u),
        "write_reduction": eager_write(u) / (wr / cap),
        "total_reduction": eager / ((rd + wr) / cap),
    }


def paper_cycle_bytes(u: UnitShape, M: int) -> dict:
    """The paper's own cycle for comparison with its printed profile: M-1 appends at fill
    0..M-2, then a fused merge step that also consumes a token (reads base + M-1 entries + token,
    writes the base + output).  State-related traffic only plus token I/O, no length words."""
    C = M - 1
    rd = sum(u.state + f * u.entry + u.token_in for f in range(C)) + u.state + C * u.entry + u.token_in
    wr = C * (u.entry + u.token_out) + u.state + u.token_out
    eager = eager_read(u) + eager_write(u)
    return {"read": rd / M, "write": wr / M, "total": (rd + wr) / M,
            "write_reduction": eager_write(u) / (wr / M), "total_reduction": eager / ((rd + wr) / M)}
