"""TEST INFRASTRUCTURE -- the parity oracle (CPU, fp64). Not part of the product path.

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` / ``--impl reference``
legs of ``bench.py`` may import this package.  It shares no code with the CUDA library and
imports nothing from it.

Contents
--------
``eager_rollout``      the eager dense recurrence of GDN / KDA / RWKV6 and of the additive family
                       (linear attention, RetNet, GLA) (Eq. 3, Table 1), compiled
                       from ``eager_oracle.c`` (plain C, fp64, OpenMP over independent units).
``logical``            the base-plus-log schedule of Algorithm 1 / Eq. 4-6 in fp64 numpy, used to
                       check the physical state (base, log, snapshots) that the GPU leaves behind.

Pins: ``tests/test_oracle_pins.py`` checks both against closed forms and invariants that do not
call into this package's arithmetic.  Nothing here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

from . import logical  # noqa: F401  (re-export)

GDN, KDA, RWKV6, LINATTN, RETNET, GLA = 0, 1, 2, 3, 4, 5
OP_BY_NAME = {"gdn": GDN, "kda": KDA, "rwkv6": RWKV6, "linattn": LINATTN, "retnet": RETNET, "gla": GLA}

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "eager_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile ``eager_oracle.c`` with gcc (fp64, no fast-math) into ``liboracle.so``."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99", str(_SRC), "-o", str(tmp), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        lib.oracle_eager_rollout.restype = ctypes.c_int
        lib.oracle_eager_rollout.argtypes = [
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
            dp, dp, dp, dp, dp, dp, dp, dp, dp, ctypes.c_int, ip, dp, ctypes.c_int,
        ]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Host threads the C oracle uses (OpenMP default)."""
    return int(_load().oracle_num_threads())


def _f64(a, shape):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if a.shape != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {a.shape}")
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


def eager_rollout(op, S0, q, k, v, lam, beta=None, bonus=None, scale=1.0, snapshot_at=(), state_bf16=False):
    """Eager fp64 recurrence over ``T`` tokens for ``N`` independent (sequence, head) units.

    Shapes: ``S0 [N,d_k,d_v]``, ``q,k [T,N,d_k]``, ``v [T,N,d_v]``, ``lam [T,N,d_lambda]`` (log-decay;
    ``d_lambda`` = 1 for GDN / RetNet, ``d_k`` for KDA / RWKV6 / GLA; ignored for plain linear
    attention), ``beta [T,N]`` (GDN / KDA), ``bonus [N,d_k]`` (RWKV6).  ``snapshot_at``: ascending 1-based token counts.
    ``state_bf16``: the state is kept in bfloat16 between tokens (rounded after every token; the
    16-bit-state variant of Section 2.2's roofline remark) -- ``S0`` should then be representable.

    Returns ``dict(out [T,N,d_v], b [T,N,d_v], S [N,d_k,d_v], snapshots [n,N,d_k,d_v])``;
    ``b`` is the value-side factor of every token (what the log's U entries must hold).
    """
    if isinstance(op, str):
        op = OP_BY_NAME[op.lower()]
    S0 = np.asarray(S0, dtype=np.float64)
    N, d_k, d_v = S0.shape
    T = int(np.asarray(q).shape[0])
    d_lambda = 1 if op in (GDN, RETNET, LINATTN) else d_k
    if op == LINATTN:
        lam = np.zeros((T, N, 1))  # no decay: the C side does not read it
    S = np.array(S0, dtype=np.float64, order="C", copy=True)
    q = _f64(q, (T, N, d_k))
    k = _f64(k, (T, N, d_k))
    v = _f64(v, (T, N, d_v))
    lam = _f64(np.asarray(lam, dtype=np.float64).reshape(T, N, d_lambda), (T, N, d_lambda))
    if op == RWKV6:
        if bonus is None:
            raise ValueError("RWKV6 needs the bonus vector")
        bonus = _f64(bonus, (N, d_k))
        beta = None
    elif op in (LINATTN, RETNET, GLA):
        beta = bonus = None
    else:
        if beta is None:
            raise ValueError("GDN / KDA need beta")
        beta = _f64(np.asarray(beta, dtype=np.float64).reshape(T, N), (T, N))
        bonus = None
    out = np.empty((T, N, d_v), dtype=np.float64)
    b = np.empty((T, N, d_v), dtype=np.float64)
    snaps = np.ascontiguousarray(np.asarray(list(snapshot_at), dtype=np.int32))
    if snaps.size and (np.any(np.diff(snaps) <= 0) or snaps[0] < 1 or snaps[-1] > T):
        raise ValueError("snapshot_at must be strictly ascending within 1..T")
    S_snap = np.empty((snaps.size, N, d_k, d_v), dtype=np.float64)
    rc = _load().oracle_eager_rollout(
        int(op), T, N, d_k, d_v, float(scale), _ptr(S), _ptr(q), _ptr(k), _ptr(v), _ptr(lam),
        _ptr(beta), _ptr(bonus), _ptr(out), _ptr(b), int(snaps.size),
        snaps.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), _ptr(S_snap), int(bool(state_bf16)),
    )
    if rc != 0:
        raise ValueError(f"oracle_eager_rollout rejected op={op}")
    return {"out": out, "b": b, "S": S, "snapshots": S_snap}
