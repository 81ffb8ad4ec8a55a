"""Seeded synthetic inputs for the recurrent-state decode workloads.

This module holds the input recipe only -- shapes, distributions, rounding to the I/O dtype -- and
none of the method's arithmetic.  It is the one piece shared by the CUDA path's callers and the
oracle's callers: both receive the very same tensors (the oracle widened to fp64).

Recipe (one ``torch.Generator`` seeded with ``seed``; draws in fp32, in this fixed order):
``S0``; RWKV6 only: ``bonus``; then for every token ``q, k, v, gate noise, beta noise``.

* ``S0 ~ N(0, 0.1^2)`` fp32.
* GDN / KDA: ``q, k ~ N(0,1)`` then L2-normalised in fp32 (``x / max(||x||, 1e-12)``) and only then
  rounded to the I/O dtype; ``v ~ N(0,1)``; log-decay ``g = -softplus(N(0,1))`` so that
  ``alpha = exp(g)`` lies in (0,1) -- one value per head for GDN, one per key channel for KDA;
  ``beta = sigmoid(N(0,1))``.
* RWKV6: ``r, k, v ~ N(0,1)`` (no normalisation); ``g = log w = -exp(N(-0.5, 0.5^2))`` per channel;
  ``bonus[H, d_k] ~ N(0, 0.1^2)`` fixed over time.

The second argument of every N(., .) above is a standard deviation.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Iterator, Optional, Tuple

import torch

GDN, KDA, RWKV6, LINATTN, RETNET, GLA = 0, 1, 2, 3, 4, 5
OP_NAMES = {GDN: "gdn", KDA: "kda", RWKV6: "rwkv6", LINATTN: "linattn", RETNET: "retnet", GLA: "gla"}


@dataclass(frozen=True)
class Workload:
    """Shape of one decode workload (one recurrent layer unless ``layers`` > 1)."""

    name: str
    op: int
    batch: int            # sequences decoded per step
    H: int
    d: int                # key dimension d_k (and d_v unless ``d_v`` is given)
    steps: int
    caps: Tuple[int, ...]  # log capacities exercised
    io_dtype: torch.dtype = torch.bfloat16
    layers: int = 1
    num_slots: Optional[int] = None   # state-pool size (>= batch); None -> batch
    staggered: bool = False           # random initial log fill per sequence
    seed: int = 0
    d_v: Optional[int] = None         # value dimension when it differs from the key dimension

    @property
    def dv(self) -> int:
        return self.d if self.d_v is None else self.d_v

    @property
    def slots(self) -> int:
        return self.num_slots if self.num_slots is not None else self.batch

    @property
    def d_lambda(self) -> int:
        return self.d if self.op in (KDA, RWKV6, GLA) else 1

    @property
    def units(self) -> int:
        """(sequence, head) pairs updated per step and layer."""
        return self.batch * self.H

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (index = position in the benchmark description).
CONFIGS: Dict[int, Workload] = {
    0: Workload("gdn_b1_h2_d64_fp32", GDN, 1, 2, 64, 64, (8,), io_dtype=torch.float32),
    1: Workload("gdn_b128_h32_d128", GDN, 128, 32, 128, 256, (4, 8, 16, 32)),
    2: Workload("kda_b256_h32_d128", KDA, 256, 32, 128, 256, (16,)),
    3: Workload("rwkv6_b256_h64_d64", RWKV6, 256, 64, 64, 256, (16,)),
    4: Workload("gdn_serving_24l_b512_h32_d128", GDN, 512, 32, 128, 128, (16,), layers=24,
                staggered=True),
}


def _l2_normalise(x: torch.Tensor) -> torch.Tensor:
    return x / x.norm(dim=-1, keepdim=True).clamp_min(1e-12)


class TokenSource:
    """Draws the initial state and then one token batch after another from a single seeded generator.

    All tensors are created on ``device`` (``"cpu"`` generators are machine-independent; a CUDA
    generator is used only where the tensors are too large to draw on the host).
    """

    def __init__(self, wl: Workload, device: str = "cpu", seed: Optional[int] = None):
        self.wl = wl
        self.device = torch.device(device)
        self.gen = torch.Generator(device=self.device)
        self.gen.manual_seed(wl.seed if seed is None else seed)
        self._drew_state = False

    def _randn(self, *shape) -> torch.Tensor:
        return torch.randn(*shape, generator=self.gen, device=self.device, dtype=torch.float32)

    def initial_state(self) -> torch.Tensor:
        """``S0 [slots, H, d, d]`` fp32 ~ N(0, 0.1^2).  Must be drawn first."""
        assert not self._drew_state, "initial_state() is the first draw"
        self._drew_state = True
        wl = self.wl
        return self._randn(wl.slots, wl.H, wl.d, wl.dv).mul_(0.1)

    def bonus(self) -> Optional[torch.Tensor]:
        """RWKV6 bonus ``[H, d] ~ N(0, 0.1^2)`` fp32 (drawn right after the state); None otherwise."""
        if self.wl.op != RWKV6:
            return None
        return self._randn(self.wl.H, self.wl.d).mul_(0.1)

    def token(self) -> Dict[str, Optional[torch.Tensor]]:
        """One token batch: ``q, k, v [B,H,d]`` in the I/O dtype, ``g`` fp32 log-decay, ``beta`` fp32."""
        wl = self.wl
        B, H, d = wl.batch, wl.H, wl.d
        q, k, v = self._randn(B, H, d), self._randn(B, H, d), self._randn(B, H, wl.dv)
        if wl.op == RWKV6:
            g = -torch.exp(self._randn(B, H, d).mul_(0.5).sub_(0.5))
            _ = self._randn(B, H)  # keeps the draw order uniform across operators
            beta = None
        elif wl.op in (LINATTN, RETNET, GLA):
            # additive family: L2-normalised q, k (for plain linear attention after the positive feature
            # map elu(x) + 1, which the caller of the library applies); RetNet's decay is the fixed
            # per-head gamma_h = 1 - 2^(-5-h mod 8); GLA's gate is drawn like KDA's; no beta
            if wl.op == LINATTN:
                q, k = torch.nn.functional.elu(q) + 1.0, torch.nn.functional.elu(k) + 1.0
            q, k = _l2_normalise(q), _l2_normalise(k)
            noise = self._randn(B, H, d)   # drawn for every operator of the family: uniform draw order
            if wl.op == GLA:
                g = -torch.nn.functional.softplus(noise)
            elif wl.op == RETNET:
                h = torch.arange(H, device=self.device, dtype=torch.float32) % 8
                g = torch.log1p(-torch.pow(2.0, -5.0 - h)).expand(B, H)
            else:
                g = None
            _ = self._randn(B, H)
            beta = None
        else:
            q, k = _l2_normalise(q), _l2_normalise(k)
            gate_shape = (B, H) if wl.op == GDN else (B, H, d)
            g = -torch.nn.functional.softplus(self._randn(*gate_shape))
            beta = torch.sigmoid(self._randn(B, H))
        dt = wl.io_dtype
        return {"q": q.to(dt), "k": k.to(dt), "v": v.to(dt), "g": g.contiguous() if g is not None else None,
                "beta": beta}

    def tokens(self, n: int) -> Iterator[Dict[str, Optional[torch.Tensor]]]:
        for _ in range(n):
            yield self.token()


def slot_permutation(wl: Workload, seed: Optional[int] = None, pad_every: int = 0) -> torch.Tensor:
    """int32 ``[batch]`` row -> slot map: a seeded random choice of distinct slots from the pool.

    ``pad_every`` > 0 marks every ``pad_every``-th row as padding (slot -1).
    """
    g = torch.Generator().manual_seed((wl.seed if seed is None else seed) + 7919)
    idx = torch.randperm(wl.slots, generator=g)[: wl.batch].to(torch.int32)
    if pad_every > 0:
        idx[::pad_every] = -1
    return idx


def fill_offsets(wl: Workload, cap: int, seed: Optional[int] = None) -> torch.Tensor:
    """int64 ``[batch]`` initial log fill per sequence, uniform on {0..cap-1} (staggered merges)."""
    g = torch.Generator().manual_seed((wl.seed if seed is None else seed) + 104729)
    return torch.randint(0, cap, (wl.batch,), generator=g)
