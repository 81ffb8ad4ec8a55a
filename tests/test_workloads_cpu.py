"""The seeded input recipe: shapes, dtypes, value ranges, determinism."""
import torch

import workloads
from workloads import CONFIGS, GDN, KDA, RWKV6


def test_benchmark_configs_have_the_stated_shapes():
    c = CONFIGS
    assert (c[0].op, c[0].batch, c[0].H, c[0].d, c[0].steps, c[0].caps, c[0].io_dtype) == \
        (GDN, 1, 2, 64, 64, (8,), torch.float32)
    assert (c[1].op, c[1].batch, c[1].H, c[1].d, c[1].steps, c[1].caps) == (GDN, 128, 32, 128, 256, (4, 8, 16, 32))
    assert (c[2].op, c[2].batch, c[2].H, c[2].d, c[2].steps, c[2].caps) == (KDA, 256, 32, 128, 256, (16,))
    assert (c[3].op, c[3].batch, c[3].H, c[3].d, c[3].steps, c[3].caps) == (RWKV6, 256, 64, 64, 256, (16,))
    assert (c[4].op, c[4].batch, c[4].H, c[4].d, c[4].steps, c[4].layers, c[4].staggered) == \
        (GDN, 512, 32, 128, 128, 24, True)
    assert c[1].units * c[1].d * c[1].d * 4 == 256 * 2 ** 20      # 256 MiB of base state


def _tiny(op):
    return workloads.Workload("t", op, 5, 3, 64, 4, (4,))


def test_recipe_ranges_and_dtypes():
    for op in (GDN, KDA, RWKV6):
        wl = _tiny(op)
        src = workloads.TokenSource(wl)
        S0 = src.initial_state()
        assert S0.shape == (5, 3, 64, 64) and S0.dtype == torch.float32 and 0.08 < S0.std() < 0.12
        bonus = src.bonus()
        tok = src.token()
        assert tok["q"].dtype == torch.bfloat16 and tok["q"].shape == (5, 3, 64)
        assert tok["g"].dtype == torch.float32 and bool((tok["g"] < 0).all())
        if op == RWKV6:
            assert bonus.shape == (3, 64) and tok["beta"] is None and tok["g"].shape == (5, 3, 64)
            assert 0.5 < tok["k"].float().std() < 1.5               # not normalised
        else:
            assert bonus is None
            assert tok["g"].shape == ((5, 3) if op == GDN else (5, 3, 64))
            assert bool(((tok["beta"] > 0) & (tok["beta"] < 1)).all())
            norms = tok["k"].float().norm(dim=-1)
            assert bool(((norms - 1).abs() < 1e-2).all())           # unit norm up to bf16 rounding


def test_same_seed_same_bytes_and_different_seed_differs():
    wl = _tiny(KDA)
    a, b, c = workloads.TokenSource(wl), workloads.TokenSource(wl), workloads.TokenSource(wl, seed=1)
    assert torch.equal(a.initial_state(), b.initial_state())
    ta, tb = a.token(), b.token()
    assert all(torch.equal(ta[k], tb[k]) for k in ta)
    c.initial_state()
    assert not torch.equal(ta["q"], c.token()["q"])


def test_slot_permutation_and_fill_offsets():
    wl = workloads.Workload("t", GDN, 8, 2, 64, 4, (4,), num_slots=20)
    idx = workloads.slot_permutation(wl, pad_every=4)
    live = idx[idx >= 0]
    assert idx.dtype == torch.int32 and idx.shape == (8,) and idx[0] == -1 and idx[4] == -1
    assert len(set(live.tolist())) == live.numel() and int(live.max()) < 20
    f = workloads.fill_offsets(CONFIGS[4], 16)
    assert f.shape == (512,) and int(f.min()) == 0 and int(f.max()) == 15
