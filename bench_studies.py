#!/usr/bin/env python
"""Kernel-level studies of the paper, repeated on this hardware (its Section 5.2: merge-interval
sweep with the U-shaped latency curve, state-size scaling, the split-preparation ablation and the
per-phase costs).  Synthetic inputs of configuration 1's shape (GDN, H = 32, d = 128, bf16 I/O).

    python bench_studies.py [--study m_sweep|state_size|phases|ablation|precision|multi_token|all] [--steps K] [--small]

Prints one JSON object per study.  ``--small`` runs every study on a few rows and points (seconds in all):
it exists so that a test can check that each study runs and what it prints.  Everything is timed with CUDA events on the launch stream after
warm-up; cycles are replayed from CUDA graphs exactly as in bench.py, whose rig this script reuses.
One GPU, no CPU path.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys

import torch

import bench
import workloads
from paper_2608_15533_b200 import traffic

CAPS = (1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64)
BATCHES = (4, 8, 16, 32, 64, 128, 256, 512)
SMALL = False   # --small: a few rows, a few points


def base_workload():
    wl = workloads.CONFIGS[1]
    return wl.scaled(batch=8, name="gdn_b8_h32_d128") if SMALL else wl


def caps():
    return (1, 3, 4, 16) if SMALL else CAPS


def batches():
    return (2, 8) if SMALL else BATCHES


def _steps_for(g_len: int, steps: int) -> int:
    return max(steps // g_len, 1) * g_len


def _split_cycle_ms(rig: bench.Rig, steps: int) -> float:
    """ms per step of the split cycle (cap appends + token-less merge), CUDA-graph replays."""
    for t in range(max(rig.cap, 3)):  # first launches of every kernel outside the capture
        rig.step(t)
    rig.reset_logs()
    n = _steps_for(bench.graph_steps(rig.cap), steps)
    region = bench.Region(rig, n, use_graph=True)
    return statistics.median(bench.timed_passes(rig, region.enqueue, region.stream, None, rig.device)) / n


def _eager_ms(rig: bench.Rig, steps: int) -> float:
    n, total = bench.time_eager_loop(rig, rig.states[0].S_base, steps)
    return total / n


def study_m_sweep(device, steps: int) -> dict:
    """Latency against the log capacity: both cycles, with the byte model beside the measurement."""
    wl = base_workload()
    u = bench.unit_shape(wl)
    eager_bytes = traffic.eager_read(u) + traffic.eager_write(u)
    rows = []
    for cap in caps():
        rig = bench.Rig(wl, cap, device)
        split_ms = _split_cycle_ms(rig, steps)
        p_steps, p_ms, fused_ms = bench.time_paper_cycle(rig, steps)
        assert all(s == 0 for s in rig.status())
        cyc, pc = traffic.cycle_bytes(u, cap), traffic.paper_cycle_bytes(u, cap + 1)
        rows.append({
            "cap": cap, "split_us_per_step": split_ms * 1e3, "paper_us_per_step": p_ms / p_steps * 1e3,
            "fused_step_us": fused_ms * 1e3,
            "split_bytes_per_unit_step": cyc["total"], "paper_bytes_per_unit_step": pc["total"],
            "split_hbm_gbs": cyc["total"] * wl.units / (split_ms * 1e-3) / 1e9,
            "paper_hbm_gbs": pc["total"] * wl.units / (p_ms / p_steps * 1e-3) / 1e9,
            "write_reduction_vs_eager": cyc["write_reduction"],
            "decode_kernel": "pipelined" if cap % 4 == 0 else "one CTA per unit",
        })
        del rig
        torch.cuda.empty_cache()
    rig = bench.Rig(wl, 16, device)
    eager_ms = _eager_ms(rig, steps)
    best = min(rows, key=lambda r: r["split_us_per_step"])
    return {"study": "m_sweep", "workload": wl.name, "eager_us_per_step": eager_ms * 1e3,
            "eager_bytes_per_unit_step": eager_bytes, "best_cap_split": best["cap"], "rows": rows}


def study_state_size(device, steps: int) -> dict:
    """Latency against the size of the base state (batch sweep at H = 32, d = 128, cap 16): where the
    state stops fitting the L2 cache the eager step pays DRAM for its write-back."""
    base = workloads.CONFIGS[1]
    u = bench.unit_shape(base)
    rows = []
    for batch in batches():
        wl = base.scaled(batch=batch, name=f"gdn_b{batch}_h32_d128")
        rig = bench.Rig(wl, 16, device)
        split_ms = _split_cycle_ms(rig, steps)
        p_steps, p_ms, _ = bench.time_paper_cycle(rig, steps)
        rig.reset_logs()
        eager_ms = _eager_ms(rig, steps)
        assert all(s == 0 for s in rig.status())
        cyc = traffic.cycle_bytes(u, 16)
        rows.append({"batch": batch, "state_mib": wl.units * u.state / 2**20,
                     "split_us_per_step": split_ms * 1e3, "paper_us_per_step": p_ms / p_steps * 1e3,
                     "eager_us_per_step": eager_ms * 1e3, "speedup_split_vs_eager": eager_ms / split_ms,
                     "split_algorithmic_gbs": cyc["total"] * wl.units / (split_ms * 1e-3) / 1e9})
        del rig
        torch.cuda.empty_cache()
    return {"study": "state_size", "cap": 16, "l2_mib": 126, "rows": rows}


def study_phases(device, steps: int) -> dict:
    """Cost of each launch of a cycle at cap 16: the decode step at every log fill (does appending
    get slower as the log grows?), the token-less merge and the fused merge step.  Plain launches with
    one event pair around each; the cost of an empty event pair is reported beside them."""
    wl, cap = base_workload(), 16
    rig = bench.Rig(wl, cap, device)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    per_fill = [[] for _ in range(cap)]
    merge_ms, fused_ms, empty_ms = [], [], []
    cycles = max(steps // cap, 8)
    rig.reset_logs()
    for c in range(cycles + 2):
        fused_cycle = c % 2 == 1
        for t in range(cap):
            a, b = ev(), ev()
            a.record(); rig.decode(t); b.record()
            per_fill[t].append((a, b))
        a, b = ev(), ev()
        a.record()
        (rig.fused(cap) if fused_cycle else rig.merge())
        b.record()
        (fused_ms if fused_cycle else merge_ms).append((a, b))
        a, b = ev(), ev()
        a.record(); b.record()
        empty_ms.append((a, b))
    torch.cuda.synchronize()
    med = lambda pairs: statistics.median(a.elapsed_time(b) for a, b in pairs[2:]) * 1e3
    u = bench.unit_shape(wl)
    return {"study": "phases", "workload": wl.name, "cap": cap, "empty_event_pair_us": med(empty_ms),
            "decode_us_by_fill": [med(p) for p in per_fill],
            "decode_bytes_by_fill": [(traffic.decode_read(u, f) + traffic.decode_write(u)) * wl.units for f in range(cap)],
            "merge_us": med(merge_ms), "fused_step_us": med(fused_ms),
            "merge_bytes": (traffic.merge_read(u, cap) + traffic.merge_write(u)) * wl.units,
            "fused_step_bytes": (traffic.fused_read(u, cap) + traffic.fused_write(u)) * wl.units}


def study_ablation(steps: int) -> dict:
    """The paper's split-preparation ablation, in this library's terms: the decode step with the
    preparation of the replay coefficients as a concurrent pipeline stage (persistent kernel) against
    the kernel in which every CTA prepares, streams and finishes its unit in sequence.  The variant is
    chosen by an environment variable that the library reads once, hence one process per variant."""
    rows = []
    for name, impl in (("pipelined (preparation as a pipeline stage)", "2"), ("one CTA per unit (sequential phases)", "1")):
        env = dict(os.environ, DELTALOG_DECODE_IMPL=impl)
        out = subprocess.run([sys.executable, str(bench.ROOT / "bench.py"), "--no-extras", "--steps", str(steps)],
                             env=env, capture_output=True, text=True, check=True).stdout.strip().splitlines()[-1]
        line = json.loads(out)
        rows.append({"variant": name, "us_per_step": line["ms_per_step"] * 1e3,
                     "decode_us": line["amortized"]["decode_ms_per_launch"] * 1e3,
                     "plain_launch_us_per_step": line["amortized"]["plain_launch_ms_per_step"] * 1e3,
                     "decode_algorithmic_frac_of_measured_peak": line["roofline"]["frac_algorithmic_incl_l2"]})
    return {"study": "ablation", "workload": workloads.CONFIGS[1].name, "cap": 16, "rows": rows}


def study_precision(device, steps: int) -> dict:
    """The value-side log of the delta rule in fp32 (default; meets the 1e-4 state bar) against the
    16-bit variant (does not: see tests/test_ulog_precision.py): what the smaller entries buy.  And the
    16-bit dense state (tests/test_gpu_bf16_base.py): half the dense bytes, for the log schedule and for
    the eager kernel, per capacity -- with a smaller base the replay of the log weighs more, so the best
    capacity moves down."""
    wl = base_workload()
    rows = []
    variants = [("fp32 state, U log fp32 (default)", False, False, 16), ("fp32 state, U log bf16", True, False, 16)]
    variants += [(f"bf16 state, U log fp32, cap {c}", False, True, c) for c in ((8,) if SMALL else (4, 8, 16, 32))]
    variants += [("bf16 state, U log bf16, cap 16", True, True, 16)]
    for name, u16, b16, cap in variants:
        rig = bench.Rig(wl, cap, device, ulog16=u16, base16=b16)
        ms = _split_cycle_ms(rig, steps)
        assert all(s == 0 for s in rig.status())
        u = bench.unit_shape(wl, ulog16=u16, base16=b16)
        cyc = traffic.cycle_bytes(u, cap)
        row = {"variant": name, "cap": cap, "state_bytes": u.state, "entry_bytes": u.entry, "us_per_step": ms * 1e3,
               "bytes_per_unit_step": cyc["total"], "hbm_gbs": cyc["total"] * wl.units / (ms * 1e-3) / 1e9,
               "write_reduction_vs_eager": cyc["write_reduction"]}
        if cap == 16 and not u16:
            rig.reset_logs()
            e_ms = _eager_ms(rig, steps)
            row["eager_us_per_step"] = e_ms * 1e3
            row["eager_hbm_gbs"] = (traffic.eager_read(u) + traffic.eager_write(u)) * wl.units / (e_ms * 1e-3) / 1e9
            row["speedup_vs_eager_kernel"] = e_ms / ms
        rows.append(row)
        del rig
        torch.cuda.empty_cache()
    return {"study": "precision", "workload": wl.name, "rows": rows}


def study_multi_token(device, steps: int) -> dict:
    """Blocks of T tokens per call (deltalog_decode_steps: one read of the base tile per block) against
    single-token steps, on configuration 1's shape at cap 16: a cycle is 16 / T block calls and the
    merge, replayed from a CUDA graph.  Per-token cost and algorithmic bytes."""
    import paper_2608_15533_b200 as dl

    wl, cap = base_workload(), 16
    rig = bench.Rig(wl, cap, device)
    u = bench.unit_shape(wl)
    rows = []
    for T in ((1, 4) if SMALL else (1, 2, 4, 8, 16)):
        blocks = [{k: (torch.stack([rig.rings[0][(i * T + t) % rig.RING][k] for t in range(T)], dim=1).contiguous()
                       if rig.rings[0][0][k] is not None else None) for k in rig.rings[0][0]}
                  for i in range(rig.RING)]
        out = torch.empty(wl.batch, T, wl.H, wl.d, dtype=wl.io_dtype, device=device)
        rig.reset_logs()

        def cycle(i0):
            for i in range(cap // T):
                tok = blocks[(i0 + i) % rig.RING]
                dl.decode_steps(rig.desc, rig.states[0], tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                                out=out)
            rig.merge()

        cycle(0)
        stream = torch.cuda.Stream(device=device)
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        n_cycles_graph = 8
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                for c in range(n_cycles_graph):
                    cycle(c)
            graph.replay()
        torch.cuda.synchronize()
        reps = max(steps // (cap * n_cycles_graph), 1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            a.record()
            for _ in range(reps):
                graph.replay()
            b.record()
        torch.cuda.synchronize()
        assert all(s == 0 for s in rig.status())
        us_per_token = a.elapsed_time(b) * 1e3 / (reps * n_cycles_graph * cap)
        # bytes per unit and token: one base read per block, the live log once per block, token I/O and appends per token
        blocks_per_cycle = cap // T
        rd = sum(u.state + (i * T) * u.entry + traffic.LEN_WORD for i in range(blocks_per_cycle)) + cap * u.token_in
        wr = cap * (u.entry + u.token_out) + blocks_per_cycle * traffic.LEN_WORD
        total = rd + wr + traffic.merge_read(u, cap) + traffic.merge_write(u)
        rows.append({"T": T, "us_per_token": us_per_token, "bytes_per_unit_token": total / cap,
                     "hbm_gbs": total / cap * wl.units / (us_per_token * 1e-6) / 1e9,
                     "kernel": "one CTA per unit, tile in registers"})
    return {"study": "multi_token", "workload": wl.name, "cap": cap,
            "note": "T = 1 through deltalog_decode_steps uses the one-CTA-per-unit kernel; the single-token entry point "
                    "(persistent kernel) runs the same cycle at the figure bench.py reports", "rows": rows}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--study", default="all", choices=["m_sweep", "state_size", "phases", "ablation", "precision", "multi_token", "all"])
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--small", action="store_true", help="a few rows and a few points per study (a smoke run)")
    args = ap.parse_args()
    global SMALL
    SMALL = args.small
    assert torch.cuda.is_available(), "the studies need a CUDA device (there is no CPU path)"
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    todo = ["m_sweep", "state_size", "phases", "ablation", "precision", "multi_token"] if args.study == "all" else [args.study]
    for name in todo:
        if name == "m_sweep":
            res = study_m_sweep(device, args.steps)
        elif name == "state_size":
            res = study_state_size(device, args.steps)
        elif name == "phases":
            res = study_phases(device, args.steps)
        elif name == "precision":
            res = study_precision(device, args.steps)
        elif name == "multi_token":
            res = study_multi_token(device, args.steps)
        else:
            res = study_ablation(args.steps)
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
