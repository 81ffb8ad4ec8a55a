#!/usr/bin/env python
"""Benchmark of the DeltaLog decode hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..4] [--cap C] [--impl ours|reference]

One "step" is one decode token for the whole batch of the workload: the decode+append kernel, and
the merge kernel whenever the logs are full (every ``cap`` steps), i.e. the complete hot path.
Rank 0 prints ONE JSON line.  ``value`` is (sequence*head) state updates per second with all inputs
resident in HBM; ``e2e`` is the same metric through ``deltalog_decode_step_host`` with the token
tensors in pinned host memory and the output read back to the host every step.

With N > 1 (one process per GPU, launched by ``torch.distributed.run``) every rank decodes its own
shard of batch rows -- the path has no exchange step -- and the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import torch  # noqa: E402

import workloads  # noqa: E402
from paper_2608_15533_b200 import launch, traffic  # noqa: E402

METRIC = "state-update (seq*head)-steps/s"
UNIT = "(seq*head)-steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the decode kernel, from the ncu
# captures summarised under profiles/ (bytes per (sequence, head) unit; None = not captured).
# Captured with `--cache-control none` and only these two counters (one pass, so ncu neither flushes L2
# nor saves and restores memory around the launch): L2 is as the previous launch left it, which is the
# condition of the timed loop -- part of the live log and of the base tiles is then served by L2.  With
# ncu's default flush before every launch the figures are 73 729 / 78 150 / 21 539 B (DRAM read ==
# algorithmic read).
NCU_DECODE_TRAFFIC_PER_UNIT = {(1, 16): 58505.0, (2, 16): 72364.0, (3, 16): 18637.0}


def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, flag in zip(names, r[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def unit_shape(wl: workloads.Workload, ulog16: bool = False, base16: bool = False) -> traffic.UnitShape:
    io = 4 if wl.io_dtype == torch.float32 else 2
    ul = 4 if wl.op in (workloads.GDN, workloads.KDA) and not ulog16 else io  # b = v keeps the I/O dtype
    return traffic.UnitShape(wl.op, wl.d, wl.d, io_bytes=io, klog_bytes=io, ulog_bytes=ul,
                             state_bytes=2 if base16 else 4)


class Rig:
    """Device-resident state and a ring of pre-generated token batches for one workload / capacity."""

    RING = 8

    def __init__(self, wl, cap, device, seed_offset=0, layers=1, ulog16=False, base16=False):
        import paper_2608_15533_b200 as dl

        self.dl, self.wl, self.cap, self.device, self.layers = dl, wl, cap, device, layers
        io = dl.F32 if wl.io_dtype == torch.float32 else dl.BF16
        base = dl.BF16 if base16 else dl.F32   # the 16-bit dense state is a variant; the configurations name fp32
        self.desc = dl.Desc(op=wl.op, num_slots=wl.slots, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=io,
                            ulog_dtype=io if ulog16 else None, base_dtype=base)
        # the same problem with the promise that the launch in front of a decode step leaves the base
        # alone (true for every decode step of a cycle but the first after a merge)
        self.desc_chained = dl.Desc(op=wl.op, num_slots=wl.slots, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=io,
                                    ulog_dtype=io if ulog16 else None, hints=dl.HINT_BASE_UNTOUCHED, base_dtype=base)
        self.chain = os.environ.get("DELTALOG_BENCH_CHAIN", "1") != "0"
        self.states, self.rings, self.bonus = [], [], []
        for layer in range(layers):
            src = workloads.TokenSource(wl, device=device, seed=wl.seed + 1000 * seed_offset + layer)
            S0 = src.initial_state()
            self.states.append(dl.State(self.desc, S0.to(torch.bfloat16) if base16 else S0))
            self.bonus.append(src.bonus())
            self.rings.append([src.token() for _ in range(self.RING)])
        self.out = torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype, device=device)
        self.slot_idx = None
        self.staggered = bool(wl.staggered)
        self.predicate_merge = False   # staggered batches: one predicate merge over the whole batch instead of listed rows
        self.phase = 0
        # several layers with staggered fills: merges off the critical path, on a side stream
        self.overlap_merges = (bool(wl.staggered) and layers > 1 and
                               os.environ.get("DELTALOG_BENCH_OVERLAP", "1") != "0")
        if self.staggered:  # serving shape: rows address a shuffled slot pool, every row at its own log fill
            self.slot_idx = workloads.slot_permutation(wl).to(device)
            self.delay = ((cap - workloads.fill_offsets(wl, cap)) % cap).to(device)
            # the host knows every row's phase from its step counter: before step t the rows with
            # delay == t mod cap hold a full log; their slots, listed per residue, are what the merge gets
            self.full_slots = [self.slot_idx[self.delay == r].contiguous() for r in range(cap)]

    def decode(self, t, layer=0, slot_idx=None, chained=False):
        """``chained``: the launch in front of this one on the stream was a decode step of this state."""
        tok = self.rings[layer][t % self.RING]
        self.dl.decode_step(self.desc_chained if (chained and self.chain) else self.desc, self.states[layer], tok["q"], tok["k"], tok["v"], tok["g"],
                            beta=tok["beta"], u_bonus=self.bonus[layer],
                            slot_idx=self.slot_idx if slot_idx is None else slot_idx, out=self.out)

    def fused(self, t, layer=0):
        tok = self.rings[layer][t % self.RING]
        self.dl.decode_merge_step(self.desc, self.states[layer], tok["q"], tok["k"], tok["v"], tok["g"],
                                  beta=tok["beta"], u_bonus=self.bonus[layer], slot_idx=self.slot_idx, out=self.out)

    def merge(self, layer=0, only_if_full=None):
        if only_if_full is None:   # a uniform batch folds every row at once; a staggered one uses the predicate
            only_if_full = self.staggered
        self.dl.merge(self.desc, self.states[layer], slot_idx=self.slot_idx, n=self.wl.batch,
                      only_if_full=only_if_full)

    def stag_merge(self, layer=0):
        """Staggered batch, before a decode step: fold the rows whose log is full -- listed by the host,
        which knows every row's phase (``self.phase`` = steps since the fills were laid out, mod cap),
        or found by the predicate merge over the whole batch."""
        if self.predicate_merge:
            return self.merge(layer, only_if_full=True)
        slots = self.full_slots[self.phase]
        if slots.numel():
            self.dl.merge(self.desc, self.states[layer], slot_idx=slots, n=slots.numel(), only_if_full=False)

    def end_layer(self, layer):
        if self.staggered and layer == self.layers - 1:
            self.phase = (self.phase + 1) % self.cap

    def step(self, t, layer=0):
        """One step of the hot path for one layer.  Uniform batch: decode, and the merge after every
        cap-th step.  Staggered batch: a merge of the rows whose log is full (about 1/cap of the rows per
        step), then decode."""
        if self.staggered:
            self.stag_merge(layer)
            self.decode(t, layer)
            self.end_layer(layer)
        else:
            self.decode(t, layer, chained=(self.layers == 1 and t % self.cap != 0))
            if (t + 1) % self.cap == 0:
                self.merge(layer)

    def reset_logs(self):
        """Fold everything; a staggered batch is then rolled forward so that row b holds
        (cap - delay_b) entries: rows sit out (slot -1) until their start step, real decode steps
        fill the logs (nothing is fabricated)."""
        for layer in range(self.layers):
            self.merge(layer, only_if_full=False)
        if self.staggered:
            for t in range(self.cap):
                slots = torch.where(self.delay <= t, self.slot_idx, torch.full_like(self.slot_idx, -1))
                for layer in range(self.layers):
                    self.decode(t, layer, slot_idx=slots)
        self.phase = 0   # before the next step exactly the rows with delay 0 hold a full log

    def status(self):
        return [int(s.status.item()) for s in self.states]


def time_cycle_loop(rig: Rig, steps: int, per_kernel: bool = True):
    """Time exactly ``steps`` steps (decode every step, merge after every cap-th) as plain launches
    on the current stream.  With ``per_kernel`` two events per cycle split the time into decode
    launches and the merge launch (an event between every pair of launches would itself cost
    several microseconds per step); returns total ms, summed decode ms, summed merge ms, merges."""
    cap = rig.cap
    ev = lambda: torch.cuda.Event(enable_timing=True)
    start, end = ev(), ev()
    marks = []  # (event before the first decode of a cycle, event after its last decode, event after its merge)
    launch.barrier()
    torch.cuda.synchronize()
    start.record()
    for t in range(steps):
        for layer in range(rig.layers):
            if rig.staggered:
                if per_kernel and layer == 0:  # one layer in `layers` carries the events
                    marks.append([ev(), ev(), ev()])
                    marks[-1][1].record()       # merge first here: [1] -> merge -> [2]=[0] -> decode -> end
                    rig.stag_merge(layer)
                    marks[-1][0].record()
                    rig.decode(t, layer)
                    marks[-1][2].record()
                    rig.end_layer(layer)
                else:
                    rig.step(t, layer)
                continue
            if per_kernel and layer == 0 and t % cap == 0:
                marks.append([ev(), None, None])
                marks[-1][0].record()
            rig.decode(t, layer, chained=(rig.layers == 1 and t % cap != 0))
            if (t + 1) % cap == 0:
                if per_kernel and layer == 0:
                    marks[-1][1] = ev(); marks[-1][1].record()
                rig.merge(layer)
                if per_kernel and layer == 0:
                    marks[-1][2] = ev(); marks[-1][2].record()
    end.record()
    torch.cuda.synchronize()
    launch.barrier()
    total = start.elapsed_time(end)
    full = [m for m in marks if m[2] is not None]
    if rig.staggered:  # per step: [1] merge [0] decode [2]
        dec = sum(a.elapsed_time(c) for a, _, c in full) if per_kernel else None
        mrg = sum(b.elapsed_time(a) for a, b, _ in full) if per_kernel else None
    else:              # per cycle: [0] cap decodes [1] merge [2]
        dec = sum(a.elapsed_time(b) for a, b, _ in full) if per_kernel else None
        mrg = sum(b.elapsed_time(c) for _, b, c in full) if per_kernel else None
    return total, dec, mrg, len(full)


def graph_steps(cap: int, staggered: bool = False) -> int:
    """Steps per captured graph: whole cycles that also return to the start of the token ring (in a
    staggered batch the list of rows to fold repeats with period cap as well)."""
    import math

    return cap * Rig.RING // math.gcd(cap, Rig.RING)


def capture_steps_with_merges_on_a_side_stream(rig: Rig, n_steps: int, main: "torch.cuda.Stream"):
    """Serving shape (several layers, staggered fills), called inside a graph capture on ``main``: the
    token-less merge of a layer depends on nothing but that layer's own previous decode step, not on
    activations, so it does not have to sit on the critical path between two layers.  The merges run
    on a side stream -- merge(layer, step t) after decode(layer, step t-1) -- and each decode step only
    waits for its own layer's merge: the merge CTAs share the SMs with the persistent decode CTA of
    another layer (their shared memory and registers fit beside it)."""
    side = torch.cuda.Stream(device=rig.device)
    ev = lambda: torch.cuda.Event()
    fork = ev()
    fork.record(main)
    side.wait_event(fork)
    decoded = [None] * rig.layers          # event after the latest decode step of every layer
    for t in range(n_steps):
        merged = []
        with torch.cuda.stream(side):
            for layer in range(rig.layers):
                if decoded[layer] is not None:
                    side.wait_event(decoded[layer])
                rig.stag_merge(layer)
                merged.append(ev())
                merged[-1].record(side)
        with torch.cuda.stream(main):
            for layer in range(rig.layers):
                main.wait_event(merged[layer])
                rig.decode(t, layer)
                decoded[layer] = ev()
                decoded[layer].record(main)
        rig.phase = (rig.phase + 1) % rig.cap
    join = ev()
    join.record(side)
    main.wait_event(join)


def time_graph_loop(rig: Rig, steps: int):
    """Time exactly ``steps`` steps replayed from one CUDA graph that holds ``graph_steps`` steps
    (decode launches and the merge launches between them), the way a serving loop would run the
    cycle.  ``steps`` must be a multiple of the graph length.  Returns total ms."""
    g_len = graph_steps(rig.cap, rig.staggered)
    assert steps % g_len == 0
    stream = torch.cuda.Stream(device=rig.device)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            if rig.overlap_merges:
                capture_steps_with_merges_on_a_side_stream(rig, g_len, stream)
            else:
                for t in range(g_len):
                    for layer in range(rig.layers):
                        rig.step(t, layer)
        graph.replay()  # warm the replay path; a graph holds whole cycles, so every replay starts in the same phase
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launch.barrier()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        start.record()
        for _ in range(steps // g_len):
            graph.replay()
        end.record()
    torch.cuda.synchronize()
    launch.barrier()
    return start.elapsed_time(end)


def time_paper_cycle(rig: Rig, steps: int):
    """The paper's own cycle (Algorithm 1): cap appends, then one fused step that consumes a token and
    materialises; cap + 1 tokens per dense write.  Uniform batch: one launch per step.  Staggered batch
    (fills uniform on 0..cap): every step is two launches over phase-split batches -- the append
    call sees slot -1 for the rows whose log is full, the fused-step call gets exactly those rows as
    its batch; the host knows each row's phase from its step counter, so the lists are precomputed for
    one period.
    Timed as CUDA-graph replays of whole cycles; on a single-layer uniform batch the fused step alone
    is then timed over plain launches with one event pair per cycle.
    Returns (steps timed, total ms, mean ms of a fused-step launch or None)."""
    import math

    cap, M = rig.cap, rig.cap + 1
    g_len = M * Rig.RING // math.gcd(M, Rig.RING)
    steps = max(steps // g_len, 1) * g_len
    for layer in range(rig.layers):
        rig.merge(layer, only_if_full=False)
    dl = rig.dl
    app_lists = blocks = slots_sorted = None
    if rig.staggered:
        # Rows are relabelled so that the rows of one phase are consecutive (the token tensors are
        # synthetic, the relabelling only permutes which slot a row addresses): the merge-phase batch
        # of a step is then a contiguous slice of the token tensors, as a runtime with separate append
        # and merge queues would hand it over.
        delay, order = torch.sort(workloads.fill_offsets(rig.wl, M).to(rig.device))  # row b starts `delay` steps late
        slots_sorted = rig.slot_idx[order].contiguous()
        skip = torch.full_like(slots_sorted, -1)
        for t in range(cap):
            slots = torch.where(delay <= t, slots_sorted, skip)
            for layer in range(rig.layers):
                rig.decode(t, layer, slot_idx=slots)
        app_lists, blocks = [], []
        for tau in range(M):                                   # a row is full before step tau iff delay == tau
            full = delay == tau
            app_lists.append(torch.where(full, skip, slots_sorted))
            idx = torch.nonzero(full).flatten()
            blocks.append((int(idx[0]), int(idx[-1]) + 1) if idx.numel() else None)

    def one(t, layer):
        tok = rig.rings[layer][t % rig.RING]
        args = (rig.desc, rig.states[layer], tok["q"], tok["k"], tok["v"], tok["g"])
        kw = dict(beta=tok["beta"], u_bonus=rig.bonus[layer], out=rig.out)
        if rig.staggered:
            dl.decode_step(*args, slot_idx=app_lists[t % M], **kw)
            if blocks[t % M] is not None:
                lo, hi = blocks[t % M]
                dl.decode_merge_step(rig.desc, rig.states[layer], tok["q"][lo:hi], tok["k"][lo:hi], tok["v"][lo:hi],
                                     tok["g"][lo:hi], beta=tok["beta"][lo:hi] if tok["beta"] is not None else None,
                                     u_bonus=rig.bonus[layer], slot_idx=slots_sorted[lo:hi], out=rig.out[lo:hi])
        elif t % M == M - 1:
            dl.decode_merge_step(*args, slot_idx=rig.slot_idx, **kw)
        else:   # every append but the first after the fused step follows a decode step of this state
            desc = rig.desc_chained if (rig.chain and rig.layers == 1 and t % M != 0) else rig.desc
            dl.decode_step(desc, *args[1:], slot_idx=rig.slot_idx, **kw)

    stream = torch.cuda.Stream(device=rig.device)
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            for t in range(g_len):
                for layer in range(rig.layers):
                    one(t, layer)
        graph.replay()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        start.record()
        for _ in range(steps // g_len):
            graph.replay()
        end.record()
    torch.cuda.synchronize()
    total = start.elapsed_time(end)
    fused_ms = None
    if not rig.staggered and rig.layers == 1:
        marks = []
        for t in range(min(steps, 32 * M)):
            if t % M == M - 1:
                marks.append((torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)))
                marks[-1][0].record()
                one(t, 0)
                marks[-1][1].record()
            else:
                one(t, 0)
        torch.cuda.synchronize()
        fused_ms = statistics.mean(a.elapsed_time(b) for a, b in marks)
    return steps, total, fused_ms


def time_eager_loop(rig: Rig, S: torch.Tensor, steps: int, use_graph: bool = True):
    """The eager dense comparator on the same token ring, launched the same way as the main loop."""
    dl = rig.dl

    def launch_steps(n):
        for t in range(n):
            tok = rig.rings[0][t % rig.RING]
            dl.eager_step(rig.desc, S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                          u_bonus=rig.bonus[0], out=rig.out)

    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    use_graph = use_graph and steps % rig.RING == 0
    stream = torch.cuda.Stream(device=rig.device) if use_graph else torch.cuda.current_stream()
    graph = None
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        if use_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                launch_steps(rig.RING)
            graph.replay()
        else:
            launch_steps(rig.RING)
        torch.cuda.synchronize()
        start.record()
        if use_graph:
            for _ in range(steps // rig.RING):
                graph.replay()
        else:
            launch_steps(steps)
        end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end)


def time_e2e_loop(rig: Rig, steps: int, use_graph: bool = True):
    """The same cycle through the host-buffer entry point: every step copies q, k, v, g, beta from
    pinned host memory and reads the output back to pinned host memory.  Copy-in, kernel and
    copy-out run on three streams over two staging sets (``deltalog_decode_step_host_overlapped``),
    so the copies of step t+1 and t-1 overlap the kernel of step t."""
    dl, wl = rig.dl, rig.wl
    streams = [torch.cuda.Stream(device=rig.device) for _ in range(3)]
    sets = [(dl.HostStaging(rig.desc, wl.batch, rig.device), dl.HostLane(*streams),
             torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory()) for _ in range(2)]
    for staging, _, _ in sets:
        staging.packed = True   # host tokens below come from packed_host_tokens: one copy per step
    host_ring = []
    for tok in rig.rings[0]:   # pinned host tokens, packed so that a step's inputs travel in one copy
        host = dl.packed_host_tokens(rig.desc, wl.batch)
        for k, v in tok.items():
            if v is not None:
                host[k].copy_(v)
            else:
                host[k] = None
        host_ring.append(host)
    rig.reset_logs()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def run(n):
        with torch.cuda.stream(streams[1]):  # merges go to the compute stream
            if rig.staggered:
                rig.merge(0)   # rows whose log is full fold before the first decode
            for t in range(n):
                tok = host_ring[t % rig.RING]
                staging, lane, host_out = sets[t % 2]
                dl.decode_step_host_overlapped(rig.desc, rig.states[0], staging, lane, tok["q"], tok["k"], tok["v"],
                                               tok["g"], tok["beta"], host_out, u_bonus=rig.bonus[0],
                                               slot_idx=rig.slot_idx)
                if rig.staggered or (t + 1) % rig.cap == 0:
                    rig.merge(0)   # predicate merge: after the step here, i.e. before the next decode

    run(rig.cap)  # warm the copy path, ends on a merge
    for st in streams:
        st.synchronize()
    # The serving-loop form: whole cycles of the three-stream pipeline (copies in, kernels, copies out,
    # with their event dependencies) captured once into a CUDA graph through the same entry point and
    # replayed; the host then only refills the pinned token buffers.  Falls back to plain calls.
    import math
    g_len = rig.cap * rig.RING // math.gcd(rig.cap, rig.RING)
    graph = None
    if use_graph and steps % g_len == 0 and not rig.staggered:
        try:
            graph = torch.cuda.CUDAGraph()
            fork, j_in, j_out = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
            with torch.cuda.graph(graph, stream=streams[1]):
                fork.record(streams[1])                      # bring the copy streams into the capture
                streams[0].wait_event(fork)
                streams[2].wait_event(fork)
                for _, lane, _ in sets:                      # the lanes' events must belong to the capture
                    lane.in_done.record(streams[0])
                    lane.compute_done.record(streams[1])
                    lane.out_done.record(streams[2])
                run(g_len)
                j_in.record(streams[0])
                j_out.record(streams[2])
                streams[1].wait_event(j_in)
                streams[1].wait_event(j_out)
            graph.replay()
            torch.cuda.synchronize()
        except Exception as exc:  # capture not possible here: time the plain calls instead
            print(f"[bench] end-to-end graph capture failed ({type(exc).__name__}: {exc}); timing plain calls", file=sys.stderr)
            graph = None
            torch.cuda.synchronize()
            rig.reset_logs()
            torch.cuda.synchronize()
    launch.barrier()
    torch.cuda.synchronize()
    if graph is not None:
        with torch.cuda.stream(streams[1]):
            start.record(streams[1])
            for _ in range(steps // g_len):
                graph.replay()
            end.record(streams[1])
    else:
        start.record(streams[1])
        run(steps)
        for st in streams:
            st.synchronize()
        end.record(streams[1])
    torch.cuda.synchronize()
    launch.barrier()
    assert all(s == 0 for s in rig.status()), f"device status bits set: {rig.status()}"
    staging = sets[0][0]
    return start.elapsed_time(end), staging.h2d_bytes(rig.desc), staging.d2h_bytes()


def cpu_baseline(wl, units: int, steps: int, chunk_units: int = 1024):
    """Time the fp64 oracle, as it stands, on a bounded sample of the workload's units.

    The sample is rolled through the oracle in chunks of ``chunk_units`` units (only the oracle
    call itself is timed) so that the fp64 copies of the inputs stay small on the host.
    """
    import numpy as np

    import oracle

    done, dt = 0, 0.0
    while done < units:
        n_units = min(chunk_units, units - done)
        small = wl.scaled(batch=max(1, n_units // wl.H), num_slots=None, seed=wl.seed + done)
        src = workloads.TokenSource(small, device="cpu")
        S0 = src.initial_state().double().numpy().reshape(-1, wl.d, wl.d)
        bonus = src.bonus()
        N = S0.shape[0]
        toks = [src.token() for _ in range(steps)]
        f = lambda key: np.stack([t[key].double().numpy().reshape(N, -1) for t in toks])
        q, k, v, g = f("q"), f("k"), f("v"), f("g")
        beta = f("beta")[..., 0] if wl.op != workloads.RWKV6 else None
        bon = np.tile(bonus.double().numpy(), (small.batch, 1)) if bonus is not None else None
        t0 = time.perf_counter()
        oracle.eager_rollout(wl.op, S0, q, k, v, g, beta=beta, bonus=bon)
        dt += time.perf_counter() - t0
        done += N
    return {"value": done * steps / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{done} (seq*head) units x {steps} tokens of {wl.name}, fp64 eager recurrence, "
                      f"{dt:.2f} s on {oracle.num_threads()} threads"}, dt


def run_reference(args, wl):
    """``--impl reference``: the CPU oracle timed on the host cores (rank 0 only)."""
    rank, size, _ = launch.world()
    if rank != 0:
        return
    units = 512 if args.steps <= 256 else 128   # bounds the fp64 input copies on the host (units x steps)
    base, dt = cpu_baseline(wl, units, max(args.steps, 1))
    n_units = max(1, units // wl.H) * wl.H
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "sample_units_per_step": n_units,
                   "note": "each step is one token over a bounded sample of the workload's units on the host"},
        "cpu_baseline": {**base},
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2048)
    ap.add_argument("--warmup", type=int, default=256)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, choices=[1, 2, 3, 4])
    ap.add_argument("--cap", type=int, default=16, help="log capacity of the headline number")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of CUDA-graph replays")
    ap.add_argument("--no-extras", action="store_true", help="skip the capacity sweep, eager and CPU legs")
    ap.add_argument("--state", default="fp32", choices=["fp32", "bf16"],
                    help="dtype of the dense state; bf16 is the 16-bit-state variant (the configurations name fp32)")
    ap.add_argument("--only-hot-loop", action="store_true",
                    help="warm-up and timed loop only (for profiler captures)")
    args = ap.parse_args()
    wl = workloads.CONFIGS[args.config]
    if args.impl == "reference":
        return run_reference(args, wl)

    rank, size, local = launch.init("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    import paper_2608_15533_b200 as dl

    cap = args.cap
    warmup = max(args.warmup, 3)
    layers = wl.layers
    base16 = args.state == "bf16"
    rig = Rig(wl, cap, device, seed_offset=rank, layers=layers, base16=base16)
    stag = rig.staggered
    g_len = graph_steps(cap, stag)
    u = unit_shape(wl, base16=base16)
    units = wl.units

    # ---- warm-up, then the timed region: exactly K steps ---------------------------------------
    launches0 = dl.launch_count()
    rig.reset_logs()
    for t in range(warmup):
        for layer in range(layers):
            rig.step(t, layer)
    if not stag:
        rig.reset_logs()   # a uniform batch starts the timed region on empty logs
    torch.cuda.synchronize()
    warm_launches = dl.launch_count() - launches0
    if args.only_hot_loop:
        time_cycle_loop(rig, args.steps, per_kernel=False)
        return launch.finalize()
    use_graph = (not args.no_graph) and args.steps % g_len == 0
    with ClockSampler(local) as clocks:
        l0 = dl.launch_count()
        if use_graph:
            total_ms = time_graph_loop(rig, args.steps)
            # kernels executed by the replays (the host-side counter only sees the capture)
            gpu_launches = layers * (2 * args.steps if stag else args.steps + args.steps // cap)
        else:
            total_ms, _, _, _ = time_cycle_loop(rig, args.steps, per_kernel=False)
            gpu_launches = dl.launch_count() - l0
        # same steps again as plain launches with two events per cycle: the split into decode and merge time
        split_ms, dec_ms, mrg_ms, n_merges = time_cycle_loop(rig, args.steps)
    assert all(s == 0 for s in rig.status()), f"device status bits set: {rig.status()}"
    total_ms = launch.max_over_ranks(total_ms, device)
    all_units = launch.sum_over_ranks(units * layers, device)
    ms_per_step = total_ms / args.steps
    value = all_units * args.steps / (total_ms * 1e-3)

    cyc = traffic.cycle_bytes(u, cap)
    peak, peak_kind = measured_peak_gbs()
    fills = [t % cap for t in range(args.steps)]
    dec_bytes = statistics.mean(traffic.decode_read(u, f) + traffic.decode_write(u) for f in fills) * units
    # events bracket cap decode launches per mark in a uniform batch, one decode launch per mark in a staggered one
    dec_ms_avg = dec_ms / (n_merges * (1 if stag else cap)) if n_merges else float("nan")
    achieved = dec_bytes / (dec_ms_avg * 1e-3) / 1e9
    traffic_ncu = None if base16 else NCU_DECODE_TRAFFIC_PER_UNIT.get((args.config, cap))
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": size, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": f"configs[{args.config}] {wl.name}", "op": workloads.OP_NAMES[wl.op], "batch": wl.batch,
            "H": wl.H, "d_k": wl.d, "d_v": wl.d, "layers": layers, "log_capacity": cap, "state": args.state,
            "io": str(wl.io_dtype).replace("torch.", ""), "merge": ("before every step the rows whose log is full (listed by the host from its step counters) are folded; fills staggered over 0..cap-1"
                      + ("; the merges run on a side stream, overlapped with other layers' decode steps" if rig.overlap_merges and use_graph else "") if stag
                      else f"after every {cap}th step"),
            "launch": (f"one CUDA graph of {g_len} steps, replayed" if use_graph else "plain launches"),
            "l2": f"inputs larger than L2: {units * u.state * layers / 2**20:.0f} MiB of base state per step, no flush",
            "parallelism": f"rows sharded over {size} GPU(s), no collective",
        },
        "clocks": clocks.summary(),
        "gpu_launches": gpu_launches,
        "roofline": {
            "bound": "hbm", "kernel": "decode_pipelined_kernel" if wl.d == 128 else "decode_append_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic_ncu * units if traffic_ncu else None,
            "traffic_note": ("ncu --cache-control none (L2 as the previous launch left it, as in the timed loop): base tiles are "
                             "read evict-first, so part of the live log is served by L2 and DRAM traffic is below the "
                             "algorithmic bytes that `achieved` counts"),
            "algorithmic_bytes_per_launch": dec_bytes, "avg_launch_ms": dec_ms_avg,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        },
        "amortized": {
            "algorithmic_bytes_per_unit_step": cyc["total"],
            "hbm_gbs": cyc["total"] * all_units / (ms_per_step * 1e-3) / 1e9,
            "bytes_written_per_unit_step": cyc["write"], "write_reduction_vs_eager": cyc["write_reduction"],
            "decode_ms_per_step": dec_ms_avg, "merge_ms_per_merge": (mrg_ms / n_merges) if n_merges else None,
            "plain_launch_ms_per_step": split_ms / args.steps,
        },
    }
    line["amortized"]["frac_of_nominal_8TBs"] = line["amortized"]["hbm_gbs"] / NOMINAL_HBM_GBS / size
    line["amortized"]["frac_of_measured"] = line["amortized"]["hbm_gbs"] / peak / size

    # ---- end-to-end leg: token tensors from pinned host memory, output back to the host --------
    e2e_ms, h2d, d2h = time_e2e_loop(rig, args.steps, use_graph)
    e2e_ms = launch.max_over_ranks(e2e_ms, device)
    e2e_units = launch.sum_over_ranks(units, device)
    line["e2e"] = {"value": e2e_units * args.steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps,
                   "note": "state stays resident; q,k,v,g,beta in and out back every step, layer 0"}

    if not args.no_extras and rank == 0:
        # eager dense comparator on the same inputs
        rig.reset_logs()
        S = rig.states[0].S_base
        eager_ms = time_eager_loop(rig, S, args.steps, use_graph) / args.steps
        eager_bytes = (traffic.eager_read(u) + traffic.eager_write(u)) * units
        line["eager_kernel"] = {"ms_per_step": eager_ms, "value": units / (eager_ms * 1e-3),
                                "hbm_gbs": eager_bytes / (eager_ms * 1e-3) / 1e9,
                                "bytes_written_per_unit_step": traffic.eager_write(u)}
        line["speedup_vs_eager_kernel"] = eager_ms / (ms_per_step / layers)
        # the paper's own cycle: cap appends + one fused merge step (cap + 1 tokens per dense write)
        p_steps, p_ms, fused_ms = time_paper_cycle(rig, args.steps)
        pc = traffic.paper_cycle_bytes(u, cap + 1)
        p_step_ms = p_ms / p_steps
        line["paper_cycle"] = {
            "ms_per_step": p_step_ms, "value": units * layers * p_steps / (p_ms * 1e-3), "steps": p_steps,
            "merge_interval_M": cap + 1, "algorithmic_bytes_per_unit_step": pc["total"],
            "hbm_gbs": pc["total"] * units * layers / (p_step_ms * 1e-3) / 1e9,
            "launch": ("two launches per layer-step over phase-split batches" if stag else "one launch per step"),
            "speedup_vs_eager_kernel": eager_ms / (p_step_ms / layers)}
        if fused_ms is not None:
            fused_bytes = (traffic.fused_read(u, cap) + traffic.fused_write(u)) * units
            line["paper_cycle"]["fused_step_ms"] = fused_ms
            line["paper_cycle"]["fused_step_hbm_gbs"] = fused_bytes / (fused_ms * 1e-3) / 1e9
        assert all(s == 0 for s in rig.status()), f"device status bits set: {rig.status()}"
        sweep = {}
        for c in wl.caps:
            if c == cap and layers == 1:
                sweep[str(c)] = {"ms_per_step": ms_per_step, "value": value,
                                 "write_reduction_vs_eager": cyc["write_reduction"],
                                 "hbm_gbs": line["amortized"]["hbm_gbs"]}
                continue
            if layers > 1:
                continue
            del rig
            torch.cuda.empty_cache()
            rig = Rig(wl, c, device, seed_offset=rank, base16=base16)
            for t in range(max(c, 3)):
                rig.decode(t);
                if (t + 1) % c == 0:
                    rig.merge()
            rig.reset_logs()
            ms = time_graph_loop(rig, args.steps) if use_graph and args.steps % graph_steps(c) == 0 else \
                time_cycle_loop(rig, args.steps, per_kernel=False)[0]
            cc = traffic.cycle_bytes(u, c)
            sweep[str(c)] = {"ms_per_step": ms / args.steps, "value": units * args.steps / (ms * 1e-3),
                             "write_reduction_vs_eager": cc["write_reduction"],
                             "hbm_gbs": cc["total"] * units / (ms / args.steps * 1e-3) / 1e9}
        line["capacity_sweep"] = sweep
        small = wl.scaled(layers=1)
        line["cpu_baseline"], _ = cpu_baseline(small, min(wl.units, 4096), 128)
    if rank == 0:
        print(json.dumps(line))
    launch.finalize()


if __name__ == "__main__":
    main()
