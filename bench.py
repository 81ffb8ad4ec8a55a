#!/usr/bin/env python
"""Benchmark of the DeltaLog decode hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..4] [--cap C] [--impl ours|reference]

One "step" is one decode token for the whole batch of the workload: the decode+append kernel, and
the merge kernel whenever the logs are full (after every ``cap``-th step), i.e. the complete hot path.
The timed region is EXACTLY K steps starting from empty logs, so it contains ``K // cap`` merges; any
K >= 1 works.  A short region is repeated (the logs are emptied before every repetition, outside the
timed region) and the median over the repetitions is reported; ``steps`` stays K.
Rank 0 prints ONE JSON line.  ``value`` is (sequence*head) state updates per second with all inputs
resident in HBM; ``e2e`` is the same metric through ``deltalog_decode_step_host_overlapped`` with the
token tensors in pinned host memory and the output read back to the host every step.

``roofline`` describes the decode kernel.  Two byte counts appear side by side: ``traffic`` is DRAM
traffic per launch measured by ncu (``profiles/dram_traffic.json``, valid only for the library build
it was captured on -- ``null`` otherwise), and ``algorithmic_bytes_per_launch`` is what the method
must move; since the kernels ask L2 to keep the live log, part of the algorithmic bytes never reach
DRAM.  ``achieved`` / ``frac`` are the DRAM figures when a matching capture exists
(``achieved_kind`` says which); the algorithmic ones are always given as ``*_algorithmic_incl_l2``.

With N > 1 (one process per GPU, launched by ``torch.distributed.run``) every rank decodes its own
shard of the global batch rows -- the path has no exchange step -- and the time is the maximum over
ranks.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
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
from paper_2608_15533_b200 import launch, ncu_traffic, traffic  # noqa: E402

METRIC = "state-update (seq*head)-steps/s"
UNIT = "(seq*head)-steps/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
TARGET_TIMED_MS = 300.0     # a short K-step region is repeated until about this much has been timed
MAX_REPEATS, MIN_REPEATS = 25, 3


def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons while the timed regions run: NVML from a thread every
    2 ms (a K-step region can be shorter than a millisecond, far below what ``nvidia-smi -lms`` resolves),
    ``nvidia-smi`` as the fallback.  Samples taken while ``busy`` is set count as "under load"."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu, self.rows, self.busy, self.stop = gpu_index, [], False, False
        self.proc = self.thread = self.nvml = self.handle = None
        self.sm_max = None

    def _nvml_handle(self):
        import pynvml

        pynvml.nvmlInit()
        self.nvml = pynvml
        props = torch.cuda.get_device_properties(self.gpu)
        uuid = getattr(props, "uuid", None)
        if uuid is not None:
            try:
                return pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                pass
        return pynvml.nvmlDeviceGetHandleByIndex(self.gpu)

    def __enter__(self):
        try:
            self.handle = self._nvml_handle()
            self.sm_max = float(self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll_nvml, daemon=True)
            self.thread.start()
            return self
        except Exception:
            self.handle = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read_smi, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _poll_nvml(self):
        n = self.nvml
        reasons_fn = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(n, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self.stop:
            try:
                sm = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                mask = int(reasons_fn(self.handle))
                self.rows.append((sm, self.sm_max, [name for name, bit in self.REASONS if mask & bit], self.busy))
            except Exception:
                pass
            time.sleep(0.002)

    def _read_smi(self):
        names = [name for name, _ in self.REASONS]
        for line in self.proc.stdout:
            r = [c.strip() for c in line.split(",")]
            try:
                self.rows.append((float(r[0]), float(r[1]),
                                  [nm for nm, flag in zip(names, r[3:7]) if flag.lower().startswith("active")],
                                  self.busy))
            except (ValueError, IndexError):
                continue

    def __exit__(self, *exc):
        self.stop = True
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)

    def summary(self):
        rows = list(self.rows)
        loaded = [r for r in rows if r[3]]
        use = loaded if len(loaded) >= 3 else rows
        if not use:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(r[0] for r in use), "sm_max_mhz": max(r[1] for r in use),
                "reasons": sorted({name for r in use for name in r[2]}), "samples": len(use),
                "samples_under_load": len(loaded), "source": "nvml" if self.handle is not None else "nvidia-smi"}


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
        # the same problem with the promise that the launch in front of a decode step writes neither the
        # base nor the slot list (true for every decode step of a cycle but the first after a merge)
        self.desc_chained = dl.Desc(op=wl.op, num_slots=wl.slots, H=wl.H, d_k=wl.d, d_v=wl.d, cap=cap, io_dtype=io,
                                    ulog_dtype=io if ulog16 else None,
                                    hints=dl.HINT_BASE_UNTOUCHED | dl.HINT_SLOTS_STABLE, base_dtype=base)
        self.chain = os.environ.get("DELTALOG_BENCH_CHAIN", "1") != "0"
        # Consecutive decode steps of a state walk over the batch in alternating directions (an ordering hint, same
        # results): a step then starts with the base tiles the step before read last, which are still in L2.
        self.alternate = os.environ.get("DELTALOG_BENCH_ALTERNATE", "1") != "0"
        self._descs = {}
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

    def desc_for(self, chained=False, down=False):
        """The descriptor with the hints of one decode call: ``chained`` = the launch in front of it on the stream
        was a decode step of this state; ``down`` = walk over the batch from the last unit to the first."""
        hints = (self.desc_chained.hints if (chained and self.chain) else 0) | \
                (self.dl.HINT_WALK_DOWN if (down and self.alternate) else 0)
        if hints not in self._descs:
            self._descs[hints] = dataclasses.replace(self.desc, hints=hints)
        return self._descs[hints]

    def decode(self, t, layer=0, slot_idx=None, chained=False, fill=None):
        """``chained``: the launch in front of this one on the stream was a decode step of this state.  ``fill``: the
        step's place in its cycle (default t mod cap): odd places walk downwards -- the merge and the fused step walk
        downwards themselves, so place 0 walks upwards."""
        tok = self.rings[layer][t % self.RING]
        place = (t % self.cap) if fill is None else fill
        self.dl.decode_step(self.desc_for(chained, down=bool(place & 1)), self.states[layer], tok["q"], tok["k"], tok["v"], tok["g"],
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
        """Step ``t`` (counted from the last ``reset_logs``) of the hot path for one layer.  Uniform batch:
        decode, and the merge after every cap-th step.  Staggered batch: a merge of the rows whose log is
        full (about 1/cap of the rows per step), then decode."""
        if self.staggered:
            self.stag_merge(layer)
            self.decode(t, layer)
            self.end_layer(layer)
        else:
            self.decode(t, layer, chained=(self.layers == 1 and t % self.cap != 0))
            if (t + 1) % self.cap == 0:
                self.merge(layer)

    def reset_logs(self):
        """Fold everything, so that the next step is step 0 of a cycle; a staggered batch is then rolled
        forward so that row b holds (cap - delay_b) entries: rows sit out (slot -1) until their start step,
        real decode steps fill the logs (nothing is fabricated)."""
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

    def check_status(self, where):
        st = self.status()
        if any(st):
            raise RuntimeError(f"{where}: device status bits set: {st} (1 = log full, 2 = bad slot, 4 = wait timed out)")


def merges_in(steps: int, cap: int) -> int:
    """Merges inside a region of ``steps`` steps that starts on empty logs (uniform batch)."""
    return steps // cap


def graph_steps(cap: int) -> int:
    """Steps per captured graph: whole cycles that also return to the start of the token ring (in a
    staggered batch the list of rows to fold repeats with period cap as well)."""
    return cap * Rig.RING // math.gcd(cap, Rig.RING)


def segments(steps: int, seg: int):
    """Split ``steps`` into ``(full segments of length seg, remainder)``."""
    return steps // seg, steps % seg


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


class Region:
    """Enqueues EXACTLY ``steps`` steps of the hot path, starting from what ``reset_logs`` leaves.

    With ``use_graph`` the steps are replayed from CUDA graphs the way a serving loop would run the
    cycle: one graph of ``graph_steps(cap)`` steps (whole cycles that also return to the start of the
    token ring) replayed ``steps // graph_steps`` times, and a second graph holding the remaining
    ``steps % graph_steps`` steps; otherwise the steps are plain launches.  ``launches`` is the number of
    kernels one pass over the region executes."""

    def __init__(self, rig: Rig, steps: int, use_graph: bool):
        self.rig, self.steps, self.use_graph = rig, steps, use_graph
        self.stream = torch.cuda.Stream(device=rig.device)
        self.plan, self.launches = [], None
        if use_graph:
            g_len = graph_steps(rig.cap)
            n_full, tail = segments(steps, g_len)
            self.launches = 0
            for n, reps in ((g_len, n_full), (tail, 1)):
                if n and reps:
                    graph, count = self._capture(n)
                    self.plan.append((graph, reps))
                    self.launches += count * reps
            self.describe = (f"CUDA graphs: {n_full} replay(s) of a {g_len}-step graph"
                             + (f" + one {tail}-step graph" if tail else ""))
        else:
            self.describe = "plain launches"

    def _capture(self, n):
        rig, dl = self.rig, self.rig.dl
        graph = torch.cuda.CUDAGraph()
        rig.phase = 0     # every captured segment starts at the beginning of a cycle
        torch.cuda.synchronize()
        count0 = dl.launch_count()
        with torch.cuda.stream(self.stream):
            with torch.cuda.graph(graph, stream=self.stream):
                if rig.overlap_merges:
                    capture_steps_with_merges_on_a_side_stream(rig, n, self.stream)
                else:
                    for t in range(n):
                        for layer in range(rig.layers):
                            rig.step(t, layer)
        rig.phase = 0
        return graph, dl.launch_count() - count0   # the host-side counter sees the capture, not the replays

    def enqueue(self):
        """Called with ``self.stream`` current."""
        rig = self.rig
        if self.use_graph:
            for graph, reps in self.plan:
                for _ in range(reps):
                    graph.replay()
        else:
            count0 = rig.dl.launch_count()
            for t in range(self.steps):
                for layer in range(rig.layers):
                    rig.step(t, layer)
            self.launches = rig.dl.launch_count() - count0


def run_region_once(rig: Rig, steps: int, use_graph: bool) -> Region:
    """Empty the logs, then run exactly ``steps`` steps the way the timed region runs them (untimed)."""
    region = Region(rig, steps, use_graph)
    rig.reset_logs()
    torch.cuda.synchronize()
    with torch.cuda.stream(region.stream):
        region.enqueue()
    torch.cuda.synchronize()
    return region


def timed_passes(rig: Rig, enqueue, stream, clocks: "ClockSampler | None", device, reset=None):
    """Time the region ``enqueue`` puts on ``stream``: logs emptied, barrier + synchronize, events on the
    launching stream around the region, synchronize + barrier.  The first pass decides how often the
    region is repeated (about TARGET_TIMED_MS in all, between MIN_REPEATS and MAX_REPEATS passes; the
    count is taken from the maximum over ranks so that all ranks agree).  Returns the per-pass
    milliseconds, each the maximum over ranks."""
    reset = reset or rig.reset_logs
    reset()                       # one untimed pass first: graph upload, instruction caches, clocks
    torch.cuda.synchronize()      # (the reset runs on another stream than the region)
    with torch.cuda.stream(stream):
        enqueue()
    torch.cuda.synchronize()
    times = []
    n_pass = MAX_REPEATS
    while len(times) < n_pass:
        reset()
        torch.cuda.synchronize()
        launch.barrier()
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if clocks is not None:
            clocks.busy = True
        with torch.cuda.stream(stream):
            start.record()
            enqueue()
            end.record()
        torch.cuda.synchronize()
        if clocks is not None:
            clocks.busy = False
        launch.barrier()
        times.append(launch.max_over_ranks(start.elapsed_time(end), device))
        if len(times) == 1:
            n_pass = int(min(MAX_REPEATS, max(MIN_REPEATS, math.ceil(TARGET_TIMED_MS / max(times[0], 1e-3)))))
    return times


def time_kernel_split(rig: Rig, steps: int, passes: int = 3):
    """The same K steps as plain launches with events that split the time into decode launches and
    merge launches: one event pair around every run of consecutive decode launches (an event between
    every pair of launches would itself cost several microseconds per step) and one around every
    merge.  Returns ``(decode ms per launch, merge ms per launch or None, plain-launch ms per step)``,
    each the median over ``passes`` passes."""
    cap = rig.cap
    ev = lambda: torch.cuda.Event(enable_timing=True)
    dec_avg, mrg_avg, total = [], [], []
    for _ in range(passes):
        rig.reset_logs()
        torch.cuda.synchronize()
        start, end = ev(), ev()
        runs, merges = [], []   # (event, event, decode launches between them), (event, event)
        start.record()
        for t in range(steps):
            for layer in range(rig.layers):
                mark = layer == 0   # one layer carries the events
                if not mark:
                    rig.step(t, layer)
                    continue
                if rig.staggered:   # per step: merge of the listed rows, then the decode launch
                    a = ev(); a.record()
                    rig.stag_merge(layer)
                    b = ev(); b.record()
                    rig.decode(t, layer)
                    c = ev(); c.record()
                    rig.end_layer(layer)
                    if mark:
                        merges.append((a, b))
                        runs.append((b, c, 1))
                    continue
                if mark and t % cap == 0:
                    a = ev(); a.record()
                    run_start, run_n = a, 0
                rig.decode(t, layer, chained=(rig.layers == 1 and t % cap != 0))
                if mark:
                    run_n += 1
                last_of_run = (t + 1) % cap == 0 or t == steps - 1
                if mark and last_of_run:
                    b = ev(); b.record()
                    runs.append((run_start, b, run_n))
                if (t + 1) % cap == 0:
                    rig.merge(layer)
                    if mark:
                        c = ev(); c.record()
                        merges.append((b, c))
        end.record()
        torch.cuda.synchronize()
        dec_avg.append(sum(a.elapsed_time(b) for a, b, _ in runs) / sum(n for _, _, n in runs))
        if merges:
            mrg_avg.append(sum(a.elapsed_time(b) for a, b in merges) / len(merges))
        total.append(start.elapsed_time(end) / steps)
    return statistics.median(dec_avg), (statistics.median(mrg_avg) if mrg_avg else None), statistics.median(total)


def time_merge_alone(rig: Rig, passes: int = 3):
    """A merge of full logs on its own (uniform batch): used when the timed region holds no merge."""
    ev = lambda: torch.cuda.Event(enable_timing=True)
    res = []
    for _ in range(passes):
        rig.reset_logs()
        for t in range(rig.cap):
            rig.decode(t, 0)
        a, b = ev(), ev()
        torch.cuda.synchronize()
        a.record()
        rig.merge(0, only_if_full=False)
        b.record()
        torch.cuda.synchronize()
        res.append(a.elapsed_time(b))
    return statistics.median(res)


def time_paper_cycle(rig: Rig, steps: int):
    """The paper's own cycle (Algorithm 1): cap appends, then one fused step that consumes a token and
    materialises; cap + 1 tokens per dense write.  Uniform batch: one launch per step.  Staggered batch
    (fills uniform on 0..cap): every step is two launches over phase-split batches -- the append
    call sees slot -1 for the rows whose log is full, the fused-step call gets exactly those rows as
    its batch; the host knows each row's phase from its step counter, so the lists are precomputed for
    one period.
    Timed as CUDA-graph replays of whole cycles (the step count is rounded to whole graphs, at least
    one); on a single-layer uniform batch the fused step alone is then timed over plain launches with
    one event pair per cycle.
    Returns (steps timed, total ms, mean ms of a fused-step launch or None)."""
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
            desc = rig.desc_for(chained=(rig.layers == 1 and t % M != 0), down=bool((t % M) & 1))
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


class PhaseGraphs:
    """The paper's cycle the way a runtime that replays ONE graph per decode step runs it (Section 4):
    two phase-specialised CUDA graphs per batch descriptor -- an append graph holding one
    ``deltalog_decode_step`` and a merge graph holding one ``deltalog_decode_merge_step`` -- captured once
    over FIXED token, slot-list and output buffers; every step the host (which knows each row's phase
    from its step counter) refreshes the buffers and replays the graph of the phase.

    Uniform batch: all rows are in the same phase, one replay per step.  Staggered batch: both graphs are
    replayed every step over phase-split slot lists (a row sits out of a call with slot -1).  The token of
    a step reaches the fixed buffers with one device copy from the packed token ring, standing in for
    the projections that would write there."""

    def __init__(self, rig: Rig, layer: int = 0):
        dl = rig.dl
        self.rig, self.layer = rig, layer
        self.names = [k for k, v in rig.rings[layer][0].items() if v is not None]
        # token ring and the fixed buffers in one packed layout (256-byte aligned sections): one copy per step
        spans, off = {}, 0
        for k in self.names:
            t = rig.rings[layer][0][k]
            spans[k] = (off, t.numel() * t.element_size(), t.dtype, t.shape)
            off += (t.numel() * t.element_size() + 255) // 256 * 256
        self.packed_ring = []
        for tok in rig.rings[layer]:
            block = torch.zeros(off, dtype=torch.uint8, device=rig.device)
            for k in self.names:
                o, nb, _, _ = spans[k]
                block[o:o + nb].copy_(tok[k].reshape(-1).view(torch.uint8))
            self.packed_ring.append(block)
        self.fixed = torch.zeros(off, dtype=torch.uint8, device=rig.device)
        self.tok = {k: self.fixed[o:o + nb].view(dt).view(shape) for k, (o, nb, dt, shape) in spans.items()}
        B = rig.wl.batch
        rows = rig.slot_idx if rig.slot_idx is not None else torch.arange(B, dtype=torch.int32, device=rig.device)
        self.rows = rows
        self.app_slots, self.mrg_slots = rows.clone(), rows.clone()
        self.stream = torch.cuda.Stream(device=rig.device)
        args = (rig.desc, rig.states[layer], self.tok["q"], self.tok["k"], self.tok["v"], self.tok.get("g"))
        kw = dict(beta=self.tok.get("beta"), u_bonus=rig.bonus[layer], out=rig.out)
        for fn, slots in ((dl.decode_step, self.app_slots), (dl.decode_merge_step, self.mrg_slots)):
            fn(*args, slot_idx=torch.full_like(rows, -1), **kw)     # first launch of the kernel outside any capture
        torch.cuda.synchronize()
        self.append_graph, self.merge_graph = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.stream(self.stream):
            with torch.cuda.graph(self.append_graph, stream=self.stream):
                dl.decode_step(*args, slot_idx=self.app_slots, **kw)
            with torch.cuda.graph(self.merge_graph, stream=self.stream):
                dl.decode_merge_step(*args, slot_idx=self.mrg_slots, **kw)
        torch.cuda.synchronize()

    def step(self, t: int, merge_rows=None):
        """Step ``t`` on ``self.stream``.  Uniform batch: ``merge_rows`` is None and the phase follows from
        ``t`` (every (cap + 1)-th step is the merge step).  Staggered batch: ``merge_rows`` is the boolean
        mask of the rows whose log is full."""
        self.fixed.copy_(self.packed_ring[t % self.rig.RING], non_blocking=True)
        if merge_rows is None:
            (self.merge_graph if t % (self.rig.cap + 1) == self.rig.cap else self.append_graph).replay()
            return
        skip = torch.full_like(self.rows, -1)
        self.app_slots.copy_(torch.where(merge_rows, skip, self.rows))
        self.mrg_slots.copy_(torch.where(merge_rows, self.rows, skip))
        self.append_graph.replay()
        self.merge_graph.replay()


def time_phase_graphs(rig: Rig, steps: int):
    """The paper's cycle on a uniform single-layer batch through ``PhaseGraphs``: one graph replay per step,
    selected by the host's step counter.  Returns (steps timed, total ms)."""
    M = rig.cap + 1
    steps = max(steps // M, 2) * M
    rig.reset_logs()
    pg = PhaseGraphs(rig)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    with torch.cuda.stream(pg.stream):
        for t in range(M):          # one untimed cycle
            pg.step(t)
        start.record()
        for t in range(steps):
            pg.step(t)
        end.record()
    torch.cuda.synchronize()
    return steps, start.elapsed_time(end)


def time_eager_loop(rig: Rig, S: torch.Tensor, steps: int, use_graph: bool = True):
    """The eager dense comparator on the same token ring, launched the same way as the main loop (a
    graph of one trip round the token ring, replayed; the step count is rounded to whole trips, at
    least one).  Returns (steps timed, total ms)."""
    dl = rig.dl

    def launch_steps(n):
        for t in range(n):
            tok = rig.rings[0][t % rig.RING]
            # (the comparator gets the same courtesy as the decode steps: alternating walking directions)
            dl.eager_step(rig.desc_for(down=bool(t & 1)), S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                          u_bonus=rig.bonus[0], out=rig.out)

    steps = max(steps // rig.RING, 2) * rig.RING
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.Stream(device=rig.device)
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
    return steps, start.elapsed_time(end)


def time_e2e(rig: Rig, steps: int, use_graph: bool, clocks, device):
    """The same K steps through the host-buffer entry point: every step copies q, k, v, g, beta from
    pinned host memory and reads the output back to pinned host memory.  Copy-in, kernel and copy-out
    run on three streams over two staging sets (``deltalog_decode_step_host_overlapped``), so the copies
    of step t+1 and t-1 overlap the kernel of step t.  The recurrent state stays resident (it is state,
    not input).  Returns (per-pass ms, h2d bytes per step, d2h bytes per step, how it was launched)."""
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

    def run(n):
        """Steps 0..n-1 from freshly reset logs; merges go to the compute stream."""
        with torch.cuda.stream(streams[1]):
            for t in range(n):
                if rig.staggered:
                    rig.merge(0)   # predicate merge: the rows whose log is full fold before the decode
                tok = host_ring[t % rig.RING]
                staging, lane, host_out = sets[t % 2]
                dl.decode_step_host_overlapped(rig.desc, rig.states[0], staging, lane, tok["q"], tok["k"], tok["v"],
                                               tok["g"], tok["beta"], host_out, u_bonus=rig.bonus[0],
                                               slot_idx=rig.slot_idx)
                if not rig.staggered and (t + 1) % rig.cap == 0:
                    rig.merge(0)

    def join_copy_streams():
        j_in, j_out = torch.cuda.Event(), torch.cuda.Event()
        j_in.record(streams[0])
        j_out.record(streams[2])
        streams[1].wait_event(j_in)
        streams[1].wait_event(j_out)

    def reset():
        for st in streams:
            st.synchronize()
        rig.reset_logs()

    reset()
    run(min(steps, rig.cap))  # warm the copy path
    for st in streams:
        st.synchronize()
    # The serving-loop form: the three-stream pipeline (copies in, kernels, copies out, with their event
    # dependencies) captured into CUDA graphs through the same entry point and replayed, segmented like
    # the device-resident region; the host then only refills the pinned token buffers.
    plan, how = None, "plain calls"
    if use_graph:
        try:
            g_len = graph_steps(rig.cap)
            n_full, tail = segments(steps, g_len)
            plan = []
            for n, reps in ((g_len, n_full), (tail, 1)):
                if not (n and reps):
                    continue
                graph = torch.cuda.CUDAGraph()
                fork = torch.cuda.Event()
                with torch.cuda.graph(graph, stream=streams[1]):
                    fork.record(streams[1])                      # bring the copy streams into the capture
                    streams[0].wait_event(fork)
                    streams[2].wait_event(fork)
                    for _, lane, _ in sets:                      # the lanes' events must belong to the capture
                        lane.in_done.record(streams[0])
                        lane.compute_done.record(streams[1])
                        lane.out_done.record(streams[2])
                    run(n)
                    join_copy_streams()
                plan.append((graph, reps))
            how = (f"CUDA graphs: {n_full} replay(s) of a {g_len}-step graph" + (f" + one {tail}-step graph" if tail else ""))
        except Exception as exc:  # capture not possible here: time the plain calls instead
            print(f"[bench] end-to-end graph capture failed ({type(exc).__name__}: {exc}); timing plain calls", file=sys.stderr)
            plan = None
            torch.cuda.synchronize()

    def enqueue():
        if plan is not None:
            for graph, reps in plan:
                for _ in range(reps):
                    graph.replay()
        else:
            run(steps)
            join_copy_streams()

    times = timed_passes(rig, enqueue, streams[1], clocks, device, reset=reset)
    rig.check_status("end-to-end leg")
    staging = sets[0][0]
    return times, staging.h2d_bytes(rig.desc), staging.d2h_bytes(), how


def cpu_baseline(wl, units: int, steps: int, chunk_units: int = 1024, warmup: int = 0):
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
        if done == 0 and warmup > 0:   # untimed: pages the library in and starts the worker threads
            w = min(warmup, steps)
            oracle.eager_rollout(wl.op, S0, q[:w], k[:w], v[:w], g[:w], beta=beta[:w] if beta is not None else None, bonus=bon)
        t0 = time.perf_counter()
        oracle.eager_rollout(wl.op, S0, q, k, v, g, beta=beta, bonus=bon)
        dt += time.perf_counter() - t0
        done += N
    return {"value": done * steps / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{done} (seq*head) units x {steps} tokens of {wl.name}, fp64 eager recurrence, "
                      f"{dt:.2f} s on {oracle.num_threads()} threads"}, dt


def run_reference(args, wl, config_name):
    """``--impl reference``: the CPU oracle timed on the host cores (rank 0 only; the other ranks leave
    without work)."""
    rank, size, _ = launch.world()
    if rank != 0:
        return
    steps = max(args.steps, 1)
    units = 512 if steps <= 256 else 128   # bounds the fp64 input copies on the host (units x steps)
    small = wl.scaled(layers=1)
    base, dt = cpu_baseline(small, units, steps, warmup=max(args.warmup, 0))
    n_units = max(1, units // wl.H) * wl.H
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": config_name, "sample_units_per_step": n_units,
                   "note": "each step is one token over a bounded sample of the workload's units on the host"},
        "cpu_baseline": {**base},
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def dram_traffic(dl, config: int, cap: int, state: str):
    """ncu DRAM bytes per launch for this configuration, or (None, why) when there is no capture of the
    library build that is being timed."""
    doc = ncu_traffic.load()
    if not doc:
        return None, "no profiles/dram_traffic.json"
    if doc.get("build_id") != dl.build_id():
        return None, f"profiles/dram_traffic.json is of build {doc.get('build_id')}, the library is build {dl.build_id()}"
    cap_rec = doc.get("captures", {}).get(ncu_traffic.capture_key(config, cap, state))
    if not cap_rec:
        return None, "no capture of this configuration and capacity"
    return cap_rec["kernels"], None


def hot_loop_for_profilers(rig: Rig, args):
    """``--only-hot-loop``: warm-up was done; run the steps as plain launches and leave."""
    kind = args.hot_loop_kind
    if kind == "cycle":
        for t in range(args.steps):
            for layer in range(rig.layers):
                rig.step(t, layer)
    elif kind == "eager":
        S = rig.states[0].S_base
        for t in range(args.steps):
            tok = rig.rings[0][t % rig.RING]
            rig.dl.eager_step(rig.desc_for(down=bool(t & 1)), S, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"],
                              u_bonus=rig.bonus[0], out=rig.out)
    else:   # the paper's cycle: cap appends, then the fused merge step
        M = rig.cap + 1
        for t in range(args.steps):
            (rig.fused if t % M == M - 1 else rig.decode)(t, 0)
    torch.cuda.synchronize()
    rig.check_status("hot loop")


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
    ap.add_argument("--layers", type=int, default=0,
                    help="with --only-hot-loop: run this many layers of a multi-layer configuration instead of all "
                         "(a profiler capture of the serving shape that holds a few GB instead of 29)")
    ap.add_argument("--only-hot-loop", action="store_true",
                    help="warm-up and then --steps steps as plain launches, nothing else (for profiler captures)")
    ap.add_argument("--hot-loop-kind", default="cycle", choices=["cycle", "eager", "paper"],
                    help="what --only-hot-loop runs: the decode/merge cycle, the eager kernel, or the paper's cycle")
    args = ap.parse_args()
    if args.steps < 1:
        ap.error("--steps must be at least 1")
    wl = workloads.CONFIGS[args.config]
    config_name = f"configs[{args.config}] {wl.name}"
    if args.impl == "reference":
        return run_reference(args, wl, config_name)

    rank, size, local = launch.init("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    import paper_2608_15533_b200 as dl

    cap, K = args.cap, args.steps
    warmup = max(args.warmup, 3)
    layers = wl.layers
    if args.layers:
        assert args.only_hot_loop and 1 <= args.layers <= wl.layers, "--layers goes with --only-hot-loop"
        layers = args.layers
    base16 = args.state == "bf16"
    # weak scaling: the global batch is `size` times the configuration's rows, sharded by rows
    first_row, n_rows = launch.shard_rows(size * wl.batch, size, rank)
    assert n_rows == wl.batch
    rig = Rig(wl, cap, device, seed_offset=first_row // wl.batch, layers=layers, base16=base16)
    stag = rig.staggered
    u = unit_shape(wl, base16=base16)
    units = wl.units

    # ---- warm-up --------------------------------------------------------------------------------
    rig.reset_logs()
    for t in range(warmup):
        for layer in range(layers):
            rig.step(t, layer)
    torch.cuda.synchronize()
    rig.check_status("warm-up")
    if args.only_hot_loop:
        rig.reset_logs()
        hot_loop_for_profilers(rig, args)
        return launch.finalize()

    # ---- the timed region: exactly K steps from empty logs, repeated, median ---------------------
    use_graph = not args.no_graph
    with ClockSampler(local) as clocks:
        region = Region(rig, K, use_graph)
        times = timed_passes(rig, region.enqueue, region.stream, clocks, device)
        rig.check_status("timed region")
        # the same steps as plain launches with events between the kernels: decode and merge time apart
        clocks.busy = True
        dec_ms, mrg_ms, plain_ms_per_step = time_kernel_split(rig, K)
        merge_note = "merges of the timed region"
        if mrg_ms is None:   # K < cap: the region holds no merge; time one on its own for the amortised figures
            mrg_ms, merge_note = time_merge_alone(rig), "no merge falls into the timed region; a merge of full logs timed on its own"
        clocks.busy = False
        rig.check_status("per-kernel pass")
        # ---- end-to-end leg: token tensors from pinned host memory, output back to the host ----------
        e2e_times, h2d, d2h, e2e_how = time_e2e(rig, K, use_graph, clocks, device)
    total_ms = statistics.median(times)
    all_units = launch.sum_over_ranks(units * layers, device)
    ms_per_step = total_ms / K
    value = all_units * K / (total_ms * 1e-3)
    n_merges = (K * layers) if stag else merges_in(K, cap) * layers

    cyc = traffic.cycle_bytes(u, cap)
    peak, peak_kind = measured_peak_gbs()
    if stag:   # fills uniform on 0..cap-1 across the rows at every step
        dec_bytes = statistics.mean(traffic.decode_read(u, f) + traffic.decode_write(u) for f in range(cap)) * units
    else:
        dec_bytes = statistics.mean(traffic.decode_read(u, t % cap) + traffic.decode_write(u) for t in range(K)) * units
    algo_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    kernels, why_not = dram_traffic(dl, args.config, cap, args.state)
    dec_traffic = mrg_traffic = None
    if kernels and "decode" in kernels:
        dec_traffic = kernels["decode"]["dram_read_bytes_per_launch"] + kernels["decode"]["dram_write_bytes_per_launch"]
    if kernels and "merge" in kernels:
        mrg_traffic = kernels["merge"]["dram_read_bytes_per_launch"] + kernels["merge"]["dram_write_bytes_per_launch"]
    dram_gbs = dec_traffic / (dec_ms * 1e-3) / 1e9 if dec_traffic else None
    achieved = dram_gbs if dram_gbs is not None else algo_gbs
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": size, "steps": K, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": config_name, "op": workloads.OP_NAMES[wl.op], "batch": wl.batch,
            "H": wl.H, "d_k": wl.d, "d_v": wl.d, "layers": layers, "log_capacity": cap, "state": args.state,
            "io": str(wl.io_dtype).replace("torch.", ""),
            "merge": ("before every step the rows whose log is full (listed by the host from its step counters) are folded; fills staggered over 0..cap-1"
                      + ("; the merges run on a side stream, overlapped with other layers' decode steps" if rig.overlap_merges and use_graph else "") if stag
                      else f"after every {cap}th step"),
            "merges_in_timed_region": n_merges,
            "timed_region": f"exactly {K} steps from empty logs; repeated {len(times)} times (logs emptied in between, untimed), median reported",
            "timed_region_ms_all": [round(x, 4) for x in times],
            "launch": region.describe,
            "l2": f"inputs larger than L2: {units * u.state * layers / 2**20:.0f} MiB of base state per step, no flush",
            "parallelism": f"global batch of {size * wl.batch} rows sharded by rows over {size} GPU(s), no collective",
        },
        "clocks": clocks.summary(),
        "gpu_launches": region.launches,
        "roofline": {
            "bound": "hbm", "kernel": "decode_pipelined_kernel" if wl.d == 128 else "decode_append_kernel",
            "achieved": achieved, "achieved_kind": "dram bytes (ncu) / launch time" if dram_gbs is not None else "algorithmic bytes / launch time (no ncu capture of this build)",
            "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
            "traffic": dec_traffic, "traffic_unavailable": why_not,
            "traffic_note": ("dram__bytes_read.sum + dram__bytes_write.sum per launch, mean over the launches of a cycle, ncu "
                             "--cache-control none (L2 as the previous launch left it, as in the timed loop): base tiles are "
                             "read evict-first and the live log is kept in L2, so DRAM traffic is below the algorithmic bytes"),
            "algorithmic_bytes_per_launch": dec_bytes, "avg_launch_ms": dec_ms,
            "achieved_algorithmic_incl_l2": algo_gbs, "frac_algorithmic_incl_l2": algo_gbs / peak,
            "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
        },
    }
    # amortised over a whole cycle from the per-kernel times: cap decode launches + one merge
    if stag:
        cycle_ms_per_step = (dec_ms + mrg_ms) * layers
    else:
        cycle_ms_per_step = dec_ms + mrg_ms / cap
    am = {
        "algorithmic_bytes_per_unit_step": cyc["total"],
        "algorithmic_gbs_incl_l2": cyc["total"] * units * layers / (cycle_ms_per_step * 1e-3) / 1e9,
        "bytes_written_per_unit_step": cyc["write"], "write_reduction_vs_eager": cyc["write_reduction"],
        "decode_ms_per_launch": dec_ms, "merge_ms_per_launch": mrg_ms, "merge_time_from": merge_note,
        "cycle_ms_per_step_from_kernel_times": cycle_ms_per_step, "plain_launch_ms_per_step": plain_ms_per_step,
    }
    am["algorithmic_frac_of_nominal_8TBs"] = am["algorithmic_gbs_incl_l2"] / NOMINAL_HBM_GBS
    am["algorithmic_frac_of_measured"] = am["algorithmic_gbs_incl_l2"] / peak
    if dec_traffic and mrg_traffic and not stag:
        per_step = dec_traffic + mrg_traffic / cap
        am["dram_bytes_per_unit_step"] = per_step / units
        am["dram_gbs"] = per_step / (cycle_ms_per_step * 1e-3) / 1e9
        am["dram_frac_of_measured"] = am["dram_gbs"] / peak
        am["dram_frac_of_nominal_8TBs"] = am["dram_gbs"] / NOMINAL_HBM_GBS
        am["dram_bytes_written_per_unit_step"] = (kernels["decode"]["dram_write_bytes_per_launch"]
                                                  + kernels["merge"]["dram_write_bytes_per_launch"] / cap) / units
        if "eager" in kernels:
            am["dram_bytes_written_per_unit_step_eager"] = kernels["eager"]["dram_write_bytes_per_launch"] / units
            am["dram_write_reduction_vs_eager"] = (am["dram_bytes_written_per_unit_step_eager"]
                                                   / am["dram_bytes_written_per_unit_step"])
    line["amortized"] = am

    e2e_ms = statistics.median(e2e_times)
    e2e_units = launch.sum_over_ranks(units, device)
    line["e2e"] = {"value": e2e_units * K / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / K, "launch": e2e_how, "repeats": len(e2e_times),
                   "note": "state stays resident; q,k,v,g,beta in and out back every step, layer 0"}

    if not args.no_extras and rank == 0:
        # eager dense comparator on the same inputs
        rig.reset_logs()
        S = rig.states[0].S_base
        e_steps, e_total = time_eager_loop(rig, S, K, use_graph)
        eager_ms = e_total / e_steps
        eager_bytes = (traffic.eager_read(u) + traffic.eager_write(u)) * units
        line["eager_kernel"] = {"ms_per_step": eager_ms, "value": units / (eager_ms * 1e-3), "steps": e_steps,
                                "algorithmic_gbs": eager_bytes / (eager_ms * 1e-3) / 1e9,
                                "bytes_written_per_unit_step": traffic.eager_write(u)}
        line["speedup_vs_eager_kernel"] = eager_ms / (cycle_ms_per_step / layers)
        # the paper's own cycle: cap appends + one fused merge step (cap + 1 tokens per dense write)
        p_steps, p_ms, fused_ms = time_paper_cycle(rig, K)
        pc = traffic.paper_cycle_bytes(u, cap + 1)
        p_step_ms = p_ms / p_steps
        line["paper_cycle"] = {
            "ms_per_step": p_step_ms, "value": units * layers * p_steps / (p_ms * 1e-3), "steps": p_steps,
            "merge_interval_M": cap + 1, "algorithmic_bytes_per_unit_step": pc["total"],
            "algorithmic_gbs_incl_l2": pc["total"] * units * layers / (p_step_ms * 1e-3) / 1e9,
            "launch": ("two launches per layer-step over phase-split batches" if stag else "one launch per step"),
            "speedup_vs_eager_kernel": eager_ms / (p_step_ms / layers)}
        if fused_ms is not None:
            fused_bytes = (traffic.fused_read(u, cap) + traffic.fused_write(u)) * units
            line["paper_cycle"]["fused_step_ms"] = fused_ms
            line["paper_cycle"]["fused_step_algorithmic_gbs"] = fused_bytes / (fused_ms * 1e-3) / 1e9
        if not stag and layers == 1:   # the same cycle as two phase-specialised graphs, one replay per step
            g_steps, g_ms = time_phase_graphs(rig, K)
            line["paper_cycle"]["phase_graphs"] = {
                "ms_per_step": g_ms / g_steps, "steps": g_steps,
                "launch": "an append graph and a merge graph over fixed buffers; per step one token copy and one replay, chosen by the host's step counter"}
        rig.check_status("paper cycle")
        # capacity sweep: whole cycles (at least 32 steps' worth), write reduction per capacity
        sweep = {}
        for c in ([cap] if cap in wl.caps else []) + [c for c in wl.caps if c != cap]:   # the rig at hand first
            if layers > 1:
                continue
            cc = traffic.cycle_bytes(u, c)
            n = max(K // graph_steps(c), max(1, 32 // graph_steps(c))) * graph_steps(c)   # whole graphs
            if c == cap and n == K:
                ms = ms_per_step
            else:
                if c != cap:
                    del rig
                    torch.cuda.empty_cache()
                    rig = Rig(wl, c, device, seed_offset=first_row // wl.batch, base16=base16)
                    for t in range(max(c, 3)):
                        rig.step(t)
                sweep_region = Region(rig, n, use_graph)
                ms = statistics.median(timed_passes(rig, sweep_region.enqueue, sweep_region.stream, None, device)) / n
                rig.check_status(f"capacity sweep, cap {c}")
            sweep[str(c)] = {"ms_per_step": ms, "value": units / (ms * 1e-3),
                             "bytes_written_per_unit_step": cc["write"],
                             "write_reduction_vs_eager": cc["write_reduction"],
                             "algorithmic_gbs_incl_l2": cc["total"] * units / (ms * 1e-3) / 1e9}
        if sweep:
            line["capacity_sweep"] = sweep
            line["capacity_sweep_note"] = "whole cycles per capacity (steps rounded to whole graphs); bytes from the byte model"
        small = wl.scaled(layers=1)
        line["cpu_baseline"], _ = cpu_baseline(small, min(wl.units, 4096), 128)
    if rank == 0:
        print(json.dumps(line))
    launch.finalize()


if __name__ == "__main__":
    main()
