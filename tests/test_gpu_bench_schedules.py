"""The launch schedules bench.py times must compute what the plain sequential schedule computes:
chained decode launches, CUDA-graph replays, and -- for several layers with staggered fills -- the
token-less merges on a side stream, overlapped with other layers' decode steps."""
import pytest
import torch

import bench
import workloads
from workloads import GDN, Workload

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def state_snapshot(rig):
    torch.cuda.synchronize()
    return [(s.S_base.clone(), s.K_log.clone(), s.U_log.clone(), s.decay_log.clone(), s.log_len.clone())
            for s in rig.states]


def same(a, b):
    return all(torch.equal(x, y) for sa, sb in zip(a, b) for x, y in zip(sa, sb))


def test_side_stream_merges_equal_the_sequential_schedule():
    wl = Workload("sched_stag", GDN, 48, 4, 128, 32, (4,), layers=3, staggered=True)
    cap, n_steps = 4, 16

    def run(overlap):
        rig = bench.Rig(wl, cap, DEV, layers=wl.layers)
        rig.overlap_merges = overlap
        rig.reset_logs()
        stream = torch.cuda.Stream(device=DEV)
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                if overlap:
                    bench.capture_steps_with_merges_on_a_side_stream(rig, n_steps, stream)
                else:
                    for t in range(n_steps):
                        for layer in range(rig.layers):
                            rig.step(t, layer)
            graph.replay()
            graph.replay()
        assert all(s == 0 for s in rig.status())
        return state_snapshot(rig), rig.out.clone()

    (seq, out_seq), (ovl, out_ovl) = run(False), run(True)
    assert same(seq, ovl) and torch.equal(out_seq, out_ovl)
    assert int(seq[0][4].max()) > 0          # logs are in use: the comparison is not vacuous


def test_chained_graph_replays_equal_plain_launches():
    wl = Workload("sched_uniform", GDN, 64, 8, 128, 32, (16,))
    cap = 16

    def run(chain, use_graph):
        rig = bench.Rig(wl, cap, DEV)
        rig.chain = chain
        steps = 2 * bench.graph_steps(cap) + 5               # two replays of the cycle graph and a 5-step tail graph
        region = bench.run_region_once(rig, steps, use_graph)
        assert region.launches == steps + steps // cap
        assert all(s == 0 for s in rig.status())
        assert int(rig.states[0].log_len.min()) == int(rig.states[0].log_len.max()) == 5
        return state_snapshot(rig)

    ref = run(False, False)
    assert same(ref, run(True, False)) and same(ref, run(True, True))


def test_full_size_config1_in_the_timed_launch_configuration_against_the_oracle():
    """Configuration 1 at full size, run exactly as bench.py times it (one CUDA graph per cycle, chained
    decode launches, 256 steps): final state of sampled units against the fp64 oracle."""
    import numpy as np
    import oracle
    from harness import TOL_STATE, f64, rel_err

    wl, cap, steps = workloads.CONFIGS[1], 16, 256
    rig = bench.Rig(wl, cap, DEV)
    units = [(0, 0), (0, 31), (17, 5), (63, 12), (64, 0), (100, 30), (127, 31), (127, 0), (31, 16), (90, 7)]
    ub = torch.tensor([u[0] for u in units], device=DEV)
    uh = torch.tensor([u[1] for u in units], device=DEV)
    rig.reset_logs()
    S0 = f64(rig.states[0].S_base[ub, uh])
    bench.run_region_once(rig, steps, use_graph=True)
    assert all(s == 0 for s in rig.status()) and int(rig.states[0].log_len.abs().sum()) == 0
    ring = rig.rings[0]
    pick = lambda name: np.stack([f64(ring[t % rig.RING][name][ub, uh]).reshape(len(units), -1) for t in range(steps)])
    ref = oracle.eager_rollout(wl.op, S0, pick("q"), pick("k"), pick("v"), pick("g"), beta=pick("beta")[..., 0])
    err = rel_err(f64(rig.states[0].S_base[ub, uh]), ref["S"])
    assert err <= TOL_STATE, f"state error {err:.3e}"
    out_err = rel_err(f64(rig.out[ub, uh]), ref["out"][-1])
    assert out_err <= 2e-2, f"output error {out_err:.3e}"


@pytest.mark.parametrize("staggered", [False, True])
def test_two_phase_specialised_graphs_equal_the_sequential_paper_cycle(staggered):
    """An append graph and a merge graph over fixed buffers, selected (uniform batch) or both replayed over
    phase-split slot lists (staggered fills) by the host, against plain calls of the same cycle:
    bit-identical state, log and outputs at every step."""
    import paper_2608_15533_b200 as dl

    wl = Workload("phase_graphs", GDN, 48, 4, 128, 40, (4,), num_slots=64 if staggered else None, staggered=staggered)
    cap, M, steps = 4, 5, 23

    def fills(rig):   # staggered: row b starts `delay` steps late, so the rows' logs fill at different steps
        return workloads.fill_offsets(wl, M).to(DEV) if staggered else torch.zeros(wl.batch, dtype=torch.long, device=DEV)

    def run(use_graphs):
        rig = bench.Rig(wl, cap, DEV)
        rig.out.zero_()                                   # rows that sit out of a step are never written
        delay = fills(rig)
        rows = rig.slot_idx if rig.slot_idx is not None else torch.arange(wl.batch, dtype=torch.int32, device=DEV)
        skip = torch.full_like(rows, -1)
        pg = bench.PhaseGraphs(rig) if use_graphs else None
        outs = []
        stream = pg.stream if pg else torch.cuda.current_stream()
        with torch.cuda.stream(stream):
            for t in range(steps):
                age = t - delay                                  # steps a row has taken part in
                active = age >= 0
                full = active & (age % M == cap)                 # its log holds cap entries: merge phase
                tok = rig.rings[0][t % rig.RING]
                if use_graphs:
                    if staggered:
                        pg.rows = torch.where(active, rows, skip)
                        pg.step(t, merge_rows=full)
                    else:
                        pg.step(t)
                else:
                    args = (rig.desc, rig.states[0], tok["q"], tok["k"], tok["v"], tok["g"])
                    dl.decode_step(*args, beta=tok["beta"], slot_idx=torch.where(active & ~full, rows, skip), out=rig.out)
                    dl.decode_merge_step(*args, beta=tok["beta"], slot_idx=torch.where(full, rows, skip), out=rig.out)
                outs.append(rig.out.clone())
        torch.cuda.synchronize()
        assert all(s == 0 for s in rig.status())
        return state_snapshot(rig), torch.stack(outs)

    (ref, out_ref), (got, out_got) = run(False), run(True)
    assert same(ref, got) and torch.equal(out_ref, out_got)
    assert int(ref[0][4].max()) > 0                                  # logs are in use at the end
