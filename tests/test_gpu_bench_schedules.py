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
        rig.reset_logs()
        if use_graph:
            bench.time_graph_loop(rig, 2 * bench.graph_steps(cap))
        else:
            for t in range(3 * bench.graph_steps(cap)):     # time_graph_loop replays once to warm up
                rig.step(t)
        assert all(s == 0 for s in rig.status())
        return state_snapshot(rig)

    ref = run(False, False)
    assert same(ref, run(True, False)) and same(ref, run(True, True))
