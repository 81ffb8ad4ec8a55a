"""The give-up path of the bounded waits inside the persistent decode kernel and the resident fused-step kernel.

Every wait on an mbarrier in that kernel is bounded in time; when one runs out, the CTA raises its
abort flag, all roles leave their loops, copies still in flight are waited for (again bounded) and
DELTALOG_STATUS_TIMEOUT is OR-ed into the status word -- the launch returns instead of hanging.
This path cannot be reached with correct inputs, so a second build of the same sources is used
(``libdeltalog_testhooks.so``: waits give up after 5 ms, and the launcher passes on the index of one
unit whose first base chunk the producer never requests).  Nothing here traps, faults or waits
without a bound: the stream group simply waits 5 ms for a chunk that was never asked for.  The test
runs in a child process so that the rest of the suite keeps using the regular library."""
import subprocess
import sys
import textwrap
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r}); sys.path.insert(0, {root!r} + "/tests")
    import numpy as np, torch
    from paper_2608_15533_b200 import binding, build
    binding.LIB_PATH = build.build_test_hooks_library()
    import paper_2608_15533_b200 as dl
    import workloads
    from harness import f64, make_desc, rel_err
    import oracle

    dev = "cuda"
    wl = workloads.Workload("wait_timeout", workloads.GDN, 40, 8, 128, 4, (16,))    # 320 units: 2-3 per persistent CTA
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(dev)
    toks = [{{k: (v.to(dev) if v is not None else None) for k, v in src.token().items()}} for _ in range(3)]
    desc = make_desc(wl, 16)

    # 1. one unit's first chunk is never requested: the launch must come back with the TIMEOUT bit and no other
    os.environ["DELTALOG_TEST_DROP_ITEM"] = str(148 + 17)          # the second unit of CTA 17
    state = dl.State(desc, S0.clone())
    t = toks[0]
    dl.decode_step(desc, state, t["q"], t["k"], t["v"], t["g"], beta=t["beta"])
    torch.cuda.synchronize()                                        # returns: nothing hangs
    assert int(state.status.item()) == dl.STATUS_TIMEOUT, int(state.status.item())
    assert bool((state.S_base == S0).all())                         # the base is never written by a decode step

    # 2. the context is intact: a normal rollout on a fresh state afterwards meets the parity bar
    os.environ["DELTALOG_TEST_DROP_ITEM"] = "-1"
    state = dl.State(desc, S0.clone())
    outs = [dl.decode_step(desc, state, t["q"], t["k"], t["v"], t["g"], beta=t["beta"]) for t in toks]
    dl.merge(desc, state)
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    N = wl.batch * wl.H
    flat = lambda key: np.stack([f64(t[key]).reshape(N, -1) for t in toks])
    ref = oracle.eager_rollout(wl.op, f64(S0).reshape(N, wl.d, wl.d), flat("q"), flat("k"), flat("v"), flat("g"),
                               beta=flat("beta")[..., 0])
    assert rel_err(np.stack([f64(o).reshape(N, -1) for o in outs]), ref["out"]) <= 2e-2
    assert rel_err(f64(state.S_base).reshape(N, wl.d, wl.d), ref["S"]) <= 1e-4
    print("wait-timeout path ok")

    # 3. the resident fused-merge-step kernel has one bounded wait (for a unit's tile): the tile of one (row, head)
    # pair is never requested; the launch returns with the TIMEOUT bit alone, and a fresh state afterwards is fine
    os.environ["DELTALOG_TEST_DROP_ITEM"] = str(296 + 3)            # one (row, head) pair of the 320
    state = dl.State(desc, S0.clone())
    t = toks[0]
    dl.decode_merge_step(desc, state, t["q"], t["k"], t["v"], t["g"], beta=t["beta"])
    torch.cuda.synchronize()
    assert int(state.status.item()) == dl.STATUS_TIMEOUT, int(state.status.item())
    os.environ["DELTALOG_TEST_DROP_ITEM"] = "-1"
    state = dl.State(desc, S0.clone())
    outs = [dl.decode_merge_step(desc, state, t["q"], t["k"], t["v"], t["g"], beta=t["beta"]) for t in toks]
    torch.cuda.synchronize()
    assert int(state.status.item()) == 0
    assert rel_err(np.stack([f64(o).reshape(N, -1) for o in outs]), ref["out"]) <= 2e-2
    assert rel_err(f64(state.S_base).reshape(N, wl.d, wl.d), ref["S"]) <= 1e-4
    print("fused-step wait-timeout path ok")
""")


def test_a_wait_that_runs_out_ends_the_launch_with_the_timeout_bit_and_leaves_the_context_usable():
    proc = subprocess.run([sys.executable, "-c", CHILD.format(root=str(ROOT))], capture_output=True, text=True, timeout=900)
    assert proc.returncode == 0, proc.stdout[-2000:] + proc.stderr[-3000:]
    assert "wait-timeout path ok" in proc.stdout
    assert "fused-step wait-timeout path ok" in proc.stdout
