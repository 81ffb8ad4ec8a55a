"""The optional tensor-core merge (tcgen05, tf32 x 3 with an fp32 accumulator in tensor memory) is
chosen by an environment variable that the library reads once per process, so its parity tests run
the ordinary parity tests in a child process with the variable set."""
import os
import subprocess
import sys
from pathlib import Path

import pytest

pytestmark = pytest.mark.gpu
ROOT = Path(__file__).resolve().parent.parent


def test_parity_suite_with_the_tensor_core_merge():
    env = dict(os.environ, DELTALOG_MERGE_TC="1")
    sel = "test_small_rollout_invariant_every_step or test_predicate_merge_at_capacity_64 or test_cap1_equals_eager"
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-k", sel,
                        str(ROOT / "tests" / "test_gpu_parity.py"), str(ROOT / "tests" / "test_gpu_additive_ops.py")],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout


def test_tensor_core_merge_is_the_kernel_that_ran():
    """The child decodes 16 tokens and merges at head size 128; the launch goes to merge_tc_kernel only if
    the variable is honoured: a state folded on the tensor cores differs in the last bits from one
    folded on the fp32 pipe, while both stay within the parity bar of each other."""
    code = r'''
import sys, torch
sys.path.insert(0, "tests")
import workloads, paper_2608_15533_b200 as dl
from harness import make_desc
wl = workloads.Workload("tc", workloads.KDA, 4, 2, 128, 16, (16,))
src = workloads.TokenSource(wl, device="cpu")
S0 = src.initial_state().cuda()
desc = make_desc(wl, 16, 1.0)
state = dl.State(desc, S0.clone())
for t in range(16):
    tok = {k: (v.cuda() if v is not None else None) for k, v in src.token().items()}
    dl.decode_step(desc, state, tok["q"], tok["k"], tok["v"], tok["g"], beta=tok["beta"])
dl.merge(desc, state)
torch.cuda.synchronize()
assert int(state.status.item()) == 0 and int(state.log_len.abs().sum()) == 0
torch.save(state.S_base.cpu(), sys.argv[1])
'''
    import tempfile

    import torch

    outs = []
    with tempfile.TemporaryDirectory() as tmp:
        for flag in ("0", "1"):
            path = os.path.join(tmp, f"s{flag}.pt")
            subprocess.run([sys.executable, "-c", code, path], env=dict(os.environ, DELTALOG_MERGE_TC=flag), cwd=ROOT,
                           check=True, timeout=600)
            outs.append(torch.load(path))
    a, b = outs
    assert not torch.equal(a, b)
    assert float((a - b).abs().max() / a.abs().max()) <= 1e-5
