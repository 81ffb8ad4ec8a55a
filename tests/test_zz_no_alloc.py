"""The allocation-free host-buffer decode step (``deltalog_decode_step_host_static``).

This file sorts last on purpose: if it fails, a run that stops at the first failure has already
been through every other test.  The entry point exists for callers that cannot hand the library
device staging buffers because they are not allowed to allocate device memory (a serving loop
that must never trigger an allocation, a plug-in that is given a stream but no allocator); its
staging area is a fixed array inside the library, shared by all calls on a device.  The test
calls it through the C ABI twice in a row -- the second call finds the first call's leftovers in
the array -- and checks both results against the existing ``deltalog_decode_step_host``.
"""
import ctypes

import pytest
import torch

import workloads
from harness import make_desc
from workloads import GDN, KDA, RWKV6, Workload


def test_requests_beyond_the_built_in_area_are_rejected_on_the_host():
    import paper_2608_15533_b200 as dl
    from paper_2608_15533_b200 import binding

    lib = dl.load_library()
    # bf16, H = 32, d = 128, GDN: 257 rows need a little more than 8 MiB of staging -> rejected before
    # any CUDA call is made (the pointers below are never dereferenced)
    desc = dl.Desc(op=dl.GDN, num_slots=512, H=32, d_k=128, d_v=128, cap=8).c_struct()
    st = binding._State(*(0x1000 * (i + 1) for i in range(6)))
    fake = [0x10000 * (i + 1) for i in range(5)]
    rc = lib.deltalog_decode_step_host_static(ctypes.byref(desc), ctypes.byref(st), *fake, None, None, 263,
                                              0x90000, None)
    assert rc == binding.ERR_STATIC_LIMIT
    assert "staging" in dl.status_string(rc)
    # the limit is sharp: 254 rows fit (checked on the GPU below), 255 do not
    assert lib.deltalog_decode_step_host_static(ctypes.byref(desc), ctypes.byref(st), *fake, None, None, 255,
                                                0x90000, None) == binding.ERR_STATIC_LIMIT
    # grouped heads stage fewer query / key rows: with 8 query/key heads 300 rows fit, so the request is judged
    # on its other arguments (here: a state pointer that is not 16-byte aligned)
    grouped = dl.Desc(op=dl.GDN, num_slots=512, H=32, d_k=128, d_v=128, cap=8, H_qk=8).c_struct()
    bad_state = binding._State(0x1008, *(0x1000 * (i + 2) for i in range(5)))
    assert lib.deltalog_decode_step_host_static(ctypes.byref(grouped), ctypes.byref(bad_state), *fake, None, None, 300,
                                                0x90000, None) == binding.ERR_INVALID_ARG
    assert lib.deltalog_decode_step_host_static(ctypes.byref(desc), ctypes.byref(bad_state), *fake, None, None, 300,
                                                0x90000, None) == binding.ERR_STATIC_LIMIT
    assert lib.deltalog_decode_step_host_static(ctypes.byref(desc), ctypes.byref(st), *fake, None, None, -1,
                                                0x90000, None) == binding.ERR_INVALID_ARG
    assert lib.deltalog_decode_step_host_static(None, ctypes.byref(st), *fake, None, None, 1, 0x90000, None) == \
        binding.ERR_INVALID_ARG


@pytest.mark.gpu
@pytest.mark.parametrize("op,d,io", [(GDN, 128, torch.bfloat16), (KDA, 64, torch.float32), (RWKV6, 64, torch.bfloat16)])
def test_static_staging_matches_the_caller_staged_entry_point_on_two_calls_in_a_row(op, d, io):
    import paper_2608_15533_b200 as dl

    dev = "cuda"
    wl = Workload("noalloc", op, 6, 3, d, 4, (4,), io_dtype=io, num_slots=9)
    src = workloads.TokenSource(wl)
    S0 = src.initial_state().to(dev)
    bonus = src.bonus()
    bonus = bonus.to(dev) if bonus is not None else None
    desc = make_desc(wl, 4)
    slot_idx = workloads.slot_permutation(wl, pad_every=4).to(dev)        # rows 0 and 4 are padding
    ref_state, new_state = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    staging = dl.HostStaging(desc, wl.batch, dev)
    staging.out.zero_()                                                    # the reference staging starts clean
    for call in range(2):                                                  # the second call reuses a dirty array
        tok = {k: (v.pin_memory() if v is not None else None) for k, v in src.token().items()}
        out_ref = torch.full((wl.batch, wl.H, wl.d), 3.0, dtype=io).pin_memory()
        out_new = torch.full((wl.batch, wl.H, wl.d), 5.0, dtype=io).pin_memory()
        dl.decode_step_host(desc, ref_state, staging, tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"],
                            out_ref, u_bonus=bonus, slot_idx=slot_idx)
        dl.decode_step_host_static(desc, new_state, tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"],
                                   out_new, u_bonus=bonus, slot_idx=slot_idx)
        torch.cuda.synchronize()
        live = (slot_idx >= 0).cpu()
        assert torch.equal(out_new[live], out_ref[live]), f"call {call}"   # same kernel, same inputs: bit-identical
        assert bool((out_new[~live] == 0).all())                           # skipped rows read back as zeros
    for a, b in ((ref_state.K_log, new_state.K_log), (ref_state.U_log, new_state.U_log),
                 (ref_state.decay_log, new_state.decay_log), (ref_state.log_len, new_state.log_len)):
        assert torch.equal(a, b)
    assert int(new_state.status.item()) == 0
    assert int(new_state.log_len.max()) == 2


@pytest.mark.gpu
def test_a_request_that_fills_the_built_in_area_to_the_last_block():
    """254 rows of the benchmark shape (bf16, 32 heads, head size 128) use 8 388 096 of the 8 388 608
    bytes: the output region is the last carve-out and ends 512 bytes below the top of the array."""
    import paper_2608_15533_b200 as dl

    dev = "cuda"
    wl = Workload("noalloc_limit", GDN, 254, 32, 128, 2, (4,))
    src = workloads.TokenSource(wl, device=dev)
    S0 = src.initial_state()
    desc = make_desc(wl, 4)
    ref_state, new_state = dl.State(desc, S0.clone()), dl.State(desc, S0.clone())
    staging = dl.HostStaging(desc, wl.batch, dev)
    for call in range(2):
        tok = {k: (v.cpu().pin_memory() if v is not None else None) for k, v in src.token().items()}
        out_ref = torch.zeros(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory()
        out_new = torch.ones(wl.batch, wl.H, wl.d, dtype=wl.io_dtype).pin_memory()
        dl.decode_step_host(desc, ref_state, staging, tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], out_ref)
        dl.decode_step_host_static(desc, new_state, tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], out_new)
        torch.cuda.synchronize()
        assert torch.equal(out_new, out_ref), f"call {call}"
        assert bool(out_new[-1].float().abs().sum() > 0)            # the last row, at the top of the array, was produced
    assert torch.equal(ref_state.U_log, new_state.U_log) and torch.equal(ref_state.log_len, new_state.log_len)
    assert int(new_state.status.item()) == 0 and int(new_state.log_len.min()) == 2
