"""Chained decode launches (DELTALOG_HINT_BASE_UNTOUCHED / DELTALOG_HINT_SLOTS_STABLE) when the
launch directly in front of a decode step is the one that PRODUCES that step's inputs, as in a model
(the gate and beta projections run right before the recurrent update).

With the hint the decode kernel may start while that producer is still running; it may then read
base tiles (and, under the second hint, the slot list) early, but nothing the producer writes.  The
producer here is an elementwise kernel that fills the step's q, k, v, g, beta -- and in one variant
slot_idx as well -- from a staging copy; before it, an earlier launch overwrites the buffers with
poison (NaN bit patterns; slot -1), so a read ahead of the producer would change the result.
Results must be bit-identical to unchained launches over 48 steps of 40 x 8 units."""
import pytest
import torch

import workloads
from harness import make_desc
from workloads import GDN, KDA, RWKV6, Workload

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAMES = ("q", "k", "v", "g", "beta", "slots")


def pack(tensors):
    """The given tensors as int32 words in one block, each starting on a 256-byte boundary."""
    words, spans, off = [], {}, 0
    for name, t in tensors.items():
        w = t.contiguous().reshape(-1).view(torch.uint8)
        pad = (-w.numel()) % 256
        w = torch.cat([w, torch.zeros(pad, dtype=torch.uint8, device=w.device)])
        spans[name] = (off, t.numel() * t.element_size(), t.dtype, t.shape)
        off += w.numel()
        words.append(w)
    return torch.cat(words).view(torch.int32), spans


@pytest.mark.parametrize("op,d", [(GDN, 128), (KDA, 128), (RWKV6, 64), (GDN, 64), (RWKV6, 128)])
@pytest.mark.parametrize("slots_written", [True, False])
def test_inputs_written_by_the_launch_in_front_of_a_chained_step(op, d, slots_written):
    import paper_2608_15533_b200 as dl

    wl = Workload(f"chain_inputs_{op}_{d}", op, 40, 8, d, 48, (16,), num_slots=56)
    cap = 16
    src = workloads.TokenSource(wl, device="cpu")
    S0 = src.initial_state().to(DEV)
    bonus = src.bonus()
    bonus = bonus.to(DEV) if bonus is not None else None
    slots = workloads.slot_permutation(wl, pad_every=9).to(DEV)
    staged = []
    for _ in range(wl.steps):
        tok = {k: v.to(DEV) for k, v in src.token().items() if v is not None}
        if slots_written:
            tok["slots"] = slots
        staged.append(pack(tok))
    spans = staged[0][1]
    results = []
    for hints in (0, dl.HINT_BASE_UNTOUCHED | (0 if slots_written else dl.HINT_SLOTS_STABLE)):
        desc, desc_c = make_desc(wl, cap), make_desc(wl, cap)
        desc_c.hints = hints
        state = dl.State(desc, S0.clone())
        live = torch.empty_like(staged[0][0])      # the step's input buffers, refilled before every step
        view = {n: live.view(torch.uint8)[o:o + nb].view(dt).view(shape) for n, (o, nb, dt, shape) in spans.items()}
        slot_arg = view["slots"] if slots_written else slots
        outs = [torch.empty(wl.batch, wl.H, wl.d, dtype=wl.io_dtype, device=DEV) for _ in range(wl.steps)]
        torch.cuda.synchronize()
        for t in range(wl.steps):
            first = t % cap == 0
            if first and t:
                dl.merge(desc, state, slot_idx=slots, n=wl.batch)
            live.fill_(-1)                                  # poison: NaN patterns, slot -1
            torch.add(staged[t][0], 0, out=live)            # the producer: a kernel, directly in front of the step
            dl.decode_step(desc if first else desc_c, state, view["q"], view["k"], view["v"], view.get("g"),
                           beta=view.get("beta"), u_bonus=bonus, slot_idx=slot_arg, out=outs[t])
        dl.merge(desc, state, slot_idx=slots, n=wl.batch)
        torch.cuda.synchronize()
        assert int(state.status.item()) == 0
        results.append((torch.stack(outs), state.S_base.clone(), state.log_len.clone(), state.U_log.clone()))
    keep = slots >= 0
    assert torch.equal(results[0][0][:, keep], results[1][0][:, keep])
    for a, b in zip(results[0][1:], results[1][1:]):
        assert torch.equal(a, b)
    assert not torch.isnan(results[1][0][:, keep].float()).any()
