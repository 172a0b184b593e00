"""fsm_index_build_static: the index build for callers that cannot allocate
device memory (a plug-in whose host application owns the whole device through
its own pool, a serving loop where cudaMalloc is off limits).  It must give the
same index as fsm_index_build, call after call, while all calls share one
built-in scratch array that still holds the previous call's leftovers.

Collected last on purpose (file name), so a stop-at-first-failure run has
already exercised everything else."""
import numpy as np
import pytest
import torch

from fsm_inputs import make_config

pytestmark = pytest.mark.gpu


def _build_both(fg, w, state_dtype):
    d = w.dfa
    ref = fg.GuidedIndex(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                         state_dtype).build()
    mask = torch.full_like(ref.allowed_mask, 0x55555555)
    nxt = torch.zeros_like(ref.next_state)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rc = fg.fsm_index_build_static(ref.trans, ref.accept, ref.vocab_bytes, ref.vocab_offsets,
                                   ref.vocab_nbytes, ref.Q, ref.N, ref.dead_state, ref.eos_id,
                                   mask, nxt, state_dtype, status)
    assert rc == 0, fg.fsm_status_string(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and int(ref.status.item()) == 0
    assert torch.equal(mask, ref.allowed_mask)                     # bit-exact, as in the parity tests
    assert torch.equal(nxt.view(torch.uint8), ref.next_state.view(torch.uint8))
    return int(ref.allowed_mask.ne(0).sum().item())


def test_static_scratch_build_matches_workspace_build_twice_in_a_row():
    import paper_2307_09702_b200 as fg
    w2, w1 = make_config(2), make_config(1)
    # two different problems back to back: the second sees the first one's leftovers
    assert _build_both(fg, w2, fg.FSM_STATE_I32) > 0
    assert _build_both(fg, w1, fg.FSM_STATE_U16) > 0
    assert _build_both(fg, w2, fg.FSM_STATE_U16) > 0


def test_static_scratch_build_refuses_problems_beyond_its_array():
    import paper_2307_09702_b200 as fg
    w = make_config(3)
    rc = fg.fsm_index_build_static(0x1000, 0x2000, 0x3000, 0x4000, int(w.vocab_offsets[-1]), w.Q, w.N,
                                   w.dfa.dead, w.eos_id, 0x5000, 0x6000, 0, None)
    assert rc == -5 and "WORKSPACE" in fg.fsm_status_string(rc)
