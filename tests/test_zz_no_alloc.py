"""fsm_index_build_static: the index build for callers that cannot allocate
device memory (a plug-in whose host application owns the whole device through
its own pool, a serving loop where cudaMalloc is off limits).  It must give the
index the CPU oracle gives - and the same one as fsm_index_build - call after
call, while all calls share one built-in scratch array that still holds the
previous call's leftovers.

Collected last on purpose (file name), so a stop-at-first-failure run has
already exercised everything else."""
import numpy as np
import pytest
import torch

from fsm_inputs import bpe_like_vocab, make_config, random_class_dfa
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu


def _static_build(fg, trans, accept, vb, vo, dead, eos, state_dtype):
    """Runs the allocation-free entry point on poisoned outputs; returns host arrays."""
    dev = torch.device("cuda")
    Q, N = trans.shape[0], len(vo) - 1
    t = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a), dtype=dt).to(dev)
    d_trans, d_acc, d_vo = t(trans, torch.int32), t(accept, torch.uint8), t(vo, torch.int32)
    d_vb = t(vb if len(vb) else np.zeros(1, np.uint8), torch.uint8)
    mask = torch.full((Q, (N + 31) // 32), 0x55555555, dtype=torch.int32, device=dev)
    ndt = torch.int32 if state_dtype == fg.FSM_STATE_I32 else torch.uint16
    nxt = torch.empty((Q, N), dtype=ndt, device=dev)
    nxt.view(torch.uint8).fill_(0xEE)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = fg.fsm_index_build_static(d_trans, d_acc, d_vb, d_vo, int(vo[-1]), Q, N, dead, eos, mask, nxt,
                                   state_dtype, status)
    assert rc == 0, fg.fsm_status_string(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    got_next = nxt.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int32) \
        if ndt == torch.uint16 else nxt.cpu().numpy()
    return mask.cpu().numpy().view(np.uint32), got_next


def _check_against_oracle_and_workspace_build(fg, trans, accept, vb, vo, dead, eos, state_dtype):
    threads = max(1, len(__import__("os").sched_getaffinity(0)))
    want_mask, want_next, _ = fsm_oracle.index_build(trans, accept, vb, vo, dead, eos, threads=threads)
    got_mask, got_next = _static_build(fg, trans, accept, vb, vo, dead, eos, state_dtype)
    assert (got_mask == want_mask).all()                      # bit-exact, as in the parity tests
    assert (got_next == want_next).all()
    ref = fg.GuidedIndex(trans, accept, vb, vo, dead, eos, state_dtype).build()
    torch.cuda.synchronize()
    assert (ref.allowed_mask.cpu().numpy().view(np.uint32) == got_mask).all()
    return int((got_mask != 0).sum())


def _largest_vocabulary_that_fits(fg, Q):
    """The entry point checks the sizes against its array before it looks at any pointer, so
    NULL pointers tell whether a size fits (FSM_ERR_NULL) or not (FSM_ERR_WORKSPACE) without
    anything being launched."""
    def fits(N):
        rc = fg.fsm_index_build_static(None, None, None, None, 4 * N, Q, N, Q - 1, -1, None, None, 0, None)
        assert rc in (-1, -5), rc
        return rc == -1
    lo, hi = 1, 4_000_000
    assert fits(lo) and not fits(hi)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        lo, hi = (mid, hi) if fits(mid) else (lo, mid)
    return lo


def test_static_scratch_build_matches_the_oracle_twice_in_a_row():
    import paper_2307_09702_b200 as fg
    w2, w1 = make_config(2), make_config(1)
    # different problems back to back: each sees the leftovers of the one before
    for w, sd in ((w2, fg.FSM_STATE_I32), (w1, fg.FSM_STATE_U16), (w2, fg.FSM_STATE_U16)):
        d = w.dfa
        assert _check_against_oracle_and_workspace_build(fg, d.trans, d.accept, w.vocab_bytes,
                                                         w.vocab_offsets, d.dead, w.eos_id, sd) > 0


def test_static_scratch_build_with_more_states_than_sms():
    """300 states x 5,000 tokens: here the workspace build takes the row-wise walk, the
    allocation-free one the dense walk; both must give the oracle's index."""
    import paper_2307_09702_b200 as fg
    d, _ = random_class_dfa(300, n_live=300, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 5000, zero_length_ids=(4999,))
    for _ in range(2):
        _check_against_oracle_and_workspace_build(fg, d.trans, d.accept, vb, vo, d.dead, 4999,
                                                  fg.FSM_STATE_I32)


def test_static_scratch_build_at_the_edge_of_its_array():
    """The largest vocabulary the array takes for 1,000 states, built twice back to back,
    and one token more, which is refused before anything is launched."""
    import paper_2307_09702_b200 as fg
    Q = 1000
    n_max = _largest_vocabulary_that_fits(fg, Q)
    assert 30_000 < n_max < 120_000
    d, _ = random_class_dfa(41, n_live=Q - 1, n_classes=64, live_classes_per_state=12)
    vb, vo = bpe_like_vocab(43, n_max, zero_length_ids=(n_max - 1,))
    for _ in range(2):
        _check_against_oracle_and_workspace_build(fg, d.trans, d.accept, vb, vo, d.dead, n_max - 1,
                                                  fg.FSM_STATE_U16)
    rc = fg.fsm_index_build_static(0x1000, 0x2000, 0x3000, 0x4000, 4 * (n_max + 1), Q, n_max + 1, Q - 1,
                                   -1, 0x5000, 0x6000, 0, None)
    assert rc == -5 and "WORKSPACE" in fg.fsm_status_string(rc)


def test_static_scratch_build_refuses_problems_beyond_its_array():
    import paper_2307_09702_b200 as fg
    w = make_config(3)
    rc = fg.fsm_index_build_static(0x1000, 0x2000, 0x3000, 0x4000, int(w.vocab_offsets[-1]), w.Q, w.N,
                                   w.dfa.dead, w.eos_id, 0x5000, 0x6000, 0, None)
    assert rc == -5 and "WORKSPACE" in fg.fsm_status_string(rc)
