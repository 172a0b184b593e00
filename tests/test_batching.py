"""Stacked automata (several FSMs indexed by one build): the stacked table's index, row
range by row range, equals each automaton's own index after renumbering.  The CPU part
checks the renumbering against the oracle; the GPU part checks the one-call build."""
import numpy as np
import pytest
import torch

from fsm_inputs import compile_regex, make_config, signed_decimal_dfa
from oracle import fsm_oracle
from paper_2307_09702_b200.batching import local_state_ids, stack_automata

PATTERNS = [r"[0-9]+", r"(ab|cd)*e?", r"\"[a-z ]*\"", r"-?(0|[1-9][0-9]*)(\.[0-9]+)?"]


def _automata():
    ds = [compile_regex(p) for p in PATTERNS] + [signed_decimal_dfa()]
    # one automaton whose dead state is not its last state
    d = ds[1]
    perm = np.arange(d.trans.shape[0])
    perm[[0, d.dead]] = perm[[d.dead, 0]]            # swap state 0 and the dead state
    inv = np.argsort(perm)
    swapped = (inv[d.trans[perm]].astype(np.int32), d.accept[perm], int(inv[d.dead]))
    return [(x.trans, x.accept, x.dead) for x in ds] + [swapped]


def _expected_rows(automata, w, dead_all, offsets):
    rows_mask, rows_next = [], []
    for k, (trans, accept, dead) in enumerate(automata):
        mask, nxt, _ = fsm_oracle.index_build(trans, accept, w.vocab_bytes, w.vocab_offsets, dead, w.eos_id)
        ids = local_state_ids(trans.shape[0], dead, int(offsets[k]), dead_all)
        live = [q for q in range(trans.shape[0]) if q != dead]
        rows_mask.append(mask[live])
        rows_next.append(ids[nxt[live]].astype(np.int32))
    W = rows_mask[0].shape[1]
    rows_mask.append(np.zeros((1, W), np.uint32))
    rows_next.append(np.full((1, rows_next[0].shape[1]), dead_all, np.int32))
    return np.vstack(rows_mask), np.vstack(rows_next)


def test_stacked_table_indexes_like_its_parts():
    w = make_config(1)
    automata = _automata()
    trans, accept, dead_all, offsets = stack_automata(automata)
    assert trans.shape[0] == sum(a[0].shape[0] - 1 for a in automata) + 1
    assert (trans[dead_all] == dead_all).all() and accept[dead_all] == 0
    got_mask, got_next, _ = fsm_oracle.index_build(trans, accept, w.vocab_bytes, w.vocab_offsets,
                                                   dead_all, w.eos_id)
    want_mask, want_next = _expected_rows(automata, w, dead_all, offsets)
    assert (got_mask == want_mask).all() and (got_next == want_next).all()


def test_out_of_range_transitions_count_as_dead():
    trans = np.array([[5] * 256, [1] * 256], dtype=np.int32)     # state 0 points outside
    t, a, dead, off = stack_automata([(trans, np.array([1, 0], np.uint8), 1)])
    assert (t[0] == dead).all() and dead == 1 and off.tolist() == [0, 1]
    with pytest.raises(ValueError):
        stack_automata([(trans, np.zeros(2, np.uint8), 2)])


@pytest.mark.gpu
def test_one_build_call_indexes_every_automaton():
    import paper_2307_09702_b200 as fg
    w = make_config(2)                                           # 32,000-token vocabulary
    automata = _automata()
    trans, accept, dead_all, offsets = stack_automata(automata)
    want_mask, want_next = _expected_rows(automata, w, dead_all, offsets)
    for algo in (1, 2, 0):
        fg.fsm_debug_set(6, algo)
        idx = fg.GuidedIndex(trans, accept, w.vocab_bytes, w.vocab_offsets, dead_all, w.eos_id).build()
        torch.cuda.synchronize()
        assert (idx.allowed_mask.cpu().numpy().view(np.uint32) == want_mask).all()
        assert (idx.next_state.cpu().numpy() == want_next).all()
        only = fg.GuidedIndex(trans, accept, w.vocab_bytes, w.vocab_offsets, dead_all, w.eos_id,
                              want_next=False).build()
        torch.cuda.synchronize()
        assert (only.allowed_mask.cpu().numpy().view(np.uint32) == want_mask).all()
        assert int(idx.status.item()) == 0 and int(only.status.item()) == 0
    fg.fsm_debug_set(6, 0)
