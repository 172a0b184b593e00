"""Several automata indexed by one ``fsm_index_build`` call.

The paper's extension to context-free grammars (Section 4) needs one vocabulary index
per parser state: many small automata over the same vocabulary.  Index rows are
independent, so K automata can be stacked into one table with disjoint state ranges
and a single shared dead state, and built in one launch sequence; rows
``offsets[k] .. offsets[k+1]-1`` of the result are the index of automaton k (its live
states in their original order).  Only state renumbering happens here - no part of
the index is computed on the host.
"""
from __future__ import annotations

import numpy as np


def stack_automata(automata):
    """``automata``: sequence of ``(trans int32 [Q_k, 256], accept uint8 [Q_k], dead_k)``.

    Returns ``(trans, accept, dead, offsets)``: the stacked table with
    ``sum(Q_k - 1) + 1`` states, its accepting flags, the shared dead state (the last
    state) and ``offsets`` (int64 [K+1]) with automaton k's live states at
    ``offsets[k] + rank`` where ``rank`` counts its live states in increasing order.
    """
    offsets = [0]
    for trans, accept, dead in automata:
        Q = int(np.asarray(trans).shape[0])
        if not 0 <= dead < Q:
            raise ValueError("dead state out of range")
        offsets.append(offsets[-1] + Q - 1)
    total = offsets[-1] + 1
    dead_all = total - 1
    out_trans = np.full((total, 256), dead_all, dtype=np.int32)
    out_accept = np.zeros(total, dtype=np.uint8)
    for k, (trans, accept, dead) in enumerate(automata):
        trans = np.asarray(trans, dtype=np.int32)
        accept = np.asarray(accept, dtype=np.uint8)
        Q = trans.shape[0]
        # live states keep their order; the automaton's own dead state maps to the shared one
        new_id = np.empty(Q, dtype=np.int64)
        live = np.array([q for q in range(Q) if q != dead], dtype=np.int64)
        new_id[live] = offsets[k] + np.arange(Q - 1)
        new_id[dead] = dead_all
        bad = (trans < 0) | (trans >= Q)
        mapped = new_id[np.where(bad, dead, trans)]
        out_trans[offsets[k]:offsets[k + 1]] = mapped[live]
        out_accept[offsets[k]:offsets[k + 1]] = accept[live]
    return out_trans, out_accept, dead_all, np.asarray(offsets, dtype=np.int64)


def local_state_ids(automaton_states: int, dead: int, offset: int, dead_all: int):
    """Map from automaton k's own state ids to the stacked numbering (int64 [Q_k])."""
    ids = np.empty(automaton_states, dtype=np.int64)
    live = [q for q in range(automaton_states) if q != dead]
    ids[live] = offset + np.arange(automaton_states - 1)
    ids[dead] = dead_all
    return ids
