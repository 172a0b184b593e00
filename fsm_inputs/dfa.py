"""Hand-built and seeded random byte-level DFAs (inputs only).

All tables follow the dense form of the paper's Definition 1: ``trans[q, b]``
is delta(q, b) for the 256 byte values, ``accept[q]`` marks F, and one
designated absorbing dead state stands for "delta is undefined".  Live states
are 0..Q-2, the dead state is Q-1, the start state is 0.
"""
from __future__ import annotations

import numpy as np

from .regex_dfa import DFA

_DIGITS = list(range(0x30, 0x3A))


def _blank(Q: int):
    dead = Q - 1
    return np.full((Q, 256), dead, dtype=np.int32), np.zeros(Q, dtype=np.uint8), dead


def signed_decimal_dfa() -> DFA:
    """``[+-]?[0-9]+(\\.[0-9]+)?``: 0 start, 1 after sign, 2 integer digits
    (accepting), 3 after the dot, 4 fraction digits (accepting), 5 dead."""
    trans, accept, dead = _blank(6)
    trans[0, [ord("+"), ord("-")]] = 1
    trans[0, _DIGITS] = 2
    trans[1, _DIGITS] = 2
    trans[2, _DIGITS] = 2
    trans[2, ord(".")] = 3
    trans[3, _DIGITS] = 4
    trans[4, _DIGITS] = 4
    accept[[2, 4]] = 1
    return DFA(trans, accept, 0, dead)


def paper_float_example_dfa() -> DFA:
    """The un-reduced automaton of the paper's Example 1 (Section 3, regex
    ``([0-9]*)?\\.?[0-9]*``).  The figure is not available; the numbering is fixed
    by the text: generation starts in state 0, ".2" leads to state 3 and "1" to
    state 1.  0 -digit-> 1, 1 -digit-> 1, 0/1 -'.'-> 2, 2 -digit-> 3,
    3 -digit-> 3; every live state accepts; 4 is dead."""
    trans, accept, dead = _blank(5)
    trans[0, _DIGITS] = 1
    trans[1, _DIGITS] = 1
    trans[0, ord(".")] = 2
    trans[1, ord(".")] = 2
    trans[2, _DIGITS] = 3
    trans[3, _DIGITS] = 3
    accept[[0, 1, 2, 3]] = 1
    return DFA(trans, accept, 0, dead)


def paper_name_dfa() -> DFA:
    """The three-state NAME automaton of the paper's Section 4 walk-through
    (``[^\\W\\d]\\w*``): 0 initial, 1 after the first identifier character, 2 inside
    ``\\w*``; 1 and 2 accept; 3 is dead."""
    trans, accept, dead = _blank(4)
    word = _DIGITS + list(range(0x41, 0x5B)) + list(range(0x61, 0x7B)) + [ord("_")]
    first = [b for b in word if b not in _DIGITS]
    trans[0, first] = 1
    trans[1, word] = 2
    trans[2, word] = 2
    accept[[1, 2]] = 1
    return DFA(trans, accept, 0, dead)


def random_class_dfa(seed: int, n_live: int, n_classes: int = 64,
                     live_classes_per_state: int = 12,
                     accept_fraction: float = 0.10) -> tuple[DFA, np.ndarray]:
    """Seeded random automaton with a byte-class structure.

    Each of the 256 bytes is assigned uniformly to one of ``n_classes`` classes.
    Every live state picks ``live_classes_per_state`` distinct classes, each
    leading to a uniformly random live state; every other byte leads to the dead
    state.  ``accept_fraction`` of the live states accept; any live state that
    could not reach an accepting state is made accepting (so the automaton is
    trim).  Returns the dense DFA and the generating class map (for reference
    only - consumers re-derive classes from the table)."""
    rng = np.random.default_rng(seed)
    Q = n_live + 1
    dead = Q - 1
    cls = rng.integers(0, n_classes, size=256)
    # k distinct classes per state: argpartition of iid uniforms.
    keys = rng.random((n_live, n_classes))
    live_cls = np.argpartition(keys, live_classes_per_state - 1, axis=1)[:, :live_classes_per_state]
    targets = rng.integers(0, n_live, size=(n_live, live_classes_per_state))
    ctab = np.full((Q, n_classes), dead, dtype=np.int32)
    np.put_along_axis(ctab[:n_live], live_cls, targets.astype(np.int32), axis=1)
    accept = np.zeros(Q, dtype=np.uint8)
    accept[:n_live] = rng.random(n_live) < accept_fraction
    # Backward reachability from the accepting states.
    good = accept.astype(bool).copy()
    while True:
        reach = good[ctab].any(axis=1)
        reach[dead] = False
        new = good | reach
        if (new == good).all():
            break
        good = new
    fix = ~good
    fix[dead] = False
    accept[fix] = 1
    trans = np.ascontiguousarray(ctab[:, cls])
    return DFA(trans, accept, 0, dead), cls
