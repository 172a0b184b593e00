"""TEST INFRASTRUCTURE: the paper's Algorithms 3 and 4 in their own token-major
order and notation, in pure Python (small inputs only).

``find_sub_sequences`` returns, for one vocabulary string v, the state sequences
the automaton traverses when it reads v from each start state that can read
v's first character.  Two readings fix points where the printed algorithm and
the paper's own Section 4 example disagree:

  * a sequence is the start state followed by the state after *each* character
    (the example gives (0,1), (1,2), (2,2) for the one-character string "f"),
    so it has len(v) + 1 elements;
  * an abandoned walk contributes nothing (the printed listing would append an
    empty sequence, whose first element Algorithm 4 could not take).

``map_states_to_vocab`` is Algorithm 4: sigma(z_0) gains v for every sequence z.
"""
from __future__ import annotations


def find_sub_sequences(trans, dead, v: bytes):
    res = []
    if len(v) == 0:
        return res
    Q = len(trans)
    # delta^{-1}(., v_0): the states that read v_0
    for q in range(Q):
        if q == dead or trans[q][v[0]] == dead:
            continue
        r = int(trans[q][v[0]])
        p = [q, r]
        for i in range(1, len(v)):          # walk the FSM
            if trans[r][v[i]] == dead:      # the FSM does not read v_i
                p = []
                break
            r = int(trans[r][v[i]])
            p.append(r)
        if p:
            res.append(tuple(p))
    return res


def map_states_to_vocab(trans, dead, vocabulary):
    """Returns ``(sigma, end)``: ``sigma[q]`` is the set of token ids allowed in
    state q, ``end[(q, v)]`` the last element of the sequence that starts in q."""
    sigma = {q: set() for q in range(len(trans))}
    end = {}
    for v_id, v in enumerate(vocabulary):   # loop through the vocabulary
        for z in find_sub_sequences(trans, dead, v):
            sigma[z[0]].add(v_id)
            end[(z[0], v_id)] = z[-1]
    return sigma, end
