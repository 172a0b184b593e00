"""TEST INFRASTRUCTURE: the vocabulary index computed token by token (Section 3,
Algorithms 3 and 4), in pure Python for small inputs.  It is the second, separately
written formulation that pins the state-major C oracle.

For one token, ``state_sequences`` runs delta over the token's bytes from every state and
keeps the runs that never leave the automaton; ``index_by_token`` turns those runs around
into sigma: state -> allowed tokens, and remembers where each run ended.

Two readings, both fixed by the paper's own Section 4 example (the one-character string
"f" over the three-state NAME automaton gives (0,1), (1,2), (2,2)):

  * a run is recorded as the state it starts in followed by the state after every
    character, so a token of k bytes gives k + 1 states;
  * a run that meets an undefined transition is dropped altogether.
"""
from __future__ import annotations


def state_sequences(trans, dead, token: bytes):
    """All complete runs of ``token``: tuples (start, after byte 0, ..., after last byte)."""
    runs = []
    if len(token) == 0:
        return runs
    for start in range(len(trans)):
        if start == dead:
            continue
        visited = [start]
        for byte in token:
            nxt = int(trans[visited[-1]][byte])
            if nxt == dead:
                visited = None
                break
            visited.append(nxt)
        if visited is not None:
            assert len(visited) == len(token) + 1
            runs.append(tuple(visited))
    return runs


def index_by_token(trans, dead, vocabulary):
    """Returns ``(sigma, end)``: ``sigma[q]`` is the set of token ids whose run from q is
    complete, ``end[(q, v)]`` the state that run ends in."""
    sigma = {q: set() for q in range(len(trans))}
    end = {}
    for token_id, token in enumerate(vocabulary):
        for run in state_sequences(trans, dead, token):
            sigma[run[0]].add(token_id)
            end[(run[0], token_id)] = run[-1]
    return sigma, end
