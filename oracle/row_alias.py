"""TEST INFRASTRUCTURE: merging of identical index rows, from the definition.

The paper's index maps a state to its set of allowed tokens (Section 3, Algorithm 4) and is
built from automata that are not reduced (Section 5), so different states can carry the
same row.  ``row_alias[q]`` is the smallest state whose row equals state q's:

* for the map to sets alone (``next_state=None``): the same set of allowed tokens;
* for an index that also stores where each token leads: the same set and the same end state
  for every token in it (only then can two states share one stored row).

Plain Python over numpy rows: the first state seen with a given row is remembered under the
row's bytes (compared exactly); no hashing of our own, no shortcuts."""
from __future__ import annotations

import numpy as np


def row_alias(allowed_mask, next_state=None):
    """Returns ``(row_alias int32 [Q], n_unique)``."""
    mask = np.ascontiguousarray(allowed_mask)
    Q = mask.shape[0]
    nxt = None if next_state is None else np.ascontiguousarray(next_state)
    first = {}
    alias = np.zeros(Q, dtype=np.int32)
    for q in range(Q):
        row = mask[q].tobytes() if nxt is None else mask[q].tobytes() + nxt[q].tobytes()
        alias[q] = first.setdefault(row, q)
    return alias, len(first)
