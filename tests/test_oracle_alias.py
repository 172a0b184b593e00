"""Pins of the row-merging oracle (``oracle/row_alias.py``) against things other than itself:
the paper's worked example, a brute-force double loop, numpy's own row grouping, and the
cloned-state construction whose answer is known beforehand."""
import numpy as np

from fsm_inputs import make_config, paper_float_example_dfa, vocab_from_strings
from oracle import fsm_oracle
from oracle.row_alias import row_alias


def _index(d, vb, vo, eos=-1):
    mask, nxt, _ = fsm_oracle.index_build(d.trans, d.accept, vb, vo, d.dead, eos)
    return mask, nxt


def test_paper_example_states_with_equal_sets_alias():
    """Section 3, Example 1: states 0 and 1 allow {".", "42", ".2", "1"}, states 2 and 3 allow
    {"42", "1"}; the moves printed there send both members of a pair to the same states."""
    d = paper_float_example_dfa()
    vb, vo = vocab_from_strings(["A", ".", "42", ".2", "1"])
    mask, nxt = _index(d, vb, vo)
    for use_next in (None, nxt):
        alias, n = row_alias(mask, use_next)
        assert alias.tolist() == [0, 0, 2, 2, 4] and n == 3


def test_against_a_double_loop_and_numpy_grouping():
    rng = np.random.default_rng(0)
    for trial in range(20):
        Q, W, N = int(rng.integers(1, 40)), 3, 70
        pool_m = rng.integers(0, 2**32, size=(5, W), dtype=np.uint32)
        pool_n = rng.integers(0, Q, size=(6, N)).astype(np.int32)
        pm, pn = rng.integers(0, 5, size=Q), rng.integers(0, 6, size=Q)
        mask, nxt = pool_m[pm], pool_n[pn]
        for use_next in (False, True):
            got, n = row_alias(mask, nxt if use_next else None)
            want = np.zeros(Q, np.int32)
            for q in range(Q):                      # the definition, quadratically
                for r in range(q + 1):
                    if (mask[r] == mask[q]).all() and (not use_next or (nxt[r] == nxt[q]).all()):
                        want[q] = r
                        break
            assert (got == want).all()
            rows = mask.view(np.int32) if not use_next else np.concatenate([mask.view(np.int32), nxt], axis=1)
            _, inverse = np.unique(rows, axis=0, return_inverse=True)
            firsts = {}
            for q, g in enumerate(np.ravel(inverse)):
                firsts.setdefault(int(g), q)
            assert got.tolist() == [firsts[int(g)] for g in np.ravel(inverse)]
            assert n == len(firsts)
            assert (got <= np.arange(Q)).all() and (got[got] == got).all()


def test_equal_sets_with_different_moves_alias_only_as_sets():
    # states 0, 1 and 2 all read exactly the letter "a" (same token set {"a", "aa"}); 0 moves to 1
    # on it, 1 and 2 both move to 2: as stored rows only 1 and 2 are alike
    Q = 4
    trans = np.full((Q, 256), 3, dtype=np.int32)
    trans[0, 97], trans[1, 97], trans[2, 97] = 1, 2, 2
    accept = np.ones(Q, np.uint8)

    class D:
        pass
    d = D()
    d.trans, d.accept, d.dead = trans, accept, 3
    vb, vo = vocab_from_strings(["a", "b", "aa"])
    mask, nxt = _index(d, vb, vo)
    assert row_alias(mask)[0].tolist() == [0, 0, 0, 3]
    assert row_alias(mask, nxt)[0].tolist() == [0, 1, 1, 3]


def test_a_cloned_state_aliases_its_original():
    """Appending a copy of state s (same outgoing transitions, same acceptance) to an automaton
    gives a state with exactly s's index row; states that were different stay different."""
    w = make_config(1)
    d = w.dfa
    base_mask, base_next = _index(d, w.vocab_bytes, w.vocab_offsets, w.eos_id)
    base_alias, base_n = row_alias(base_mask, base_next)
    for s in (0, 2, d.Q - 2):
        trans = np.concatenate([d.trans, d.trans[s:s + 1]], axis=0)
        accept = np.concatenate([d.accept, d.accept[s:s + 1]])

        class D:
            pass
        c = D()
        c.trans, c.accept, c.dead = trans, accept, d.dead
        mask, nxt = _index(c, w.vocab_bytes, w.vocab_offsets, w.eos_id)
        alias, n = row_alias(mask, nxt)
        # EOS keeps the state, so an accepting clone differs from its original in that one entry
        if d.accept[s] and w.eos_id >= 0:
            assert alias[d.Q] == d.Q and n == base_n + 1
            assert row_alias(mask)[0][d.Q] == row_alias(mask)[0][s]
        else:
            assert alias[d.Q] == base_alias[s] and n == base_n
        assert (alias[:d.Q] == base_alias).all()
