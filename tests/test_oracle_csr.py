"""Pins of the compressed-row form of the index (sigma as token sets, the paper's own
data structure): the paper's worked example, and the round trip to the dense form."""
import numpy as np

from fsm_inputs import make_config, paper_float_example_dfa, vocab_from_strings
from oracle import fsm_oracle


def test_paper_example_rows_as_token_sets():
    """Section 3, Example 1: in state 0 the tokens ".", "42", ".2", "1" may be sampled;
    ".2" leads to state 3 and "1" to state 1; in state 3 only "42" and "1" remain."""
    d = paper_float_example_dfa()
    vb, vo = vocab_from_strings(["A", ".", "42", ".2", "1"])
    _, off, tok, nxt = fsm_oracle.index_csr(d.trans, d.accept, vb, vo, d.dead)
    assert off.tolist() == [0, 4, 8, 10, 12, 12]
    assert tok[off[0]:off[1]].tolist() == [1, 2, 3, 4]
    assert nxt[off[0]:off[1]].tolist() == [2, 1, 3, 1]
    assert tok[off[3]:off[4]].tolist() == [2, 4] and nxt[off[3]:off[4]].tolist() == [3, 3]


def test_compressed_rows_expand_to_the_dense_table():
    w = make_config(1)
    d = w.dfa
    mask, off, tok, nxt = fsm_oracle.index_csr(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets,
                                               d.dead, w.eos_id)
    _, dense, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    back = np.full_like(dense, d.dead)
    for q in range(d.Q):
        row = slice(off[q], off[q + 1])
        assert (np.diff(tok[row]) > 0).all()                 # increasing ids, no duplicates
        assert (nxt[row] != d.dead).all()                    # only surviving walks are listed
        back[q, tok[row]] = nxt[row]
    assert (back == dense).all()
    assert off[-1] == sum(bin(int(x)).count("1") for x in mask.ravel())
    assert off[d.dead + 1] == off[d.dead]                    # the dead state's set is empty
