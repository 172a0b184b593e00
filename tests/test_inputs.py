"""Checks of the synthetic input generators (no GPU): the host regex compiler
against Python's ``re``, and the shapes / statistics of the five workloads."""
import re

import numpy as np
import pytest

from fsm_inputs import (JSON_OBJECT_REGEX, compile_regex, dfa_run, make_config, random_class_dfa,
                        start_states)

PATTERNS = [
    (r"\s*([Yy]es|[Nn]o|[Nn]ever|[Aa]lways)", b" YyesNoNvrAlwa"),
    (r"\s*19[0-9]{2}", b" 1952"),
    (r"((25[0-5]|2[0-4]\d|[01]?\d\d?)\.){3}(25[0-5]|2[0-4]\d|[01]?\d\d?)", b"0125."),
    (r"[^\W\d]\w*", b"a_9 -"),
    (r"([0-9]*)?\.?[0-9]*", b"42.A"),
    (r"(?:ab|a)(?:bc|c){1,2}x{0,2}", b"abcx"),
    (r'"[^"\\\x00-\x1f]*"', b'"a\\\x01 '),
]


@pytest.mark.parametrize("pattern,alphabet", PATTERNS)
def test_compiled_dfa_agrees_with_re(pattern, alphabet):
    dfa = compile_regex(pattern)
    rx = re.compile(pattern.encode("latin-1"))
    rng = np.random.default_rng(0)
    n_match = 0
    for _ in range(4000):
        s = bytes(rng.choice(list(alphabet), size=rng.integers(0, 9)).tolist())
        got = bool(dfa.accept[dfa_run(dfa, s)])
        assert got == (rx.fullmatch(s) is not None), s
        n_match += got
    assert n_match > 0
    # trim: the dead state absorbs and nothing else is a trap
    assert (dfa.trans[dfa.dead] == dfa.dead).all() and not dfa.accept[dfa.dead]


def test_paper_section_3_1_outputs_match_their_patterns():
    """The guided outputs printed in the paper's Section 3.1 full-match the
    regular expressions they were generated under."""
    cases = [(r"\s*([Yy]es|[Nn]o|[Nn]ever|[Aa]lways)", b"Always"),
             (r"\s*19[0-9]{2}", b"1952"),
             (r"((25[0-5]|2[0-4]\d|[01]?\d\d?)\.){3}(25[0-5]|2[0-4]\d|[01]?\d\d?)", b"2.2.6.1")]
    for pattern, text in cases:
        dfa = compile_regex(pattern)
        assert dfa.accept[dfa_run(dfa, text)]


def test_json_workload_automaton():
    w = make_config(2)
    assert 70 <= w.Q <= 90 and w.N == 32000
    doc = b'{"first_name": "ann", "home_city": "x y", "email": "a@b", "age": -12, "score": 0.50}'
    assert w.dfa.accept[dfa_run(w.dfa, doc)]
    assert re.fullmatch(JSON_OBJECT_REGEX.encode(), doc)
    assert not w.dfa.accept[dfa_run(w.dfa, doc[:-1])]


@pytest.mark.parametrize("k,N,Q,live", [(3, 128256, 1001, 12), (4, 152064, 20001, 16)])
def test_random_workloads_shape(k, N, Q, live):
    w = make_config(k)
    assert w.N == N and w.Q == Q and w.dfa.dead == Q - 1
    lens = np.diff(w.vocab_offsets)
    assert lens.max() == 16 and lens.min() == 0
    assert 3.7 < lens[lens > 0].mean() < 4.2
    assert lens[w.eos_id] == 0
    t = w.dfa.trans
    assert t.min() >= 0 and t.max() < Q and (t[-1] == Q - 1).all()
    # every live state has exactly `live` live byte classes
    cols = np.unique(t.T, axis=0)
    assert len(cols) <= 64
    live_per_state = (cols.T != Q - 1).sum(axis=1)[:-1]
    assert (live_per_state <= live).all() and live_per_state.mean() > live - 3
    assert 0.05 < w.dfa.accept[:-1].mean() < 0.15
    # deterministic
    w2 = make_config(k)
    assert w.sha256() == w2.sha256()


def test_decode_workload_and_tiny():
    w5 = make_config(5)
    assert w5.B == 256 and w5.steps == 1000 and w5.logits_dtype == "bf16"
    s = start_states(w5)
    assert s.shape == (256,) and s.min() >= 0 and s.max() < w5.Q - 1
    assert make_config(3).sha256() == w5.sha256()
    w1 = make_config(1)
    assert w1.N == 1000 and w1.Q == 6 and w1.B == 1 and w1.steps == 20
    lens = np.diff(w1.vocab_offsets)
    assert lens[:-1].min() == 1 and lens.max() == 8


def test_random_dfa_is_trim():
    dfa, cls = random_class_dfa(9, n_live=50, n_classes=8, live_classes_per_state=2, accept_fraction=0.05)
    good = dfa.accept.astype(bool).copy()
    for _ in range(dfa.Q):
        good |= good[dfa.trans].any(axis=1)
        good[dfa.dead] = False
    assert good[:-1].all()
