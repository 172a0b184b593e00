"""Pins of the CPU oracle against things other than itself: the paper's worked
examples, Python's ``re`` by brute force, closed forms and special cases that
reduce to a table lookup or a NumPy one-liner.  No GPU needed."""
import itertools
import os
import re

import numpy as np
import pytest

from fsm_inputs import (compile_regex, f32_to_bf16_bits, make_config, paper_float_example_dfa,
                        paper_name_dfa, random_class_dfa, signed_decimal_dfa, token_bytes,
                        vocab_from_strings)
from oracle import fsm_oracle, token_major

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bit(mask, q, v):
    return int(mask[q, v >> 5] >> np.uint32(v & 31)) & 1


def allowed_set(mask, q, N):
    return {v for v in range(N) if bit(mask, q, v)}


# ----------------------------------------------------------------- paper examples
def test_paper_example_1_masks_and_moves():
    """Section 3, Example 1: the printed allowed sets and state moves."""
    tokens, states, moves = None, [], []
    for line in open(os.path.join(GOLDEN, "paper_example1.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "tokens":
            tokens = f[1:]
        elif f[0] == "state":
            want = set() if f[3] == "-" else set(f[3].split(","))
            states.append((int(f[1]), want))
        elif f[0] == "move":
            moves.append((int(f[1]), f[2], int(f[4])))
    assert tokens == ["A", ".", "42", ".2", "1"]
    dfa = paper_float_example_dfa()
    vb, vo = vocab_from_strings(tokens)
    mask, nxt, _ = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    assert len(states) == 5 and len(moves) >= 2
    for q, want in states:
        got = {tokens[v] for v in allowed_set(mask, q, len(tokens))}
        assert got == want, (q, got, want)
    for q, tok, q2 in moves:
        assert nxt[q, tokens.index(tok)] == q2
    # "A" is never allowed; disallowed entries carry the dead state
    assert all(nxt[q, 0] == dfa.dead for q in range(dfa.Q))


def test_paper_name_example_sequences():
    """Section 4: "f" gives the state sequences (0,1), (1,2), (2,2)."""
    want, accepting = [], None
    for line in open(os.path.join(GOLDEN, "paper_name_example.txt")):
        f = line.split()
        if f and f[0] == "sequence":
            want.append(tuple(int(x) for x in f[1:]))
        if f and f[0] == "accepting":
            accepting = {int(x) for x in f[1:]}
    dfa = paper_name_dfa()
    assert {q for q in range(dfa.Q) if dfa.accept[q]} == accepting
    assert token_major.state_sequences(dfa.trans, dfa.dead, b"f") == want
    vb, vo = vocab_from_strings(["f"])
    mask, nxt, _ = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    for z in want:
        assert bit(mask, z[0], 0) == 1 and nxt[z[0], 0] == z[-1]
    assert bit(mask, dfa.dead, 0) == 0


# ------------------------------------------- two formulations, written separately
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_token_major_algorithms_agree_with_state_major_definition(seed):
    """Algorithms 3/4 in the paper's token-major order (pure Python) against the
    state-major C oracle, on random automata with multi-byte tokens."""
    rng = np.random.default_rng(seed)
    dfa, _ = random_class_dfa(seed, n_live=7, n_classes=5, live_classes_per_state=3)
    vocab = [bytes(rng.integers(0, 256, size=rng.integers(1, 6)).tolist()) for _ in range(70)]
    vocab[13] = b""
    vb, vo = vocab_from_strings(vocab)
    mask, nxt, _ = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    sigma, end = token_major.index_by_token(dfa.trans, dfa.dead, vocab)
    for q in range(dfa.Q):
        assert allowed_set(mask, q, len(vocab)) == sigma[q]
        for v in range(len(vocab)):
            assert nxt[q, v] == end.get((q, v), dfa.dead)
    assert sum(len(s) for s in sigma.values()) > 20      # the case is not vacuous


# ------------------------------------------------------- special case: 1-byte tokens
def test_single_byte_vocabulary_is_the_transition_table():
    dfa, _ = random_class_dfa(5, n_live=40, n_classes=16, live_classes_per_state=5)
    order = np.random.default_rng(0).permutation(256)
    vb, vo = vocab_from_strings([bytes([b]) for b in order])
    mask, nxt, lookups = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    want = dfa.trans[:, order].copy()
    want[dfa.dead, :] = dfa.dead
    assert (nxt == want).all()
    bits = np.unpackbits(mask.view(np.uint8), axis=1, bitorder="little")[:, :256]
    assert (bits == (want != dfa.dead)).all()
    assert lookups == (dfa.Q - 1) * 256      # one evaluation of delta per live walk


# -------------------------------------------------- brute force against Python's re
def language_prefixes(pattern: str, alphabet: bytes, max_len: int):
    """All strings over ``alphabet`` up to ``max_len`` that full-match, and all
    their prefixes, by exhaustive enumeration with ``re``."""
    rx = re.compile(pattern.encode("latin-1"))
    lang, prefixes = set(), set()
    for n in range(max_len + 1):
        for t in itertools.product(alphabet, repeat=n):
            s = bytes(t)
            if rx.fullmatch(s):
                lang.add(s)
                for k in range(n + 1):
                    prefixes.add(s[:k])
    return lang, prefixes


# (pattern, alphabet, vocabulary, enumeration length).  The length is chosen so
# that every viable prefix no longer than three tokens has a completion within
# it: the longest chain plus the longest shortest-completion, or the length of
# the longest string when the language is finite.
BRUTE_CASES = [
    (r"a(b|c)*a", b"abc", ["a", "b", "c", "ab", "ca", "bb", "aa", "ba", ""], 6 + 1),
    (r"(ab)+c?", b"abc", ["a", "b", "c", "ab", "ba", "bc", "abc", "bab"], 9 + 2),
    (r"[ab]{2,4}c", b"abc", ["a", "b", "c", "ab", "bc", "cc", "aab"], 5),
    (r"[+-]?[0-9]+(\.[0-9]+)?", b"-1.", ["-", "1", ".", "-1", "1.", ".1", "11", "1.1", "--"], 9 + 1),
    (r"(a|ab)(c|bcd)?", b"abcd", ["a", "b", "c", "d", "ab", "bc", "cd", "bcd"], 5),
]


@pytest.mark.parametrize("pattern,alphabet,vocab,max_len", BRUTE_CASES)
def test_index_chains_match_regex_brute_force(pattern, alphabet, vocab, max_len):
    """Every concatenation of up to 3 tokens is accepted step by step by the
    index iff the bytes are a viable prefix of the language, the final state
    accepts iff they full-match, and next(next(q,a),b) equals the DFA run."""
    dfa = compile_regex(pattern)
    vb, vo = vocab_from_strings(vocab)
    mask, nxt, _ = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    toks = [t.encode() for t in vocab]
    lang, prefixes = language_prefixes(pattern, alphabet, max_len)
    n_ok = n_bad = 0
    for n in (1, 2, 3):
        for chain in itertools.product(range(len(toks)), repeat=n):
            q, ok = dfa.start, True
            for v in chain:
                if not bit(mask, q, v):
                    ok = False
                    break
                q = int(nxt[q, v])
                assert q != dfa.dead
            s = b"".join(toks[v] for v in chain)
            if any(len(toks[v]) == 0 for v in chain):
                assert not ok                   # zero-length tokens are never allowed
                continue
            assert ok == (s in prefixes), (chain, s)
            if ok:
                assert bool(dfa.accept[q]) == (s in lang), (chain, s)
                n_ok += 1
            else:
                n_bad += 1
    assert n_ok > 3 and n_bad > 3


def test_hand_built_decimal_dfa_matches_re():
    """The hand-built workload-1 automaton, indexed from every state, against
    re on all strings: allowed(q0, t) iff t is a viable prefix."""
    dfa = signed_decimal_dfa()
    _, prefixes = language_prefixes(r"[+-]?[0-9]+(\.[0-9]+)?", b"+-7.", 7)
    toks = [bytes(t) for n in range(1, 4) for t in itertools.product(b"+-7.", repeat=n)]
    vb, vo = vocab_from_strings(toks)
    mask, _, _ = fsm_oracle.index_build(dfa.trans, dfa.accept, vb, vo, dfa.dead)
    for v, t in enumerate(toks):
        assert bit(mask, 0, v) == (t in prefixes), t


# ------------------------------------------------------------- structural invariants
def test_workload_1_invariants_and_layout():
    w = make_config(1)
    d = w.dfa
    mask, nxt, lookups = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets,
                                                d.dead, w.eos_id)
    N, W = w.N, w.W
    assert mask.shape == (d.Q, W) and nxt.shape == (d.Q, N)
    # padding bits of the last word are zero
    assert N % 32 == 8 and (mask[:, -1] >> np.uint32(8)).max() == 0
    # bit set <=> next state is live, and it equals an independent run of delta*
    bits = np.unpackbits(mask.view(np.uint8), axis=1, bitorder="little")[:, :N]
    assert ((nxt != d.dead) == bits.astype(bool)).all()
    total = 0
    for q in range(d.Q):
        for v in range(N):
            if v == w.eos_id:
                continue
            s = q
            for b in token_bytes(w.vocab_bytes, w.vocab_offsets, v):
                s = int(d.trans[s, b])
                total += (q != d.dead)
                if s == d.dead:
                    break
            assert nxt[q, v] == (s if q != d.dead else d.dead)
    assert lookups == total
    # EOS column: allowed exactly in accepting states, keeps the state
    for q in range(d.Q):
        assert bit(mask, q, w.eos_id) == int(d.accept[q])
        assert nxt[q, w.eos_id] == (q if d.accept[q] else d.dead)
    # dead row is empty
    assert mask[d.dead].max() == 0 and (nxt[d.dead] == d.dead).all()


def test_dead_row_contents_are_never_consulted():
    """The walk is abandoned at the dead state (Algorithm 3), so a table whose
    dead row is not absorbing gives the same index."""
    w = make_config(1)
    d = w.dfa
    a = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    t2 = d.trans.copy()
    t2[d.dead, :] = 2
    b = fsm_oracle.index_build(t2, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all() and a[2] == b[2]


def test_row_ranges_threads_and_mask_only():
    w = make_config(2)
    d = w.dfa
    full = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    part = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                                  q_begin=11, q_end=30, threads=4)
    assert (part[0] == full[0][11:30]).all() and (part[1] == full[1][11:30]).all()
    par = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                                 threads=4, want_next=False)
    assert (par[0] == full[0]).all() and par[1] is None and par[2] == full[2]
    # zero-length special tokens (ids 0..2) are never allowed, except EOS in F
    for v in (0, 1):
        assert not any(bit(full[0], q, v) for q in range(d.Q))
    assert [bit(full[0], q, 2) for q in range(d.Q)] == list(d.accept)


def test_expected_lookups_per_walk_random_automaton():
    """Closed form: with live-transition probability p per byte and token length
    L, an abandoning walk makes (1 - p^L) / (1 - p) evaluations on average."""
    w = make_config(3)
    d = w.dfa
    _, _, lookups = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                           w.eos_id, q_begin=0, q_end=64, want_next=False, threads=4)
    lens = np.diff(w.vocab_offsets)
    lens = lens[lens > 0]
    # fraction of bytes that are live, averaged over states, for this automaton
    live_frac = (d.trans[:-1] != d.dead).mean(axis=0)          # per byte value
    p = float(live_frac[w.vocab_bytes].mean())
    want = ((1 - p ** lens) / (1 - p)).mean()
    got = lookups / (64 * len(lens))
    assert abs(got - want) / want < 0.05, (got, want, p)


# ------------------------------------------------------------------------ mask step
def np_mask_step_row(x_f32, bits):
    masked = np.where(bits, x_f32, -np.inf)
    return masked, (int(np.argmax(masked)) if bits.any() else -1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_step_against_numpy(dtype):
    """Masked output equals where(bit, x, -inf); the token is the first index of
    the maximum (NumPy's argmax returns the first maximum)."""
    rng = np.random.default_rng(11)
    Q, N, B = 9, 203, 16
    dead = Q - 1
    mask = rng.integers(0, 2**32, size=(Q, (N + 31) // 32), dtype=np.uint32)
    mask &= rng.integers(0, 2**32, size=mask.shape, dtype=np.uint32)      # about 25 % allowed
    mask[:, -1] &= np.uint32((1 << (N % 32)) - 1)
    mask[dead] = 0
    mask[3] = 0                                  # a live state with an empty row
    nxt = rng.integers(0, Q - 1, size=(Q, N)).astype(np.int32)
    x = np.round(rng.standard_normal((B, N)) * 2, 1).astype(np.float32)  # coarse grid: many ties
    x[0, :8] = [-0.0, 0.0, -0.0, 0.0, -np.inf, 0.0, -0.0, 0.0]
    states = rng.integers(0, Q - 1, size=B).astype(np.int32)
    states[5] = 3
    states[6] = dead
    finished = np.zeros(B, dtype=np.uint8)
    finished[7] = 1
    eos = 17
    mask[states[9], eos >> 5] |= np.uint32(1 << (eos & 31))
    x[9, eos] = 99.0                                      # row 9 picks EOS
    if dtype == "bf16":
        logits = f32_to_bf16_bits(x)
        xf = (logits.astype(np.uint32) << 16).view(np.float32)
        neg_inf = np.uint16(0xFF80)
    else:
        logits, xf, neg_inf = x.copy(), x, np.float32(-np.inf)
    st, fin = states.copy(), finished.copy()
    tokens, out = fsm_oracle.mask_step(logits, st, fin, mask, nxt, dead, eos)
    bits = np.unpackbits(mask.view(np.uint8), axis=1, bitorder="little")[:, :N].astype(bool)
    for i in range(B):
        if finished[i]:
            assert tokens[i] == -1 and st[i] == states[i] and fin[i] == finished[i]
            assert (out[i] == logits[i]).all()
            continue
        q = states[i]
        masked, tok = np_mask_step_row(xf[i], bits[q])
        assert tokens[i] == tok
        want_out = np.where(bits[q], logits[i], neg_inf)
        assert (out[i].view(logits.dtype) == want_out).all()      # bit-identical pass-through
        if tok < 0:
            assert fin[i] == 2 and st[i] == q
        elif tok == eos:
            assert fin[i] == 1 and st[i] == q
        else:
            assert fin[i] == 0 and st[i] == nxt[q, tok]
    assert fin[5] == 2 and fin[6] == 2 and fin[9] == 1 and tokens[9] == eos
    # select-only mode gives the same tokens and writes nothing
    st2, fin2 = states.copy(), finished.copy()
    tokens2, out2 = fsm_oracle.mask_step(logits, st2, fin2, mask, nxt, dead, eos, write_logits=False)
    assert out2 is None and (tokens2 == tokens).all() and (st2 == st).all() and (fin2 == fin).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_mask_step_orders_subnormals_like_numpy(dtype):
    """Subnormal logits, signed zeros and the smallest normal number are ordered as IEEE
    floats (NumPy's argmax on the widened values is the definition written out)."""
    rng = np.random.default_rng(23)
    N, Q = 400, 2
    mask = rng.integers(0, 2**32, size=(Q, (N + 31) // 32), dtype=np.uint32)
    mask[:, -1] &= np.uint32((1 << (N % 32)) - 1)
    mask[1] = 0
    nxt = np.zeros((Q, N), dtype=np.int32)
    if dtype == "bf16":
        pos = np.array([0x0001, 0x0003, 0x007F, 0x0080, 0x0081, 0x0000], dtype=np.uint16)
        vals = np.concatenate([pos, pos | np.uint16(0x8000)])
        widen = lambda a: (a.astype(np.uint32) << 16).view(np.float32)
    else:
        pos = np.array([1, 0x12345, 0x7FFFFF, 0x800000, 0x800001, 0], dtype=np.uint32)
        vals = np.concatenate([pos, pos | np.uint32(0x80000000)]).view(np.float32)
        widen = lambda a: a
    bits = np.unpackbits(mask.view(np.uint8), axis=1, bitorder="little")[:, :N].astype(bool)
    for trial in range(40):
        top = 1 + trial % len(pos)             # restrict the value set so that every level wins
        pool = np.concatenate([vals[:top], vals[len(pos):]])
        logits = rng.choice(pool, size=(1, N))
        st, fin = np.zeros(1, np.int32), np.zeros(1, np.uint8)
        tokens, out = fsm_oracle.mask_step(logits, st, fin, mask, nxt, Q - 1, -1)
        _, tok = np_mask_step_row(widen(logits[0]), bits[0])
        assert tokens[0] == tok
        assert widen(logits[0])[tok] == widen(logits[0])[bits[0]].max()


def test_mask_step_all_allowed_logits_minus_inf_picks_lowest_allowed_id():
    N, Q = 70, 3
    mask = np.zeros((Q, 3), dtype=np.uint32)
    for v in (41, 5, 66):
        mask[0, v >> 5] |= np.uint32(1 << (v & 31))
    nxt = np.full((Q, N), 1, dtype=np.int32)
    x = np.full((1, N), 3.0, dtype=np.float32)
    x[0, [5, 41, 66]] = -np.inf
    st, fin = np.zeros(1, np.int32), np.zeros(1, np.uint8)
    tokens, out = fsm_oracle.mask_step(x, st, fin, mask, nxt, Q - 1, -1)
    assert tokens[0] == 5 and st[0] == 1 and np.isneginf(out).all()


def test_greedy_decode_stays_inside_the_language():
    """Workload 1 decoded greedily for 20 steps: every prefix of the output is a
    viable prefix of [+-]?[0-9]+(\\.[0-9]+)? (checked with re on the hand-derived
    prefix language), and a sequence that ends with EOS full-matches."""
    w = make_config(1)
    d = w.dfa
    mask, nxt, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets,
                                          d.dead, w.eos_id)
    prefix_rx = re.compile(rb"[+-]?([0-9]+(\.[0-9]*)?)?")
    full_rx = re.compile(rb"[+-]?[0-9]+(\.[0-9]+)?")
    rng = np.random.default_rng(3)
    n_eos = 0
    for trial in range(30):
        st, fin = np.zeros(1, np.int32), np.zeros(1, np.uint8)
        text = b""
        for step in range(20):
            x = rng.standard_normal((1, w.N)).astype(np.float32)
            if step > 2 and trial % 2:
                x[0, w.eos_id] = 50.0               # EOS wins as soon as it is allowed
            tokens, _ = fsm_oracle.mask_step(x, st, fin, mask, nxt, d.dead, w.eos_id)
            if fin[0]:
                break
            text += token_bytes(w.vocab_bytes, w.vocab_offsets, int(tokens[0]))
            assert prefix_rx.fullmatch(text), text
        if fin[0] == 1:
            n_eos += 1
            assert full_rx.fullmatch(text), text
        assert len(text) > 0
    assert n_eos > 5
