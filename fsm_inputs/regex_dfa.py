"""Host-side regex -> byte-level DFA compiler used only to *generate inputs*.

The guided-generation method takes a finite automaton (Q, Sigma, delta, q0, F)
(paper Definition 1) as given and delegates its construction to an existing
regular-expression library (paper Section 1).  This module is that library for
the synthetic workloads and the tiny brute-force test cases: it holds no part
of the vocabulary-index or masking arithmetic.

Pipeline: recursive-descent parse -> Thompson NFA over byte sets -> subset
construction -> Moore minimisation -> trimming of states that cannot reach an
accepting state (they are merged into one absorbing dead state).

Alphabet: the 256 byte values.  Semantics follow Python's ``re`` on *bytes*
patterns (``\\w`` is ``[A-Za-z0-9_]``, ``.`` is any byte but ``\\n``), which
the tests use as the independent matcher.

Output convention: live states are numbered 0..Q-2 in breadth-first order from
the start state 0; the dead state is Q-1.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

ALL = (1 << 256) - 1


def _set(chars) -> int:
    m = 0
    for c in chars:
        m |= 1 << (c if isinstance(c, int) else ord(c))
    return m


def _range(lo: int, hi: int) -> int:
    return ((1 << (hi + 1)) - 1) & ~((1 << lo) - 1)


DIGIT = _range(0x30, 0x39)
WORD = DIGIT | _range(0x41, 0x5A) | _range(0x61, 0x7A) | _set("_")
SPACE = _set(" \t\n\r\x0b\x0c")
ESCAPE_SETS = {
    "d": DIGIT, "D": ALL & ~DIGIT,
    "w": WORD, "W": ALL & ~WORD,
    "s": SPACE, "S": ALL & ~SPACE,
}
ESCAPE_CHARS = {"n": 10, "t": 9, "r": 13, "f": 12, "v": 11, "0": 0, "a": 7}


# --------------------------------------------------------------------------- AST
@dataclass
class Lit:           # one byte from a set
    mask: int

@dataclass
class Cat:
    parts: list

@dataclass
class Alt:
    options: list

@dataclass
class Rep:
    node: object
    lo: int
    hi: int | None    # None = unbounded


class _Parser:
    def __init__(self, pattern: str):
        self.p = pattern
        self.i = 0

    def peek(self):
        return self.p[self.i] if self.i < len(self.p) else None

    def take(self):
        c = self.p[self.i]
        self.i += 1
        return c

    def parse(self):
        node = self.alt()
        if self.i != len(self.p):
            raise ValueError(f"unexpected {self.p[self.i]!r} at {self.i}")
        return node

    def alt(self):
        options = [self.cat()]
        while self.peek() == "|":
            self.take()
            options.append(self.cat())
        return options[0] if len(options) == 1 else Alt(options)

    def cat(self):
        parts = []
        while self.peek() is not None and self.peek() not in "|)":
            parts.append(self.quantified())
        return Cat(parts)

    def quantified(self):
        node = self.atom()
        while True:
            c = self.peek()
            if c == "*":
                self.take(); node = Rep(node, 0, None)
            elif c == "+":
                self.take(); node = Rep(node, 1, None)
            elif c == "?":
                self.take(); node = Rep(node, 0, 1)
            elif c == "{":
                save = self.i
                self.take()
                lo = self.number()
                hi = lo
                if lo is not None and self.peek() == ",":
                    self.take()
                    hi = self.number()          # None -> unbounded
                if lo is None or self.peek() != "}":
                    self.i = save               # a literal brace
                    self.take()
                    return Cat([node, Lit(_set("{"))])
                self.take()
                node = Rep(node, lo, hi)
            else:
                return node

    def number(self):
        start = self.i
        while self.peek() is not None and self.peek().isdigit():
            self.take()
        return int(self.p[start:self.i]) if self.i > start else None

    def escape(self, in_class: bool) -> int:
        c = self.take()
        if c in ESCAPE_SETS:
            return ESCAPE_SETS[c]
        if c == "x":
            v = int(self.p[self.i:self.i + 2], 16)
            self.i += 2
            return 1 << v
        if c in ESCAPE_CHARS:
            return 1 << ESCAPE_CHARS[c]
        if c == "b" and in_class:
            return 1 << 8
        if c.isalnum():
            raise ValueError(f"unsupported escape \\{c}")
        return 1 << ord(c)

    def atom(self):
        c = self.take()
        if c == "(":
            if self.p.startswith("?:", self.i):
                self.i += 2
            node = self.alt()
            if self.peek() != ")":
                raise ValueError("missing )")
            self.take()
            return node
        if c == "[":
            return Lit(self.char_class())
        if c == ".":
            return Lit(ALL & ~(1 << 10))
        if c == "\\":
            return Lit(self.escape(False))
        if c in "*+?":
            raise ValueError(f"nothing to repeat at {self.i - 1}")
        if ord(c) > 255:
            raise ValueError("byte-level patterns only")
        return Lit(1 << ord(c))

    def char_class(self) -> int:
        negate = False
        if self.peek() == "^":
            self.take()
            negate = True
        mask = 0
        first = True
        while True:
            c = self.peek()
            if c is None:
                raise ValueError("missing ]")
            if c == "]" and not first:
                self.take()
                break
            first = False
            self.take()
            if c == "\\":
                lo_mask = self.escape(True)
            else:
                lo_mask = 1 << ord(c)
            single = lo_mask & (lo_mask - 1) == 0
            if single and self.peek() == "-" and self.i + 1 < len(self.p) and self.p[self.i + 1] != "]":
                self.take()
                d = self.take()
                hi_mask = self.escape(True) if d == "\\" else 1 << ord(d)
                if hi_mask & (hi_mask - 1):
                    raise ValueError("bad range end")
                lo, hi = lo_mask.bit_length() - 1, hi_mask.bit_length() - 1
                if hi < lo:
                    raise ValueError("reversed range")
                mask |= _range(lo, hi)
            else:
                mask |= lo_mask
        return (ALL & ~mask) if negate else mask


# --------------------------------------------------------------------------- NFA
class _NFA:
    def __init__(self):
        self.eps: list[list[int]] = []
        self.edges: list[list[tuple[int, int]]] = []   # (byte-set mask, target)

    def new(self) -> int:
        self.eps.append([])
        self.edges.append([])
        return len(self.eps) - 1

    def build(self, node) -> tuple[int, int]:
        """Returns (entry, exit) of a fragment with a single exit state."""
        if isinstance(node, Lit):
            a, b = self.new(), self.new()
            self.edges[a].append((node.mask, b))
            return a, b
        if isinstance(node, Cat):
            a = self.new()
            cur = a
            for part in node.parts:
                s, e = self.build(part)
                self.eps[cur].append(s)
                cur = e
            return a, cur
        if isinstance(node, Alt):
            a, b = self.new(), self.new()
            for opt in node.options:
                s, e = self.build(opt)
                self.eps[a].append(s)
                self.eps[e].append(b)
            return a, b
        if isinstance(node, Rep):
            a = self.new()
            cur = a
            for _ in range(node.lo):
                s, e = self.build(node.node)
                self.eps[cur].append(s)
                cur = e
            if node.hi is None:
                s, e = self.build(node.node)
                loop = self.new()
                self.eps[cur].append(loop)
                self.eps[loop].append(s)
                self.eps[e].append(loop)
                cur = loop
            else:
                end = self.new()
                for _ in range(node.hi - node.lo):
                    s, e = self.build(node.node)
                    self.eps[cur].append(end)
                    self.eps[cur].append(s)
                    cur = e
                self.eps[cur].append(end)
                cur = end
            return a, cur
        raise TypeError(node)

    def closure(self, states) -> frozenset:
        seen = set(states)
        stack = list(states)
        while stack:
            s = stack.pop()
            for t in self.eps[s]:
                if t not in seen:
                    seen.add(t)
                    stack.append(t)
        return frozenset(seen)


def _byte_partition(masks) -> list[list[int]]:
    """Groups the 256 bytes by their membership pattern over all edge sets."""
    groups: dict[tuple, list[int]] = {}
    masks = list(masks)
    for b in range(256):
        key = tuple((m >> b) & 1 for m in masks)
        groups.setdefault(key, []).append(b)
    return list(groups.values())


@dataclass
class DFA:
    """Dense byte-level DFA.  ``trans[q, b]`` is delta(q, b); ``dead`` absorbs."""
    trans: np.ndarray      # int32 [Q, 256]
    accept: np.ndarray     # uint8 [Q]
    start: int
    dead: int

    @property
    def Q(self) -> int:
        return int(self.trans.shape[0])


def compile_regex(pattern: str, minimise: bool = True) -> DFA:
    """Compiles ``pattern`` (full-match semantics) to a trimmed dense DFA."""
    ast = _Parser(pattern).parse()
    nfa = _NFA()
    entry, exit_ = nfa.build(ast)
    distinct_masks = {m for edges in nfa.edges for (m, _) in edges}
    groups = _byte_partition(distinct_masks)
    reps = [g[0] for g in groups]

    start = nfa.closure([entry])
    ids = {start: 0}
    order = [start]
    rows: list[list[int]] = []
    k = 0
    while k < len(order):
        cur = order[k]
        k += 1
        row = []
        for r in reps:
            tgt = set()
            for s in cur:
                for m, t in nfa.edges[s]:
                    if (m >> r) & 1:
                        tgt.add(t)
            nxt = nfa.closure(tgt) if tgt else frozenset()
            if nxt not in ids:
                ids[nxt] = len(order)
                order.append(nxt)
            row.append(ids[nxt])
        rows.append(row)
    n = len(order)
    acc = [exit_ in s for s in order]
    G = len(groups)

    # States that can reach an accepting state (backward closure).
    rev = [[] for _ in range(n)]
    for s in range(n):
        for t in rows[s]:
            rev[t].append(s)
    useful = [False] * n
    stack = [s for s in range(n) if acc[s]]
    for s in stack:
        useful[s] = True
    while stack:
        t = stack.pop()
        for s in rev[t]:
            if not useful[s]:
                useful[s] = True
                stack.append(s)

    # Moore refinement; all useless states start (and stay) in one block.
    if minimise:
        block = [0 if not useful[s] else (1 if acc[s] else 2) for s in range(n)]
        while True:
            sig = {}
            new = []
            for s in range(n):
                key = (block[s],) + tuple(block[t] for t in rows[s])
                new.append(sig.setdefault(key, len(sig)))
            if len(sig) == len(set(block)):
                break
            block = new
        block = new
    else:
        nxt_id = iter(range(1, n + 1))
        block = [0 if not useful[s] else next(nxt_id) for s in range(n)]

    dead_block = None
    for s in range(n):
        if not useful[s]:
            dead_block = block[s]
            break
    # Breadth-first renumbering of live blocks from the start state.
    if not useful[0]:
        raise ValueError("pattern matches nothing")
    rep_of = {}
    for s in range(n):
        rep_of.setdefault(block[s], s)
    new_id = {block[0]: 0}
    queue = [block[0]]
    k = 0
    while k < len(queue):
        b = queue[k]
        k += 1
        for t in rows[rep_of[b]]:
            tb = block[t]
            if tb != dead_block and tb not in new_id:
                new_id[tb] = len(queue)
                queue.append(tb)
    Q = len(queue) + 1
    dead = Q - 1
    trans = np.full((Q, 256), dead, dtype=np.int32)
    accept = np.zeros(Q, dtype=np.uint8)
    for b in queue:
        s = rep_of[b]
        q = new_id[b]
        accept[q] = 1 if acc[s] else 0
        for g in range(G):
            tb = block[rows[s][g]]
            if tb != dead_block:
                trans[q, groups[g]] = new_id[tb]
    return DFA(trans=trans, accept=accept, start=0, dead=dead)


def dfa_run(dfa: DFA, data: bytes, state: int | None = None) -> int:
    """Plain delta* used by input self-checks (not by the oracle or the kernels)."""
    s = dfa.start if state is None else state
    for b in data:
        s = int(dfa.trans[s, b])
    return s
