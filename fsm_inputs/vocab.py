"""Seeded synthetic vocabularies (token byte strings).

A vocabulary is a set of N strings over a fixed alphabet (paper Section 2); the
real tokenizer vocabularies the paper and its follow-ups use are not available
offline, so these generators produce byte strings with the same sizes and rough
length / byte statistics.  The arrays returned here are the contract: the same
arrays are handed to the CPU oracle and to the CUDA library.

Layout: ``vocab_bytes`` uint8 [total], ``vocab_offsets`` int32 [N+1] with
token v occupying ``vocab_bytes[offsets[v]:offsets[v+1]]``.
"""
from __future__ import annotations

import numpy as np

# Approximate English letter frequencies as integer weights (per 1000).
_LETTER_WEIGHTS = {
    "e": 127, "t": 91, "a": 82, "o": 75, "i": 70, "n": 67, "s": 63, "h": 61,
    "r": 60, "d": 43, "l": 40, "c": 28, "u": 28, "m": 24, "w": 24, "f": 22,
    "g": 20, "y": 20, "p": 19, "b": 15, "v": 10, "k": 8, "j": 2, "x": 2,
    "q": 1, "z": 1,
}
_LETTERS = np.frombuffer("".join(_LETTER_WEIGHTS).encode(), dtype=np.uint8)
_LETTER_P = np.array(list(_LETTER_WEIGHTS.values()), dtype=np.float64)
_LETTER_P /= _LETTER_P.sum()
_DIGIT_PUNCT = np.frombuffer(b"0123456789\"{}:,.-_ ", dtype=np.uint8)
_NUMERIC = np.frombuffer(b"0123456789.+-", dtype=np.uint8)
_PRINTABLE = np.arange(0x20, 0x7F, dtype=np.uint8)


def _pack(lengths: np.ndarray, flat: np.ndarray):
    offsets = np.zeros(len(lengths) + 1, dtype=np.int64)
    np.cumsum(lengths, out=offsets[1:])
    assert offsets[-1] == len(flat) and offsets[-1] < 2**31
    return np.ascontiguousarray(flat, dtype=np.uint8), offsets.astype(np.int32)


def numeric_mix_vocab(seed: int, N: int, zero_length_ids=()):
    """Lengths uniform on 1..8; each byte is, with probability 0.4, uniform over
    ``0123456789.+-`` and otherwise uniform over printable ASCII."""
    rng = np.random.default_rng(seed)
    lengths = rng.integers(1, 9, size=N, dtype=np.int64)
    lengths[list(zero_length_ids)] = 0
    total = int(lengths.sum())
    numeric = rng.random(total) < 0.4
    a = _NUMERIC[rng.integers(0, len(_NUMERIC), size=total)]
    b = _PRINTABLE[rng.integers(0, len(_PRINTABLE), size=total)]
    return _pack(lengths, np.where(numeric, a, b))


def bpe_like_vocab(seed: int, N: int, zero_length_ids=(), max_len: int = 16):
    """BPE-shaped tokens: length min(max_len, 1 + Geometric(0.25)) (mean 4 before
    the cap); 5 % of bytes from digits/punctuation, the rest lowercase letters by
    English frequency; the first byte is a space with probability 0.3."""
    rng = np.random.default_rng(seed)
    lengths = np.minimum(max_len, rng.geometric(0.25, size=N)).astype(np.int64)
    zl = np.asarray(list(zero_length_ids), dtype=np.int64)
    if zl.size:
        lengths[zl] = 0
    total = int(lengths.sum())
    other = rng.random(total) < 0.05
    a = _DIGIT_PUNCT[rng.integers(0, len(_DIGIT_PUNCT), size=total)]
    b = _LETTERS[rng.choice(len(_LETTERS), size=total, p=_LETTER_P)]
    flat = np.where(other, a, b)
    starts = np.zeros(N + 1, dtype=np.int64)
    np.cumsum(lengths, out=starts[1:])
    space_first = (rng.random(N) < 0.3) & (lengths > 0)
    flat[starts[:-1][space_first]] = 0x20
    return _pack(lengths, flat)


def vocab_from_strings(tokens):
    """Packs an explicit list of byte strings (used by the worked examples)."""
    tokens = [t.encode("latin-1") if isinstance(t, str) else bytes(t) for t in tokens]
    lengths = np.array([len(t) for t in tokens], dtype=np.int64)
    flat = np.frombuffer(b"".join(tokens), dtype=np.uint8).copy()
    return _pack(lengths, flat)


def token_bytes(vocab_bytes, vocab_offsets, v: int) -> bytes:
    return bytes(vocab_bytes[int(vocab_offsets[v]):int(vocab_offsets[v + 1])])
