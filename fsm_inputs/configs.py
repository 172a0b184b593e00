"""The five seeded synthetic workloads.

Each ``make_config(k)`` returns a ``Workload`` whose arrays are the inputs of
the index build (dense transition table, accept flags, packed vocabulary) plus
the decode-loop parameters where the workload has one.  Per-workload seed =
BASE_SEED + k; draw order inside each generator is fixed.

1. tiny       hand-built DFA for a signed decimal, N = 1,000, fp32, B = 1, 20 steps
2. llama2     N = 32,000 BPE-like tokens, JSON-object regex DFA (about 80 states)
3. llama3     N = 128,256, random DFA with 1,000 live states, 12 live classes each
4. large      N = 152,064, random DFA with 20,000 live states, 16 live classes each
5. decode     workload 3's index, B = 256 bf16 logits ~ N(0, variance 2), 1,000 steps
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field

import numpy as np

from .dfa import random_class_dfa, signed_decimal_dfa
from .regex_dfa import DFA, compile_regex
from .vocab import bpe_like_vocab, numeric_mix_vocab

BASE_SEED = 230709702

_STR = r'"[^"\\\x00-\x1f]*"'
_INT = r"-?(0|[1-9][0-9]*)"
JSON_OBJECT_REGEX = (
    r'\{"first_name": ' + _STR + r', "home_city": ' + _STR + r', "email": ' + _STR
    + r', "age": ' + _INT + r', "score": ' + _INT + r"\.[0-9]+\}"
)


@dataclass
class Workload:
    name: str
    seed: int
    dfa: DFA
    vocab_bytes: np.ndarray
    vocab_offsets: np.ndarray
    eos_id: int
    B: int = 0
    steps: int = 0
    logits_dtype: str = ""
    logits_sigma: float = 1.0
    extra: dict = field(default_factory=dict)

    @property
    def Q(self) -> int:
        return self.dfa.Q

    @property
    def N(self) -> int:
        return int(len(self.vocab_offsets) - 1)

    @property
    def W(self) -> int:
        return (self.N + 31) // 32

    def sha256(self) -> dict:
        h = lambda a: hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()[:16]
        return {"trans": h(self.dfa.trans), "accept": h(self.dfa.accept),
                "vocab_bytes": h(self.vocab_bytes), "vocab_offsets": h(self.vocab_offsets)}


def make_config(k: int) -> Workload:
    seed = BASE_SEED + k
    if k == 1:
        vb, vo = numeric_mix_vocab(seed, 1000, zero_length_ids=[999])
        return Workload("tiny", seed, signed_decimal_dfa(), vb, vo, eos_id=999,
                        B=1, steps=20, logits_dtype="f32", logits_sigma=1.0)
    if k == 2:
        vb, vo = bpe_like_vocab(seed, 32000, zero_length_ids=[0, 1, 2])
        return Workload("llama2_json", seed, compile_regex(JSON_OBJECT_REGEX), vb, vo, eos_id=2)
    if k in (3, 5):
        s3 = BASE_SEED + 3
        N = 128256
        vb, vo = bpe_like_vocab(s3, N, zero_length_ids=range(N - 256, N))
        dfa, _ = random_class_dfa(s3 + 1000, 1000, 64, 12, 0.10)
        if k == 3:
            return Workload("llama3_random1k", s3, dfa, vb, vo, eos_id=128001)
        return Workload("decode_b256", seed, dfa, vb, vo, eos_id=128001, B=256, steps=1000,
                        logits_dtype="bf16", logits_sigma=float(np.sqrt(2.0)))
    if k == 4:
        N = 152064
        vb, vo = bpe_like_vocab(seed, N, zero_length_ids=range(N - 421, N))
        dfa, _ = random_class_dfa(seed + 1000, 20000, 64, 16, 0.10)
        return Workload("large_random20k", seed, dfa, vb, vo, eos_id=151643)
    raise ValueError(f"no workload {k}")


def start_states(w: Workload) -> np.ndarray:
    """Starting states of the decode loop: uniform over the live states."""
    rng = np.random.default_rng(w.seed + 77)
    if w.B == 1:
        return np.zeros(1, dtype=np.int32)
    return rng.integers(0, w.Q - 1, size=w.B).astype(np.int32)


def step_logits_numpy(w: Workload, step: int, N: int | None = None) -> np.ndarray:
    """fp32 logits [B, N] for one decode step, drawn on the host."""
    rng = np.random.default_rng([w.seed, 9, step])
    return (rng.standard_normal((w.B, N or w.N), dtype=np.float32) * np.float32(w.logits_sigma))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns
    (input conversion only; finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)
