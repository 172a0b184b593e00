"""TEST INFRASTRUCTURE: ctypes front end of the C oracle (``fsm_oracle.c``).

Argument marshalling only; every value is computed by the C file.  The shared
object is compiled with gcc on first use (or by ``build()``)."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fsm_oracle.c")
_LIB = os.path.join(_HERE, "libfsm_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compiles the oracle with gcc; returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-std=c11", "-Wall", "-Wextra", "-shared",
                               "-fPIC", "-ffp-contract=off", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.c_void_p
        i32, i64 = ctypes.c_int32, ctypes.c_int64
        lib.oracle_index_build.argtypes = [p, p, p, p, i32, i32, i32, i32, i32, i32, p, p, p, i32]
        lib.oracle_index_build.restype = ctypes.c_int
        lib.oracle_mask_step.argtypes = [p, p, i32, i64, p, p, p, p, p, i32, i32, i32, i32, i32, i32]
        lib.oracle_mask_step.restype = ctypes.c_int
        lib.oracle_sample_step.argtypes = [p, p, i32, i64, p, p, p, p, p, i32, i32, i32, i32, i32,
                                           ctypes.c_float, ctypes.c_uint64, ctypes.c_uint64, i32]
        lib.oracle_sample_step.restype = ctypes.c_int
        lib.oracle_philox4x32_10.argtypes = [p, p, p]
        lib.oracle_philox4x32_10.restype = None
        lib.oracle_ln_f32.argtypes = [ctypes.c_float]
        lib.oracle_ln_f32.restype = ctypes.c_float
        lib.oracle_gumbel_f32.argtypes = [ctypes.c_uint32]
        lib.oracle_gumbel_f32.restype = ctypes.c_float
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def index_build(trans, accept, vocab_bytes, vocab_offsets, dead_state, eos_id=-1,
                q_begin=0, q_end=None, want_next=True, threads=1):
    """Returns ``(allowed_mask uint32 [rows, W], next_state int32 [rows, N] or None,
    lookups)`` for rows ``q_begin..q_end-1``; ``lookups`` is the number of
    transition-table evaluations made by walks that stop at the dead state."""
    trans = _c(trans, np.int32)
    accept = _c(accept, np.uint8)
    vocab_bytes = _c(vocab_bytes, np.uint8)
    vocab_offsets = _c(vocab_offsets, np.int32)
    Q = trans.shape[0]
    assert trans.shape == (Q, 256) and accept.shape == (Q,)
    N = len(vocab_offsets) - 1
    q_end = Q if q_end is None else q_end
    rows = q_end - q_begin
    W = (N + 31) // 32
    mask = np.empty((rows, W), dtype=np.uint32)
    nxt = np.empty((rows, N), dtype=np.int32) if want_next else None
    lookups = np.zeros(1, dtype=np.int64)
    if vocab_bytes.size == 0:
        vocab_bytes = np.zeros(1, dtype=np.uint8)
    rc = _load().oracle_index_build(_ptr(trans), _ptr(accept), _ptr(vocab_bytes), _ptr(vocab_offsets),
                                    Q, N, dead_state, eos_id, q_begin, q_end,
                                    _ptr(mask), _ptr(nxt), _ptr(lookups), threads)
    if rc != 0:
        raise ValueError(f"oracle_index_build failed with {rc}")
    return mask, nxt, int(lookups[0])


def mask_step(logits, states, finished, allowed_mask, next_state, dead_state, eos_id,
              write_logits=True, threads=1):
    """One masked greedy step.  ``logits`` is float32 [B, N] or uint16 [B, N]
    (bf16 bit patterns).  ``states`` (int32 [B]) and ``finished`` (uint8 [B]) are
    updated in place.  Returns ``(tokens int32 [B], masked logits or None)``."""
    assert logits.ndim == 2 and logits.flags.c_contiguous
    if logits.dtype == np.float32:
        dtype = 0
    elif logits.dtype == np.uint16:
        dtype = 1
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    B, N = logits.shape
    allowed_mask = _c(allowed_mask, np.uint32)
    next_state = _c(next_state, np.int32)
    Q = allowed_mask.shape[0]
    assert allowed_mask.shape == (Q, (N + 31) // 32) and next_state.shape == (Q, N)
    assert states.dtype == np.int32 and finished.dtype == np.uint8
    assert states.flags.c_contiguous and finished.flags.c_contiguous
    out = np.empty_like(logits) if write_logits else None
    if out is not None:
        out[...] = logits          # rows of finished sequences are left as they were
    tokens = np.empty(B, dtype=np.int32)
    rc = _load().oracle_mask_step(_ptr(logits), _ptr(out), dtype, N, _ptr(states), _ptr(finished),
                                  _ptr(tokens), _ptr(allowed_mask), _ptr(next_state),
                                  Q, N, B, dead_state, eos_id, threads)
    if rc != 0:
        raise ValueError(f"oracle_mask_step failed with {rc}")
    return tokens, out


def sample_step(logits, states, finished, allowed_mask, next_state, dead_state, eos_id,
                inv_temperature, seed, draw, write_logits=True, threads=1):
    """One masked sampling step (categorical draw by Gumbel-max with Philox bits).
    Same conventions as ``mask_step``; ``seed`` and ``draw`` are 64-bit integers."""
    assert logits.ndim == 2 and logits.flags.c_contiguous
    if logits.dtype == np.float32:
        dtype = 0
    elif logits.dtype == np.uint16:
        dtype = 1
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    B, N = logits.shape
    allowed_mask = _c(allowed_mask, np.uint32)
    next_state = _c(next_state, np.int32)
    Q = allowed_mask.shape[0]
    assert allowed_mask.shape == (Q, (N + 31) // 32) and next_state.shape == (Q, N)
    assert states.dtype == np.int32 and finished.dtype == np.uint8
    out = np.empty_like(logits) if write_logits else None
    if out is not None:
        out[...] = logits
    tokens = np.empty(B, dtype=np.int32)
    rc = _load().oracle_sample_step(_ptr(logits), _ptr(out), dtype, N, _ptr(states), _ptr(finished),
                                    _ptr(tokens), _ptr(allowed_mask), _ptr(next_state),
                                    Q, N, B, dead_state, eos_id, float(np.float32(inv_temperature)),
                                    seed & 0xFFFFFFFFFFFFFFFF, draw & 0xFFFFFFFFFFFFFFFF, threads)
    if rc != 0:
        raise ValueError(f"oracle_sample_step failed with {rc}")
    return tokens, out


def philox4x32_10(ctr, key):
    """Philox4x32-10 block: ``ctr`` four and ``key`` two 32-bit words -> four words."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return [int(x) for x in out]


def ln_f32(x: float) -> float:
    return float(_load().oracle_ln_f32(float(np.float32(x))))


def gumbel_f32(bits: int) -> float:
    return float(_load().oracle_gumbel_f32(bits & 0xFFFFFFFF))


def index_csr(trans, accept, vocab_bytes, vocab_offsets, dead_state, eos_id=-1, threads=1):
    """The index in the paper's own form - sigma: state -> set of allowed tokens - as
    compressed rows: ``(allowed_mask, row_offsets int64 [Q+1], tokens int32 [nnz],
    next int32 [nnz])`` with row q's allowed tokens in increasing id order at
    ``row_offsets[q] .. row_offsets[q+1]-1`` and the state each one leads to beside it.
    Written out from the dense definition: an entry for every set bit, nothing else."""
    mask, nxt, _ = index_build(trans, accept, vocab_bytes, vocab_offsets, dead_state, eos_id,
                               threads=threads)
    Q, N = nxt.shape
    offsets = np.zeros(Q + 1, dtype=np.int64)
    toks, nexts = [], []
    for q in range(Q):
        bits = np.unpackbits(mask[q].view(np.uint8), bitorder="little")[:N]
        ids = np.flatnonzero(bits).astype(np.int32)
        toks.append(ids)
        nexts.append(nxt[q, ids])
        offsets[q + 1] = offsets[q] + len(ids)
    tokens = np.concatenate(toks) if toks else np.zeros(0, np.int32)
    nexts = np.concatenate(nexts).astype(np.int32) if nexts else np.zeros(0, np.int32)
    return mask, offsets, tokens, nexts
