"""ctypes binding of the fsmguide C ABI: argument marshalling only.

Functions carry the names of ``include/fsmguide.h``.  Array arguments are torch
CUDA tensors (or ``None`` where the header allows NULL); their ``data_ptr()`` is
passed through, the current torch CUDA stream is used unless ``stream`` is given.
Every computation happens in the library's kernels.
"""
from __future__ import annotations

import ctypes
import os

import torch

FSM_STATE_I32, FSM_STATE_U16 = 0, 1
FSM_LOGITS_F32, FSM_LOGITS_BF16 = 0, 1
FSM_DEBUG_WEAK_HASH, FSM_TUNE_MASK_CLUSTER, FSM_TUNE_WALK_CTAS, FSM_TUNE_SMEM_TABLE_BYTES = 1, 2, 3, 4
FSM_PROFILE_WALK = 5
FSM_TUNE_WALK_ALGO = 6
FSM_DEBUG_WAIT_PROBE = 7
FSM_STATIC_SCRATCH_BYTES = 2 << 20
FSM_FLAG_TRANS_RANGE, FSM_FLAG_OFFSETS, FSM_FLAG_STATE_RANGE = 1, 2, 4
FSM_FLAG_CLASS_SPLIT, FSM_FLAG_WAIT_TIMEOUT = 8, 16
FSM_FLAG_CSR_OVERFLOW, FSM_FLAG_INDEX = 32, 64
FSM_INDEX_DENSE, FSM_INDEX_BITMASK, FSM_INDEX_CSR = 0, 1, 2
FSM_ERR_IO, FSM_ERR_FORMAT = -9, -10


class IndexDesc(ctypes.Structure):
    """``fsm_index_desc`` of the header, field for field."""
    _fields_ = [("form", ctypes.c_int32), ("Q", ctypes.c_int32), ("N", ctypes.c_int32),
                ("state_dtype", ctypes.c_int32), ("dead_state", ctypes.c_int32),
                ("eos_id", ctypes.c_int32), ("nnz", ctypes.c_int64),
                ("input_digest", ctypes.c_uint8 * 32),
                ("allowed_mask", ctypes.c_void_p), ("next_state", ctypes.c_void_p),
                ("row_offsets", ctypes.c_void_p), ("csr_tokens", ctypes.c_void_p),
                ("csr_next", ctypes.c_void_p)]

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libfsmguide.so")
_lib = None


class FsmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {fsm_status_string(code)}")


def library_path() -> str:
    return _LIB_PATH


def select_library(checked: bool) -> str:
    """Switches every later call to the range-checked build of the library (``checked``) or
    back to the regular one.  The two are separate images: knobs set through
    ``fsm_debug_set`` belong to the library they were set in."""
    global _lib, _LIB_PATH
    _LIB_PATH = os.path.join(_PKG, "libfsmguide_checked.so" if checked else "libfsmguide.so")
    _lib = None
    return _LIB_PATH


def lib() -> ctypes.CDLL:
    """Loads ``libfsmguide.so``; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2307_09702_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.fsm_status_string.argtypes = [ctypes.c_int]
        L.fsm_status_string.restype = ctypes.c_char_p
        L.fsm_device_check.argtypes = []
        L.fsm_device_check.restype = ctypes.c_int
        L.fsm_debug_set.argtypes = [i32, i32]
        L.fsm_debug_set.restype = ctypes.c_int
        L.fsm_profile_read.argtypes = [vp, i32]
        L.fsm_profile_read.restype = ctypes.c_int
        L.fsm_index_workspace_bytes.argtypes = [i32, i32, i64]
        L.fsm_index_workspace_bytes.restype = sz
        L.fsm_index_build.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, i32, vp, sz, vp, vp]
        L.fsm_index_build.restype = ctypes.c_int
        L.fsm_index_build_rows.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, i32, i32, i32, vp, vp,
                                           i32, vp, sz, vp, vp]
        L.fsm_index_build_rows.restype = ctypes.c_int
        L.fsm_index_build_static.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, i32, vp, vp]
        L.fsm_index_build_static.restype = ctypes.c_int
        L.guided_mask_step.argtypes = [vp, vp, i32, i64, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32,
                                       i32, vp, vp]
        L.guided_mask_step.restype = ctypes.c_int
        L.guided_sample_step.argtypes = [vp, vp, i32, i64, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32,
                                         i32, ctypes.c_float, ctypes.c_uint64, ctypes.c_uint64, vp, vp]
        L.guided_sample_step.restype = ctypes.c_int
        L.fsm_index_build_csr.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, vp, i64,
                                          vp, sz, vp, vp]
        L.fsm_index_build_csr.restype = ctypes.c_int
        L.guided_step_csr.argtypes = [vp, vp, i32, i64, vp, vp, vp, vp, vp, vp, vp, i64, i32, i32, i32,
                                      i32, i32, i32, ctypes.c_float, ctypes.c_uint64, ctypes.c_uint64,
                                      vp, vp]
        L.guided_step_csr.restype = ctypes.c_int
        L.fsm_row_alias_workspace_bytes.argtypes = [i32]
        L.fsm_row_alias_workspace_bytes.restype = sz
        L.fsm_index_row_alias.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, sz, vp, vp]
        L.fsm_index_row_alias.restype = ctypes.c_int
        dp = ctypes.POINTER(IndexDesc)
        L.fsm_index_serialized_bytes.argtypes = [dp]
        L.fsm_index_serialized_bytes.restype = sz
        L.fsm_index_save.argtypes = [ctypes.c_char_p, dp, vp]
        L.fsm_index_save.restype = ctypes.c_int
        L.fsm_index_peek.argtypes = [ctypes.c_char_p, dp]
        L.fsm_index_peek.restype = ctypes.c_int
        L.fsm_index_load.argtypes = [ctypes.c_char_p, dp, vp]
        L.fsm_index_load.restype = ctypes.c_int
        L.fsm_sha256.argtypes = [vp, sz, vp]
        L.fsm_sha256.restype = ctypes.c_int
        L.fsm_checksum64.argtypes = [vp, sz, ctypes.c_uint64]
        L.fsm_checksum64.restype = ctypes.c_uint64
        L.fsm_index_input_digest.argtypes = [vp, vp, vp, vp, i64, i32, i32, i32, i32, vp, vp]
        L.fsm_index_input_digest.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def fsm_status_string(status: int) -> str:
    return lib().fsm_status_string(status).decode()


def fsm_device_check() -> int:
    return lib().fsm_device_check()


def fsm_debug_set(key: int, value: int) -> int:
    return lib().fsm_debug_set(key, value)


def fsm_profile_read(capacity: int = 4096):
    """Returns the walk-kernel durations (ms) recorded since the last read."""
    buf = (ctypes.c_float * capacity)()
    n = lib().fsm_profile_read(ctypes.cast(buf, ctypes.c_void_p), capacity)
    if n < 0:
        raise FsmError(n, "fsm_profile_read")
    return list(buf[:n])


def fsm_index_workspace_bytes(Q: int, N: int, vocab_nbytes: int) -> int:
    return lib().fsm_index_workspace_bytes(Q, N, vocab_nbytes)


def fsm_index_build(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state,
                    eos_id, allowed_mask, next_state, state_dtype, workspace, workspace_bytes,
                    status_word=None, stream=None) -> int:
    return lib().fsm_index_build(_ptr(dfa_trans), _ptr(accept), _ptr(vocab_bytes), _ptr(vocab_offsets),
                                 vocab_nbytes, Q, N, dead_state, eos_id, _ptr(allowed_mask),
                                 _ptr(next_state), state_dtype, _ptr(workspace), workspace_bytes,
                                 _ptr(status_word), _stream(stream))


def fsm_index_build_rows(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                         dead_state, eos_id, q_begin, q_end, allowed_mask, next_state, state_dtype,
                         workspace, workspace_bytes, status_word=None, stream=None) -> int:
    return lib().fsm_index_build_rows(_ptr(dfa_trans), _ptr(accept), _ptr(vocab_bytes),
                                      _ptr(vocab_offsets), vocab_nbytes, Q, N, dead_state, eos_id,
                                      q_begin, q_end, _ptr(allowed_mask), _ptr(next_state),
                                      state_dtype, _ptr(workspace), workspace_bytes,
                                      _ptr(status_word), _stream(stream))


def fsm_index_build_static(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                           dead_state, eos_id, allowed_mask, next_state, state_dtype,
                           status_word=None, stream=None) -> int:
    """Index build that takes its scratch from the library's built-in device array
    (``FSM_STATIC_SCRATCH_BYTES``) instead of a caller workspace; for callers that
    may not allocate device memory.  Same outputs as ``fsm_index_build``."""
    return lib().fsm_index_build_static(_ptr(dfa_trans), _ptr(accept), _ptr(vocab_bytes),
                                        _ptr(vocab_offsets), vocab_nbytes, Q, N, dead_state, eos_id,
                                        _ptr(allowed_mask), _ptr(next_state), state_dtype,
                                        _ptr(status_word), _stream(stream))


def guided_mask_step(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                     allowed_mask, next_state, state_dtype, Q, N, B, dead_state, eos_id,
                     status_word=None, stream=None) -> int:
    return lib().guided_mask_step(_ptr(logits_in), _ptr(logits_out), logits_dtype, row_stride,
                                  _ptr(states), _ptr(finished), _ptr(tokens_out), _ptr(allowed_mask),
                                  _ptr(next_state), state_dtype, Q, N, B, dead_state, eos_id,
                                  _ptr(status_word), _stream(stream))


def guided_sample_step(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                       allowed_mask, next_state, state_dtype, Q, N, B, dead_state, eos_id,
                       inv_temperature, seed, draw, status_word=None, stream=None) -> int:
    return lib().guided_sample_step(_ptr(logits_in), _ptr(logits_out), logits_dtype, row_stride,
                                    _ptr(states), _ptr(finished), _ptr(tokens_out),
                                    _ptr(allowed_mask), _ptr(next_state), state_dtype, Q, N, B,
                                    dead_state, eos_id, inv_temperature,
                                    seed & 0xFFFFFFFFFFFFFFFF, draw & 0xFFFFFFFFFFFFFFFF,
                                    _ptr(status_word), _stream(stream))


def fsm_index_build_csr(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state,
                        eos_id, allowed_mask, row_offsets, csr_tokens, csr_next, capacity, workspace,
                        workspace_bytes, status_word=None, stream=None) -> int:
    return lib().fsm_index_build_csr(_ptr(dfa_trans), _ptr(accept), _ptr(vocab_bytes),
                                     _ptr(vocab_offsets), vocab_nbytes, Q, N, dead_state, eos_id,
                                     _ptr(allowed_mask), _ptr(row_offsets), _ptr(csr_tokens),
                                     _ptr(csr_next), capacity, _ptr(workspace), workspace_bytes,
                                     _ptr(status_word), _stream(stream))


def guided_step_csr(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                    allowed_mask, row_offsets, csr_tokens, csr_next, capacity, Q, N, B, dead_state,
                    eos_id, sample=0, inv_temperature=1.0, seed=0, draw=0, status_word=None, stream=None) -> int:
    return lib().guided_step_csr(_ptr(logits_in), _ptr(logits_out), logits_dtype, row_stride,
                                 _ptr(states), _ptr(finished), _ptr(tokens_out), _ptr(allowed_mask),
                                 _ptr(row_offsets), _ptr(csr_tokens), _ptr(csr_next), capacity, Q, N,
                                 B, dead_state, eos_id, sample, inv_temperature,
                                 seed & 0xFFFFFFFFFFFFFFFF, draw & 0xFFFFFFFFFFFFFFFF,
                                 _ptr(status_word), _stream(stream))


def fsm_row_alias_workspace_bytes(Q: int) -> int:
    return lib().fsm_row_alias_workspace_bytes(Q)


def fsm_index_row_alias(allowed_mask, next_state, state_dtype, Q, N, row_alias, n_unique, workspace,
                        workspace_bytes, status_word=None, stream=None) -> int:
    return lib().fsm_index_row_alias(_ptr(allowed_mask), _ptr(next_state), state_dtype, Q, N,
                                     _ptr(row_alias), _ptr(n_unique), _ptr(workspace), workspace_bytes,
                                     _ptr(status_word), _stream(stream))


def index_desc(form, Q, N, dead_state, eos_id, state_dtype=0, nnz=0, input_digest=None,
               allowed_mask=None, next_state=None, row_offsets=None, csr_tokens=None,
               csr_next=None) -> IndexDesc:
    """Fills an ``fsm_index_desc`` (tensors become device pointers)."""
    d = IndexDesc(form, Q, N, state_dtype, dead_state, eos_id, nnz)
    if input_digest is not None:
        ctypes.memmove(d.input_digest, bytes(input_digest), 32)
    d.allowed_mask, d.next_state = _ptr(allowed_mask), _ptr(next_state)
    d.row_offsets, d.csr_tokens, d.csr_next = _ptr(row_offsets), _ptr(csr_tokens), _ptr(csr_next)
    return d


def fsm_index_serialized_bytes(desc: IndexDesc) -> int:
    return lib().fsm_index_serialized_bytes(ctypes.byref(desc))


def fsm_index_save(path: str, desc: IndexDesc, stream=None) -> int:
    return lib().fsm_index_save(os.fsencode(path), ctypes.byref(desc), _stream(stream))


def fsm_index_peek(path: str, desc: IndexDesc) -> int:
    return lib().fsm_index_peek(os.fsencode(path), ctypes.byref(desc))


def fsm_index_load(path: str, desc: IndexDesc, stream=None) -> int:
    return lib().fsm_index_load(os.fsencode(path), ctypes.byref(desc), _stream(stream))


def fsm_sha256(data: bytes) -> bytes:
    out = (ctypes.c_uint8 * 32)()
    buf = ctypes.create_string_buffer(data, len(data)) if len(data) else None
    rc = lib().fsm_sha256(ctypes.cast(buf, ctypes.c_void_p) if buf is not None else None, len(data),
                          ctypes.cast(out, ctypes.c_void_p))
    if rc != 0:
        raise FsmError(rc, "fsm_sha256")
    return bytes(out)


def fsm_checksum64(data: bytes, first_word_index: int = 0) -> int:
    buf = ctypes.create_string_buffer(data, len(data))
    return lib().fsm_checksum64(ctypes.cast(buf, ctypes.c_void_p), len(data), first_word_index)


def fsm_index_input_digest(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                           dead_state, eos_id, stream=None) -> bytes:
    out = (ctypes.c_uint8 * 32)()
    rc = lib().fsm_index_input_digest(_ptr(dfa_trans), _ptr(accept), _ptr(vocab_bytes),
                                      _ptr(vocab_offsets), vocab_nbytes, Q, N, dead_state, eos_id,
                                      ctypes.cast(out, ctypes.c_void_p), _stream(stream))
    if rc != 0:
        raise FsmError(rc, "fsm_index_input_digest")
    return bytes(out)


class GuidedIndex:
    """Holds the device buffers of one vocabulary index and forwards to the C ABI.

    Convenience for callers that keep an index around: allocation (torch), the
    two library calls, and the bookkeeping of shapes.  No arithmetic happens here.
    """

    def __init__(self, trans, accept, vocab_bytes, vocab_offsets, dead_state, eos_id=-1,
                 state_dtype=FSM_STATE_I32, want_next=True, device="cuda", q_begin=0, q_end=None):
        lib()
        dev = torch.device(device)
        self.Q, self.N = int(trans.shape[0]), int(len(vocab_offsets) - 1)
        self.W = (self.N + 31) // 32
        self.dead_state, self.eos_id, self.state_dtype = int(dead_state), int(eos_id), state_dtype
        self.q_begin, self.q_end = q_begin, self.Q if q_end is None else q_end
        as_dev = lambda a, dt: torch.as_tensor(a, dtype=dt).contiguous().to(dev)
        self.trans = as_dev(trans, torch.int32).reshape(self.Q, 256)
        self.accept = as_dev(accept, torch.uint8)
        self.vocab_nbytes = int(vocab_offsets[-1])
        vb = vocab_bytes if len(vocab_bytes) else [0]
        self.vocab_bytes = as_dev(vb, torch.uint8)
        self.vocab_offsets = as_dev(vocab_offsets, torch.int32)
        rows = self.q_end - self.q_begin
        self.allowed_mask = torch.empty((rows, self.W), dtype=torch.int32, device=dev)
        ndt = torch.int32 if state_dtype == FSM_STATE_I32 else torch.uint16
        self.next_state = torch.empty((rows, self.N), dtype=ndt, device=dev) if want_next else None
        self.workspace_bytes = fsm_index_workspace_bytes(self.Q, self.N, self.vocab_nbytes)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)

    def build(self, stream=None) -> "GuidedIndex":
        rc = fsm_index_build_rows(self.trans, self.accept, self.vocab_bytes, self.vocab_offsets,
                                  self.vocab_nbytes, self.Q, self.N, self.dead_state, self.eos_id,
                                  self.q_begin, self.q_end, self.allowed_mask, self.next_state,
                                  self.state_dtype, self.workspace, self.workspace_bytes, self.status,
                                  stream)
        if rc != 0:
            raise FsmError(rc, "fsm_index_build_rows")
        return self

    def _desc(self, digest) -> IndexDesc:
        if (self.q_begin, self.q_end) != (0, self.Q):
            raise ValueError("only a whole index is saved or loaded")
        dense = self.next_state is not None
        return index_desc(FSM_INDEX_DENSE if dense else FSM_INDEX_BITMASK, self.Q, self.N,
                          self.dead_state, self.eos_id, self.state_dtype if dense else 0, 0, digest,
                          self.allowed_mask, self.next_state)

    def input_digest(self, stream=None) -> bytes:
        return fsm_index_input_digest(self.trans, self.accept, self.vocab_bytes, self.vocab_offsets,
                                      self.vocab_nbytes, self.Q, self.N, self.dead_state, self.eos_id,
                                      stream)

    def save(self, path: str, stream=None) -> None:
        """Writes the built index to ``path`` (blocks)."""
        rc = fsm_index_save(path, self._desc(self.input_digest(stream)), stream)
        if rc != 0:
            raise FsmError(rc, "fsm_index_save")

    def load(self, path: str, stream=None) -> "GuidedIndex":
        """Fills the index from a file saved for the same inputs instead of building it
        (blocks); raises ``FsmError`` (``FSM_ERR_FORMAT``) when the file is for other inputs."""
        rc = fsm_index_load(path, self._desc(self.input_digest(stream)), stream)
        if rc != 0:
            raise FsmError(rc, "fsm_index_load")
        return self

    def step(self, logits, states, finished, tokens_out, logits_out="inplace", stream=None):
        """One masked greedy step on ``logits`` [B, >=N] (float32 or bfloat16)."""
        if logits.dtype == torch.float32:
            ldt = FSM_LOGITS_F32
        elif logits.dtype == torch.bfloat16:
            ldt = FSM_LOGITS_BF16
        else:
            raise TypeError("logits must be float32 or bfloat16")
        out = logits if isinstance(logits_out, str) else logits_out
        rc = guided_mask_step(logits, out, ldt, logits.stride(0), states, finished, tokens_out,
                              self.allowed_mask, self.next_state, self.state_dtype, self.Q, self.N,
                              logits.shape[0], self.dead_state, self.eos_id, self.status, stream)
        if rc != 0:
            raise FsmError(rc, "guided_mask_step")

    def sample(self, logits, states, finished, tokens_out, inv_temperature, seed, draw,
               logits_out="inplace", stream=None):
        """One masked sampling step (categorical draw) on ``logits`` [B, >=N]."""
        if logits.dtype == torch.float32:
            ldt = FSM_LOGITS_F32
        elif logits.dtype == torch.bfloat16:
            ldt = FSM_LOGITS_BF16
        else:
            raise TypeError("logits must be float32 or bfloat16")
        out = logits if isinstance(logits_out, str) else logits_out
        rc = guided_sample_step(logits, out, ldt, logits.stride(0), states, finished, tokens_out,
                                self.allowed_mask, self.next_state, self.state_dtype, self.Q, self.N,
                                logits.shape[0], self.dead_state, self.eos_id, inv_temperature, seed,
                                draw, self.status, stream)
        if rc != 0:
            raise FsmError(rc, "guided_sample_step")
