"""Host-side checks that need no GPU: the library loads, exports every symbol the
header declares, sizes its workspace, and rejects bad arguments before launching."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def fg():
    from paper_2307_09702_b200 import build as b
    b.build()
    import paper_2307_09702_b200 as fg
    return fg


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fsmguide.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:fsm|guided)_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(fg):
    names = declared_functions()
    assert {"fsm_index_build", "guided_mask_step", "fsm_index_build_rows"} <= set(names)
    L = ctypes.CDLL(fg.library_path())
    for n in names:
        assert hasattr(L, n), n
        assert hasattr(fg, n), f"binding lacks {n}"


def test_the_range_checked_library_is_built_and_exports_the_same_symbols(fg):
    from paper_2307_09702_b200 import binding, build as b
    assert os.path.exists(b.CHECKED_LIB_PATH) and b.CHECKED_LIB_PATH != fg.library_path()
    L = ctypes.CDLL(b.CHECKED_LIB_PATH)
    for n in declared_functions():
        assert hasattr(L, n), n
    try:
        assert binding.select_library(True) == b.CHECKED_LIB_PATH
        assert fg.fsm_debug_set(7, 5) == 0 and fg.fsm_debug_set(7, 0) == 5
    finally:
        binding.select_library(False)
    assert fg.library_path().endswith("libfsmguide.so")


def test_status_strings(fg):
    assert fg.fsm_status_string(0) == "FSM_OK"
    for code in range(-8, 0):
        assert fg.fsm_status_string(code).startswith("FSM_ERR_")
    assert fg.fsm_status_string(-99) == "FSM_ERR_UNKNOWN"


def test_workspace_query(fg):
    assert fg.fsm_index_workspace_bytes(0, 10, 10) == 0
    assert fg.fsm_index_workspace_bytes(10, 0, 10) == 0
    a = fg.fsm_index_workspace_bytes(1001, 128256, 505341)
    b = fg.fsm_index_workspace_bytes(20001, 152064, 601443)
    c = fg.fsm_index_workspace_bytes(70000, 152064, 601443)
    assert 0 < a < b < c < 512 << 20 and a % 256 == 0


def test_index_build_rejects_bad_arguments_before_any_launch(fg):
    ws = fg.fsm_index_workspace_bytes(10, 100, 400)
    ok = dict(dfa_trans=0x1000, accept=0x2000, vocab_bytes=0x3000, vocab_offsets=0x4000,
              vocab_nbytes=400, Q=10, N=100, dead_state=9, eos_id=-1, allowed_mask=0x5000,
              next_state=0x6000, state_dtype=0, workspace=0x10000, workspace_bytes=ws,
              status_word=None, stream=0)

    def call(**kw):
        a = dict(ok, **kw)
        return fg.fsm_index_build(*[a[k] for k in ok])

    assert call(Q=0) == -2 and call(N=-1) == -2
    assert call(dfa_trans=None) == -1 and call(allowed_mask=None) == -1
    assert call(state_dtype=2) == -4 and call(state_dtype=1, Q=70000, dead_state=0) == -4
    assert call(dead_state=10) == -6 and call(eos_id=100) == -6 and call(eos_id=-2) == -6
    assert call(allowed_mask=0x5002) == -3 and call(next_state=0x6002) == -3
    assert call(workspace=None) == -5 and call(workspace_bytes=ws - 1) == -5
    assert call(workspace=0x10010) == -3
    rows = dict(ok)
    args = [rows[k] for k in ok]
    bad_rows = args[:9] + [5, 3] + args[9:]
    assert fg.fsm_index_build_rows(*bad_rows) == -6
    import torch
    if not torch.cuda.is_available():
        assert call() in (-7, -8)          # valid arguments, but no usable device


def test_mask_step_rejects_bad_arguments(fg):
    ok = dict(logits_in=0x1000, logits_out=0x1000, logits_dtype=1, row_stride=128, states=0x2000,
              finished=0x3000, tokens_out=0x4000, allowed_mask=0x5000, next_state=0x6000,
              state_dtype=0, Q=10, N=128, B=4, dead_state=9, eos_id=3, status_word=None, stream=0)

    def call(**kw):
        a = dict(ok, **kw)
        return fg.guided_mask_step(*[a[k] for k in ok])

    assert call(row_stride=100) == -2 and call(B=-1) == -2
    assert call(states=None) == -1 and call(next_state=None) == -1
    assert call(logits_dtype=3) == -4
    assert call(logits_in=0x1008) == -3 and call(row_stride=129) == -3
    assert call(eos_id=128) == -6
    assert call(B=0) == 0


def test_debug_knobs(fg):
    assert fg.fsm_debug_set(99, 1) == -6
    assert fg.fsm_debug_set(2, 4) == 0 and fg.fsm_debug_set(2, 0) == 4
