"""GPU parity of fsm_index_row_alias against the CPU oracle (``oracle/row_alias.py``): the
alias map is an integer result and is compared exactly."""
import numpy as np
import pytest
import torch

from fsm_inputs import bpe_like_vocab, make_config, paper_float_example_dfa, random_class_dfa, vocab_from_strings
from oracle import fsm_oracle
from oracle.row_alias import row_alias

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from gpu_util import THREADS, gpu_index, mask_np, next_np


@pytest.fixture(autouse=True)
def _reset_knobs():
    yield
    fg.fsm_debug_set(1, 0)


def gpu_alias(mask_t, next_t, state_dtype, Q, N):
    dev = mask_t.device
    alias = torch.full((Q,), -9, dtype=torch.int32, device=dev)
    n_unique = torch.full((1,), -9, dtype=torch.int32, device=dev)
    wsb = fg.fsm_row_alias_workspace_bytes(Q)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = fg.fsm_index_row_alias(mask_t, next_t, state_dtype, Q, N, alias, n_unique, ws, wsb, status)
    assert rc == 0, fg.fsm_status_string(rc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return alias.cpu().numpy(), int(n_unique.item())


def check(trans, accept, vb, vo, dead, eos, modes=("i32", "u16", "mask")):
    """Builds the index on the GPU, merges its rows on the GPU and compares with the oracle's
    merge of the oracle's index."""
    Q, N = trans.shape[0], len(vo) - 1
    o_mask, o_next, _ = fsm_oracle.index_build(trans, accept, vb, vo, dead, eos, threads=THREADS)
    out = {}
    for mode in modes:
        sd = fg.FSM_STATE_U16 if mode == "u16" else fg.FSM_STATE_I32
        idx = gpu_index(trans, accept, vb, vo, dead, eos, sd, mode != "mask")
        want, n_want = row_alias(o_mask, None if mode == "mask" else o_next)
        for weak in (0, 1):
            if weak and Q > 400:
                continue                      # (every row meets every other: quadratic)
            fg.fsm_debug_set(1, weak)
            got, n_got = gpu_alias(idx.allowed_mask, idx.next_state, sd, Q, N)
            fg.fsm_debug_set(1, 0)
            assert (got == want).all(), (mode, weak, np.flatnonzero(got != want)[:5])
            assert n_got == n_want
        out[mode] = (want, n_want)
    return out


def with_clones(d, clones):
    """Appends copies of the given states (same outgoing transitions and acceptance)."""
    trans = np.concatenate([d.trans] + [d.trans[s:s + 1] for s in clones], axis=0)
    accept = np.concatenate([d.accept] + [d.accept[s:s + 1] for s in clones])
    return trans, accept


def test_paper_example_rows_merge_on_the_gpu():
    d = paper_float_example_dfa()
    vb, vo = vocab_from_strings(["A", ".", "42", ".2", "1"])
    out = check(d.trans, d.accept, vb, vo, d.dead, -1)
    assert out["i32"][0].tolist() == [0, 0, 2, 2, 4] and out["mask"][1] == 3


@pytest.mark.parametrize("k", [1, 2])
def test_small_workloads_and_their_clones(k):
    w = make_config(k)
    d = w.dfa
    check(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    trans, accept = with_clones(d, [0, 3, 3, d.Q - 2, 1, 0])
    out = check(trans, accept, w.vocab_bytes, w.vocab_offsets, d.dead, -1)   # no EOS: clones are exact copies
    alias = out["i32"][0]
    assert alias[d.Q] == alias[0] and alias[d.Q + 1] == alias[3] and alias[d.Q + 2] == alias[3]
    assert alias[d.Q + 5] == alias[0]


@pytest.mark.parametrize("N", [1, 31, 33, 1001, 4099])
def test_ragged_and_odd_vocabulary_sizes(N):
    """Odd N: rows of 16-bit states start at every alignment, which the row hash must not see."""
    rng = np.random.default_rng(N)
    d, _ = random_class_dfa(N, n_live=37, n_classes=9, live_classes_per_state=5)
    toks = [bytes(rng.integers(97, 110, size=rng.integers(0, 5)).tolist()) for _ in range(N)]
    vb, vo = vocab_from_strings(toks)
    trans, accept = with_clones(d, [5, 6, 5, 20, 36, 0, 7])
    out = check(trans, accept, vb, vo, d.dead, -1)
    alias = out["u16"][0]
    assert alias[d.Q] == alias[5] and alias[d.Q + 2] == alias[5] and alias[d.Q + 1] == alias[6]


def test_workload_3_with_a_tenth_of_its_states_cloned():
    w = make_config(3)
    d = w.dfa
    rng = np.random.default_rng(3)
    clones = rng.integers(0, d.Q - 1, size=100).tolist()
    trans, accept = with_clones(d, clones)
    out = check(trans, accept, w.vocab_bytes, w.vocab_offsets, d.dead, -1, modes=("i32", "u16"))
    alias, n = out["i32"]
    assert n <= d.Q and all(alias[d.Q + j] == alias[s] for j, s in enumerate(clones))


def test_argument_errors():
    assert fg.fsm_row_alias_workspace_bytes(0) == 0 and fg.fsm_row_alias_workspace_bytes(1000) > 0
    assert fg.fsm_index_row_alias(None, None, 0, 5, 5, 0x100, 0x100, 0x100, 1 << 20) == -1
    assert fg.fsm_index_row_alias(0x100, None, 0, 0, 5, 0x100, 0x100, 0x100, 1 << 20) == -2
    assert fg.fsm_index_row_alias(0x100, None, 7, 5, 5, 0x100, 0x100, 0x100, 1 << 20) == -4
    assert fg.fsm_index_row_alias(0x100, None, 0, 5, 5, 0x100, 0x100, 0x100, 16) == -5
    assert fg.fsm_index_row_alias(0x102, None, 0, 5, 5, 0x100, 0x100, 0x100, 1 << 20) == -3
