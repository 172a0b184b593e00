"""The range-checked build of the library (``-DFSM_CHECKED``) on the parity cases, and the
give-up path of the bounded waits.

In the checked build every index that a kernel computes from data it has read (a token id
out of a sorted record, a state out of the table, a position out of a counter or a prefix
sum) is compared with the size of the array it goes into; a violation raises
``FSM_FLAG_INDEX`` and the access is skipped.  The cases below must give the oracle's
result with a clean status word: no kernel reaches outside its arrays on them.

The give-up path is exercised without making any copy fail: after its table has arrived, the
walk kernel waits (a bounded number of polls) on a completion that nothing signals, raises
``FSM_FLAG_WAIT_TIMEOUT`` and returns; the next build on the same context is exact again."""
import numpy as np
import pytest
import torch

from fsm_inputs import (bpe_like_vocab, compile_regex, make_config, paper_float_example_dfa,
                        random_class_dfa, vocab_from_strings)
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200 import binding
    from gpu_util import THREADS, check_index, gpu_index, mask_np
    from test_gpu_csr import check_csr
    from test_gpu_mask_step import run_case

KNOBS = (1, 2, 3, 4, 6, 7)


@pytest.fixture
def checked():
    path = binding.select_library(True)
    assert path.endswith("libfsmguide_checked.so")
    assert fg.fsm_device_check() == 0
    yield
    for key in KNOBS:
        fg.fsm_debug_set(key, 0)
    binding.select_library(False)


@pytest.fixture(params=[1, 2, 3], ids=["dense", "rowwise", "bucket"])
def walk_algorithm(request, checked):
    fg.fsm_debug_set(6, request.param)
    return request.param


def test_checked_library_is_a_separate_image(checked):
    import ctypes
    assert binding.library_path().endswith("_checked.so")
    # a knob set here does not show in the regular library
    fg.fsm_debug_set(6, 3)
    binding.select_library(False)
    assert fg.fsm_debug_set(6, 0) == 0
    binding.select_library(True)
    assert fg.fsm_debug_set(6, 0) == 3


def test_small_workloads_under_the_checked_build(walk_algorithm):
    d = paper_float_example_dfa()
    vb, vo = vocab_from_strings(["A", ".", "42", ".2", "1"])
    check_index(d.trans, d.accept, vb, vo, d.dead)
    for k in (1, 2):
        w = make_config(k)
        check_index(w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)


@pytest.mark.parametrize("N", [1, 31, 33, 1025])
def test_ragged_vocabularies_under_the_checked_build(walk_algorithm, N):
    rng = np.random.default_rng(N)
    d, _ = random_class_dfa(N, n_live=37, n_classes=9, live_classes_per_state=5)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(0, 7)).tolist()) for _ in range(N)]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead, eos=N - 1)


def test_extreme_cases_under_the_checked_build(walk_algorithm):
    # tokens longer than the records cover
    d = compile_regex(r"(ab)*c?")
    toks = [b"ab" * 7 + b"a", b"ab" * 8, b"ab" * 8 + b"c", b"ab" * 20, b"ab" * 19 + b"cc",
            b"ab" * 8 + b"x", b"", b"ab" * 100 + b"c"]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead)
    # a state that reads everything over a large vocabulary: more chunks than the row-wise
    # walk keeps descriptors for
    w = make_config(3)
    trans = np.full((3, 256), 2, dtype=np.int32)
    trans[0, :] = 0
    trans[1, 97:123] = 0
    check_index(trans, np.array([1, 0, 0], dtype=np.uint8), w.vocab_bytes, w.vocab_offsets, 2, w.eos_id)
    # more than 127 byte classes: one-level buckets, plain row table
    d, _ = random_class_dfa(33, n_live=300, n_classes=220, live_classes_per_state=60)
    rng = np.random.default_rng(2)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(0, 6)).tolist()) for _ in range(5000)]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead, eos=77)
    # row ranges
    w2 = make_config(2)
    for (a, b) in [(0, 1), (33, 65)]:
        check_index(w2.dfa.trans, w2.dfa.accept, w2.vocab_bytes, w2.vocab_offsets, w2.dfa.dead, w2.eos_id,
                    q_begin=a, q_end=b)


def test_more_rows_than_sms_under_the_checked_build(walk_algorithm):
    """300 states x 20,000 tokens: the size at which the automatic choice takes the
    work-avoiding walks, with the table in shared memory and then through the cache."""
    d, _ = random_class_dfa(300, n_live=300, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 20_000, zero_length_ids=(19_999,))
    check_index(d.trans, d.accept, vb, vo, d.dead, 19_999)
    fg.fsm_debug_set(4, 40 * 1024)   # the table no longer fits the shared-memory budget
    check_index(d.trans, d.accept, vb, vo, d.dead, 19_999, modes=("u16", "mask"))


def test_data_faults_and_fallbacks_under_the_checked_build(walk_algorithm):
    w = make_config(1)
    d = w.dfa
    t = d.trans.copy()
    t[0, 48:53] = 99
    t[2, 55] = -7
    clamped = t.copy()
    clamped[(t < 0) | (t >= d.Q)] = d.dead
    check_index(t, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id, expect_status=1,
                oracle_trans=clamped, modes=("i32",))
    w2 = make_config(2)
    N = 3000
    vo = w2.vocab_offsets[:N + 1]
    vb = w2.vocab_bytes[:vo[-1]]
    fg.fsm_debug_set(1, 1)           # forced hash collision: the uncompressed walk
    check_index(w2.dfa.trans, w2.dfa.accept, vb, vo, w2.dfa.dead, 2, expect_status=8, modes=("i32", "mask"))


def test_decode_steps_under_the_checked_build(checked):
    rng = np.random.default_rng(5)
    for dtype in ("bf16", "f32"):
        for N in (7, 33, 1000, 4099):
            pad = (-N) % 8           # rows start on 16-byte boundaries
            run_case(rng, 17, N, 9, dtype, "inplace", k=0, stride_pad=pad)
            run_case(rng, 17, N, 9, dtype, "outofplace", k=2, stride_pad=pad, sample=(2.0, 11, 3))
    run_case(rng, 40, 32_000, 12, "bf16", "inplace", k=4, state_dtype=1, sample=(10.0, 7, 1))
    run_case(rng, 40, 32_003, 12, "bf16", "select", k=8, stride_pad=5)


def test_compressed_rows_under_the_checked_build(walk_algorithm):
    for k in (1, 2):
        w = make_config(k)
        check_csr(w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)
    d, _ = random_class_dfa(300, n_live=300, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 5_000, zero_length_ids=(4_999,))
    check_csr(d.trans, d.accept, vb, vo, d.dead, 4_999)


# ---------------------------------------------------------------------------------------
# the give-up path of the bounded waits (regular library and checked library alike)

@pytest.mark.parametrize("use_checked", [False, True], ids=["regular", "checked"])
@pytest.mark.parametrize("algo,want_next", [(1, True), (2, True), (3, False)],
                         ids=["dense", "rowwise", "bucket"])
def test_a_wait_that_nothing_ends_gives_up_and_the_context_stays_usable(use_checked, algo, want_next):
    binding.select_library(use_checked)
    try:
        d, _ = random_class_dfa(300, n_live=300, n_classes=40, live_classes_per_state=9)
        vb, vo = bpe_like_vocab(7, 5_000, zero_length_ids=(4_999,))
        fg.fsm_debug_set(6, algo)
        fg.fsm_debug_set(7, 64)      # polls before the wait gives up
        idx = gpu_index(d.trans, d.accept, vb, vo, d.dead, 4_999, want_next=want_next)   # returns: no spin
        assert int(idx.status.item()) & binding.FSM_FLAG_WAIT_TIMEOUT
        assert torch.cuda.current_stream().query()           # nothing left running
        fg.fsm_debug_set(7, 0)
        check_index(d.trans, d.accept, vb, vo, d.dead, 4_999,
                    modes=("i32", "mask") if want_next else ("mask",))
    finally:
        for key in KNOBS:
            fg.fsm_debug_set(key, 0)
        binding.select_library(False)
