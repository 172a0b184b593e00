"""GPU parity of fsm_index_build against the CPU oracle: bit-exact bitmask and
next-state table, through the C ABI, on the five workloads and on edge cases."""
import numpy as np
import pytest
import torch

from fsm_inputs import (bpe_like_vocab, compile_regex, make_config, paper_float_example_dfa,
                        random_class_dfa, vocab_from_strings)
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from gpu_util import THREADS, check_index, gpu_index, mask_np, next_np


@pytest.fixture(autouse=True, params=[1, 2, 3], ids=["dense", "rowwise", "bucket"])
def _walk_algorithm(request):
    """Every case runs with each walk algorithm; knobs are reset afterwards."""
    fg.fsm_debug_set(6, request.param)
    yield
    for key in (1, 2, 3, 4, 6):
        fg.fsm_debug_set(key, 0)


def test_device_is_blackwell():
    assert fg.fsm_device_check() == 0


def test_paper_example_on_gpu():
    d = paper_float_example_dfa()
    vb, vo = vocab_from_strings(["A", ".", "42", ".2", "1"])
    mask, nxt = check_index(d.trans, d.accept, vb, vo, d.dead)
    assert [int(x) for x in mask[:, 0]] == [0x1E, 0x1E, 0x14, 0x14, 0]


@pytest.mark.parametrize("k", [1, 2])
def test_small_workloads_full_compare(k):
    w = make_config(k)
    check_index(w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)


def test_workload_3_full_compare():
    w = make_config(3)
    check_index(w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)


def test_workload_4_full_compare_in_state_tiles():
    """20,001 states x 152,064 tokens: the GPU builds the whole index (int32 states,
    the configuration the benchmark times); the comparison runs tile by tile so
    the host never holds the 12 GB table."""
    w = make_config(4)
    d = w.dfa
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    assert int(idx.status.item()) == 0
    tile = 1024
    for q0 in range(0, d.Q, tile):
        q1 = min(d.Q, q0 + tile)
        want_mask, want_next, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes,
                                                         w.vocab_offsets, d.dead, w.eos_id,
                                                         q_begin=q0, q_end=q1, threads=THREADS)
        got_mask = idx.allowed_mask[q0:q1].cpu().numpy().view(np.uint32)
        got_next = idx.next_state[q0:q1].cpu().numpy()
        assert (got_mask == want_mask).all(), q0
        assert (got_next == want_next).all(), q0
    del idx
    # u16 states and the bitmask-only build on a sample of state slabs
    for (q0, q1) in [(0, 300), (9984, 10300), (19700, 20001)]:
        check_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                    q_begin=q0, q_end=q1, modes=("u16", "mask"))


@pytest.mark.parametrize("N", [1, 5, 31, 32, 33, 1000, 1025])
def test_ragged_vocabulary_sizes(N):
    rng = np.random.default_rng(N)
    d, _ = random_class_dfa(N, n_live=37, n_classes=9, live_classes_per_state=5)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(0, 7)).tolist()) for _ in range(N)]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead, eos=N - 1)


def test_long_tokens_cross_the_inline_record():
    """Tokens of 15, 16, 17 and 40 bytes that stay alive to the end."""
    d = compile_regex(r"(ab)*c?")
    toks = [b"ab" * 7 + b"a", b"ab" * 8, b"ab" * 8 + b"c", b"ab" * 20, b"ab" * 19 + b"cc",
            b"ab" * 8 + b"x", b"", b"ab" * 100 + b"c"]
    vb, vo = vocab_from_strings(toks)
    mask, nxt = check_index(d.trans, d.accept, vb, vo, d.dead)
    assert mask[0, 0] == 0b10001111


def test_two_state_automaton_and_extremes():
    # Q = 2: one live state looping on every byte -> every non-empty token allowed
    trans = np.zeros((2, 256), dtype=np.int32)
    trans[1, :] = 1
    accept = np.array([1, 0], dtype=np.uint8)
    rng = np.random.default_rng(0)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(1, 20)).tolist()) for _ in range(200)]
    vb, vo = vocab_from_strings(toks)
    mask, _ = check_index(trans, accept, vb, vo, 1, eos=-1)
    assert (mask[0, :6] == 0xFFFFFFFF).all() and mask[0, 6] == 0xFF
    # everything dead: the live state reads nothing
    trans[0, :] = 1
    mask, nxt = check_index(trans, accept, vb, vo, 1, eos=7)
    assert mask[0].sum() == 1 << 7 and nxt[0, 7] == 0
    # dead state is state 0, live state 1
    trans = np.zeros((2, 256), dtype=np.int32)
    trans[1, 65:91] = 1
    check_index(trans, np.array([0, 1], dtype=np.uint8), vb, vo, 0, eos=3)


def test_state_that_reads_everything_over_a_large_vocabulary():
    """A state whose every byte loops: all 128,000 non-empty tokens survive, which is
    more 32-token chunks than the sparse walk keeps descriptors for (it then walks the
    buckets unit by unit) and fills every survivor list to the brim."""
    w = make_config(3)
    trans = np.full((3, 256), 2, dtype=np.int32)
    trans[0, :] = 0                       # state 0 reads everything and stays
    trans[1, 97:123] = 0                  # state 1 reads lowercase letters only
    accept = np.array([1, 0, 0], dtype=np.uint8)
    mask, nxt = check_index(trans, accept, w.vocab_bytes, w.vocab_offsets, 2, w.eos_id)
    lens = np.diff(w.vocab_offsets)
    assert int(np.unpackbits(mask[0].view(np.uint8)).sum()) == int((lens > 0).sum()) + 1


def test_vocabulary_beyond_the_window_ranking():
    """540,000 tokens are more windows of 32 sorted tokens than the bucket walk ranks in
    shared memory (it then takes them in index order); the other walks see a long row."""
    d, _ = random_class_dfa(21, n_live=40, n_classes=30, live_classes_per_state=8)
    vb, vo = bpe_like_vocab(11, 540_000, zero_length_ids=(539_999,))
    check_index(d.trans, d.accept, vb, vo, d.dead, 539_999)


def test_more_than_127_byte_classes_uses_one_level_buckets():
    d, cls = random_class_dfa(33, n_live=300, n_classes=220, live_classes_per_state=60)
    assert len(np.unique(d.trans.T, axis=0)) > 127
    rng = np.random.default_rng(2)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(0, 6)).tolist()) for _ in range(5000)]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead, eos=77)


def test_dead_row_contents_ignored():
    w = make_config(1)
    t = w.dfa.trans.copy()
    t[w.dfa.dead, :] = 2
    check_index(t, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)


def test_row_ranges():
    w = make_config(2)
    d = w.dfa
    for (a, b) in [(0, 1), (5, 40), (d.Q - 1, d.Q), (33, 65)]:
        check_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id,
                    q_begin=a, q_end=b)


def test_uncompressed_fallback_paths():
    """A forced hash collision, and a table with 256 distinct byte columns, both
    take the uncompressed walk and stay exact."""
    w = make_config(2)
    d = w.dfa
    N = 3000
    vo = w.vocab_offsets[:N + 1]
    vb = w.vocab_bytes[:vo[-1]]
    fg.fsm_debug_set(1, 1)
    check_index(d.trans, d.accept, vb, vo, d.dead, 2, expect_status=8, modes=("i32",))
    fg.fsm_debug_set(1, 0)
    rng = np.random.default_rng(4)
    Q = 300
    trans = rng.integers(0, Q, size=(Q, 256)).astype(np.int32)      # columns all distinct
    trans[rng.random((Q, 256)) < 0.6] = Q - 1
    toks = [bytes(rng.integers(0, 256, size=rng.integers(1, 5)).tolist()) for _ in range(500)]
    vb2, vo2 = vocab_from_strings(toks)
    check_index(trans, np.ones(Q, np.uint8), vb2, vo2, Q - 1, eos=11, modes=("i32", "mask"))


def test_state_tiled_path_on_a_small_table():
    """With the shared-memory budget capped, the table no longer fits: start-state
    rows are staged tile by tile and later bytes read the table from global memory."""
    w = make_config(2)
    d = w.dfa
    fg.fsm_debug_set(4, 40 * 1024)
    check_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    w3 = make_config(3)
    d3 = w3.dfa
    check_index(d3.trans, d3.accept, w3.vocab_bytes, w3.vocab_offsets, d3.dead, w3.eos_id,
                q_begin=100, q_end=777, modes=("u16",))


def test_more_than_65535_states_uses_wide_entries():
    Q = 70001
    d, _ = random_class_dfa(21, n_live=Q - 1, n_classes=20, live_classes_per_state=9)
    rng = np.random.default_rng(1)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(1, 6)).tolist()) for _ in range(257)]
    vb, vo = vocab_from_strings(toks)
    check_index(d.trans, d.accept, vb, vo, d.dead, eos=256, modes=("i32", "mask"))
    idx_err = fg.fsm_index_build(0, 0, 0, 0, 0, Q, 257, 0, -1, 0, 0, fg.FSM_STATE_U16, 0, 0)
    assert idx_err != 0


def test_data_faults_are_flagged_not_fatal():
    w = make_config(1)
    d = w.dfa
    t = d.trans.copy()
    t[0, 48:53] = 99          # out of range: counts as dead
    t[2, 55] = -7
    clamped = t.copy()
    clamped[(t < 0) | (t >= d.Q)] = d.dead
    check_index(t, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id, expect_status=1,
                oracle_trans=clamped, modes=("i32",))
    # a decreasing offset: that token is treated as empty
    vo = w.vocab_offsets.copy()
    vo[500] = vo[499] - 1
    fixed = vo.copy()
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, vo, d.dead, w.eos_id)
    assert int(idx.status.item()) & 2
    got = mask_np(idx)
    assert all(((got[q, 499 >> 5] >> np.uint32(499 & 31)) & 1) == 0 for q in range(d.Q))
