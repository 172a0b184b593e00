"""GPU parity of the compressed-row index (fsm_index_build_csr) and of the decode step on it
(guided_step_csr) against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from fsm_inputs import (bpe_like_vocab, f32_to_bf16_bits, make_config, random_class_dfa, start_states,
                        vocab_from_strings)
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from gpu_util import THREADS


def build_csr(trans, accept, vb, vo, dead, eos, capacity):
    dev = torch.device("cuda")
    Q, N = trans.shape[0], len(vo) - 1
    W = (N + 31) // 32
    t = lambda a, dt: torch.as_tensor(np.ascontiguousarray(a), dtype=dt).to(dev)
    d_trans, d_acc, d_vo = t(trans, torch.int32), t(accept, torch.uint8), t(vo, torch.int32)
    d_vb = t(vb if len(vb) else np.zeros(1, np.uint8), torch.uint8)
    mask = torch.full((Q, W), -1431655766, dtype=torch.int32, device=dev)
    off = torch.full((Q + 1,), -7, dtype=torch.int64, device=dev)
    tok = torch.full((max(capacity, 1),), -7, dtype=torch.int32, device=dev)
    nxt = torch.full((max(capacity, 1),), -7, dtype=torch.int32, device=dev)
    nbytes = int(vo[-1])
    wsb = fg.fsm_index_workspace_bytes(Q, N, nbytes)
    ws = torch.empty(wsb, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = fg.fsm_index_build_csr(d_trans, d_acc, d_vb, d_vo, nbytes, Q, N, dead, eos, mask, off, tok, nxt,
                                capacity, ws, wsb, status)
    assert rc == 0, fg.fsm_status_string(rc)
    torch.cuda.synchronize()
    return mask, off, tok, nxt, int(status.item())


def check_csr(trans, accept, vb, vo, dead, eos):
    want_mask, want_off, want_tok, want_next = fsm_oracle.index_csr(trans, accept, vb, vo, dead, eos,
                                                                    threads=THREADS)
    nnz = int(want_off[-1])
    mask, off, tok, nxt, status = build_csr(trans, accept, vb, vo, dead, eos, nnz)
    assert status == 0
    assert (mask.cpu().numpy().view(np.uint32) == want_mask).all()
    assert (off.cpu().numpy() == want_off).all()
    assert (tok.cpu().numpy()[:nnz] == want_tok).all()
    assert (nxt.cpu().numpy()[:nnz] == want_next).all()
    return (mask, off, tok, nxt), (want_mask, want_off, want_tok, want_next)


@pytest.mark.parametrize("k", [1, 2, 3])
def test_workloads_compressed_rows(k):
    w = make_config(k)
    check_csr(w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)


@pytest.mark.parametrize("N", [1, 31, 33, 1025])
def test_ragged_vocabularies_and_empty_rows(N):
    rng = np.random.default_rng(N)
    d, _ = random_class_dfa(N, n_live=37, n_classes=9, live_classes_per_state=5)
    toks = [bytes(rng.integers(0, 256, size=rng.integers(0, 7)).tolist()) for _ in range(N)]
    vb, vo = vocab_from_strings(toks)
    check_csr(d.trans, d.accept, vb, vo, d.dead, N - 1)


@pytest.mark.parametrize("n_live", [199, 255, 300])
def test_automata_around_the_dense_table_threshold(n_live):
    # under 256 states the rows are cut out of a dense table built into the workspace (by the
    # row-wise walk once there is a row per SM), from 256 states on out of the bucket walk's bitmask
    d, _ = random_class_dfa(n_live, n_live=n_live, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 5000, zero_length_ids=(4999,))
    check_csr(d.trans, d.accept, vb, vo, d.dead, 4999)


def test_capacity_too_small_is_flagged_and_offsets_stay_complete():
    w = make_config(1)
    d = w.dfa
    _, want_off, want_tok, want_next = fsm_oracle.index_csr(d.trans, d.accept, w.vocab_bytes,
                                                            w.vocab_offsets, d.dead, w.eos_id)
    cap = int(want_off[-1]) // 2
    _, off, tok, nxt, status = build_csr(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                         w.eos_id, cap)
    assert status == 32
    assert (off.cpu().numpy() == want_off).all()
    assert (tok.cpu().numpy()[:cap] == want_tok[:cap]).all()
    assert (nxt.cpu().numpy()[:cap] == want_next[:cap]).all()


@pytest.mark.parametrize("sample", [0, 1])
def test_decode_steps_on_compressed_rows_match_the_oracle(sample):
    """Workload 5's shape at a reduced batch: 4 steps in lock step with the oracle (which
    uses the dense table: the two forms of the index must decode alike)."""
    w = make_config(5)
    d = w.dfa
    (mask, off, tok, nxt), (o_mask, _, _, _) = check_csr(d.trans, d.accept, w.vocab_bytes,
                                                         w.vocab_offsets, d.dead, w.eos_id)
    _, o_next, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                          w.eos_id, threads=THREADS)
    B = 64
    st_o = start_states(w)[:B].copy()
    fin_o = np.zeros(B, np.uint8)
    d_st = torch.from_numpy(st_o.copy()).cuda()
    d_fin = torch.zeros(B, dtype=torch.uint8, device="cuda")
    d_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(11)
    for step in range(4):
        x = (rng.standard_normal((B, w.N)).astype(np.float32) * 1.5)
        bits = f32_to_bf16_bits(x)
        if sample:
            tok_o, out_o = fsm_oracle.sample_step(bits, st_o, fin_o, o_mask, o_next, d.dead, w.eos_id,
                                                  10.0, 77, step, threads=THREADS)
        else:
            tok_o, out_o = fsm_oracle.mask_step(bits, st_o, fin_o, o_mask, o_next, d.dead, w.eos_id,
                                                threads=THREADS)
        dx = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
        rc = fg.guided_step_csr(dx, dx, fg.FSM_LOGITS_BF16, w.N, d_st, d_fin, d_tok, mask, off, tok, nxt,
                                tok.numel(), d.Q, w.N, B, d.dead, w.eos_id, sample, 10.0, 77, step,
                                status)
        assert rc == 0
        torch.cuda.synchronize()
        assert (d_tok.cpu().numpy() == tok_o).all()
        assert (d_st.cpu().numpy() == st_o).all() and (d_fin.cpu().numpy() == fin_o).all()
        assert (dx.view(torch.int16).cpu().numpy().view(np.uint16) == out_o).all()
    assert int(status.item()) == 0


def test_decode_step_on_an_overflowed_index_stays_inside_the_arrays():
    """An index built with half the capacity it needs: row_offsets is complete, the entry
    arrays end at `capacity`.  The step must not look beyond them (the words behind are
    canaries that would send a row to a wrong state): a chosen token whose entry exists
    advances as usual, one whose entry is missing goes to the dead state."""
    w = make_config(2)
    d = w.dfa
    o_mask, want_off, want_tok, want_next = fsm_oracle.index_csr(
        d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id, threads=THREADS)
    total = int(want_off[-1])
    cap = total // 2
    mask, off, tok, nxt, status = build_csr(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                            w.eos_id, cap)
    assert status == 32
    # entry arrays followed by canaries: every token id, each "leading" to state 1
    canary_tok = torch.arange(w.N, dtype=torch.int32, device="cuda").repeat(4)
    tok_c = torch.cat([tok[:cap], canary_tok])
    nxt_c = torch.cat([nxt[:cap], torch.ones_like(canary_tok)])
    live = [q for q in range(d.Q) if want_off[q + 1] > want_off[q]]
    B = len(live)
    states = np.array(live, dtype=np.int32)
    d_st = torch.from_numpy(states.copy()).cuda()
    d_fin = torch.zeros(B, dtype=torch.uint8, device="cuda")
    d_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    st_word = torch.zeros(1, dtype=torch.int32, device="cuda")
    rng = np.random.default_rng(5)
    x = rng.standard_normal((B, w.N)).astype(np.float32)
    dx = torch.from_numpy(x).cuda()
    rc = fg.guided_step_csr(dx, None, fg.FSM_LOGITS_F32, w.N, d_st, d_fin, d_tok, mask, off, tok_c,
                            nxt_c, cap, d.Q, w.N, B, d.dead, w.eos_id, 0, 1.0, 0, 0, st_word)
    assert rc == 0
    torch.cuda.synchronize()
    got_tok, got_st = d_tok.cpu().numpy(), d_st.cpu().numpy()
    n_missing = 0
    for i, q in enumerate(live):
        lo, hi = int(want_off[q]), int(want_off[q + 1])
        row_tok = want_tok[lo:hi]
        choice = int(row_tok[np.argmax(x[i, row_tok])])        # allowed token with the largest logit
        assert got_tok[i] == choice
        if choice == w.eos_id:
            continue
        at = lo + int(np.searchsorted(row_tok, choice))
        if at < cap:
            assert got_st[i] == want_next[at]
        else:
            n_missing += 1
            assert got_st[i] == d.dead
    assert n_missing > 0


@pytest.mark.parametrize("algo", [1, 2])
def test_compressed_rows_under_every_walk_algorithm(algo):
    """300 states: the rows are cut out of the bitmask (no dense table in the workspace),
    whichever walk built it."""
    d, _ = random_class_dfa(300, n_live=300, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 5000, zero_length_ids=(4999,))
    fg.fsm_debug_set(6, algo)
    try:
        check_csr(d.trans, d.accept, vb, vo, d.dead, 4999)
    finally:
        fg.fsm_debug_set(6, 0)
