"""The multi-GPU split driven through the CUDA library on one GPU: the state slabs that
`sharding.state_slab` hands to the ranks, each built with fsm_index_build_rows, put together
give the oracle's index; the batch slices of `sharding.batch_slice`, each stepped with
guided_mask_step / guided_sample_step against the whole index, give the oracle's step.
(The ranks run one after the other here; between GPUs the slabs meet in an all-gather,
which the gloo test covers on CPU.)"""
import numpy as np
import pytest
import torch

from fsm_inputs import bpe_like_vocab, f32_to_bf16_bits, make_config, random_class_dfa
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200 import sharding
    from gpu_util import THREADS, gpu_index, mask_np, next_np


def _problems():
    w = make_config(2)
    yield "config2", (w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id)
    d, _ = random_class_dfa(5, n_live=700, n_classes=50, live_classes_per_state=10)
    vb, vo = bpe_like_vocab(9, 30_000, zero_length_ids=(29_999,))
    yield "701 states", (d.trans, d.accept, vb, vo, d.dead, 29_999)


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("mode", ["i32", "u16", "mask"])
def test_state_slabs_built_by_the_library_concatenate_to_the_oracles_index(world, mode):
    sd = fg.FSM_STATE_U16 if mode == "u16" else fg.FSM_STATE_I32
    for name, (trans, accept, vb, vo, dead, eos) in _problems():
        Q = trans.shape[0]
        want_mask, want_next, _ = fsm_oracle.index_build(trans, accept, vb, vo, dead, eos, threads=THREADS)
        masks, nexts = [], []
        for rank in range(world):
            q0, q1 = sharding.state_slab(Q, rank, world)
            slab = gpu_index(trans, accept, vb, vo, dead, eos, sd, mode != "mask", q_begin=q0, q_end=q1)
            assert int(slab.status.item()) == 0
            assert slab.allowed_mask.shape[0] == q1 - q0
            masks.append(slab.allowed_mask)
            nexts.append(slab.next_state)
        got_mask = torch.cat(masks, dim=0).cpu().numpy().view(np.uint32)
        assert got_mask.shape == want_mask.shape and (got_mask == want_mask).all(), name
        if mode != "mask":
            got = torch.cat(nexts, dim=0)
            got = got.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int32) if mode == "u16" \
                else got.cpu().numpy()
            assert (got == want_next).all(), name


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("sample", [None, (1.5, 99, 4)], ids=["greedy", "drawn"])
def test_batch_slices_stepped_by_the_library_give_the_oracles_step(world, sample):
    w = make_config(2)
    d = w.dfa
    N, B = w.N, 11
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    o_mask, o_next, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                               w.eos_id, threads=THREADS)
    rng = np.random.default_rng(world)
    x = f32_to_bf16_bits(np.round(rng.standard_normal((B, N)).astype(np.float32) * 2, 1))
    states = rng.integers(0, d.Q - 1, size=B).astype(np.int32)
    finished = np.zeros(B, np.uint8)
    finished[5] = 1
    st_o, fin_o = states.copy(), finished.copy()
    if sample is None:
        tok_o, out_o = fsm_oracle.mask_step(x, st_o, fin_o, o_mask, o_next, d.dead, w.eos_id, threads=THREADS)
    else:
        tok_o, out_o = fsm_oracle.sample_step(x, st_o, fin_o, o_mask, o_next, d.dead, w.eos_id, *sample,
                                              threads=THREADS)
    dev = torch.device("cuda")
    toks, sts, fins, outs = [], [], [], []
    for rank in range(world):
        b0, b1 = sharding.batch_slice(B, rank, world)
        logits = torch.from_numpy(x[b0:b1].view(np.int16)).to(dev).view(torch.bfloat16).contiguous()
        st = torch.from_numpy(states[b0:b1]).to(dev)
        fin = torch.from_numpy(finished[b0:b1]).to(dev)
        tok = torch.full((b1 - b0,), -9, dtype=torch.int32, device=dev)
        if b1 > b0:
            if sample is None:
                idx.step(logits, st, fin, tok)
            else:
                idx.sample(logits, st, fin, tok, *sample)
        toks.append(tok), sts.append(st), fins.append(fin), outs.append(logits.view(torch.int16))
    torch.cuda.synchronize()
    got_tok = torch.cat(toks).cpu().numpy()
    if sample is None:
        assert (got_tok == tok_o).all()
        assert (torch.cat(sts).cpu().numpy() == st_o).all() and (torch.cat(fins).cpu().numpy() == fin_o).all()
        live = finished == 0
        assert (torch.cat(outs).cpu().numpy()[live] == out_o.view(np.int16)[live]).all()
    else:
        # The random numbers of a draw are keyed by the row's position inside the call, so a
        # slice draws what the oracle draws for that slice (not what the whole batch would
        # have drawn in one call); the masked logits do not depend on the draw.
        live = finished == 0
        assert (torch.cat(outs).cpu().numpy()[live] == out_o.view(np.int16)[live]).all()
        for rank in range(world):
            b0, b1 = sharding.batch_slice(B, rank, world)
            if b1 == b0:
                continue
            s2, f2 = states[b0:b1].copy(), finished[b0:b1].copy()
            t2, _ = fsm_oracle.sample_step(np.ascontiguousarray(x[b0:b1]), s2, f2, o_mask, o_next, d.dead,
                                           w.eos_id, *sample, threads=THREADS)
            assert (toks[rank].cpu().numpy() == t2).all()
            assert (sts[rank].cpu().numpy() == s2).all() and (fins[rank].cpu().numpy() == f2).all()
