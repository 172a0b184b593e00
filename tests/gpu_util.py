"""Helpers shared by the GPU parity tests (marshalling and comparison only)."""
import os

import numpy as np
import torch

from oracle import fsm_oracle
import paper_2307_09702_b200 as fg

THREADS = max(1, len(os.sched_getaffinity(0)))


def gpu_index(trans, accept, vb, vo, dead, eos=-1, state_dtype=fg.FSM_STATE_I32, want_next=True,
              q_begin=0, q_end=None):
    idx = fg.GuidedIndex(trans, accept, vb, vo, dead, eos, state_dtype, want_next,
                         q_begin=q_begin, q_end=q_end)
    # poison the outputs so that unwritten words show up
    idx.allowed_mask.fill_(-1431655766)
    if idx.next_state is not None:
        idx.next_state.view(torch.uint8).fill_(0xEE)
    idx.build()
    torch.cuda.synchronize()
    return idx


def mask_np(idx):
    return idx.allowed_mask.cpu().numpy().view(np.uint32)


def next_np(idx):
    if idx.next_state is None:
        return None
    if idx.next_state.dtype == torch.uint16:
        return idx.next_state.view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int32)
    return idx.next_state.cpu().numpy()


def check_index(trans, accept, vb, vo, dead, eos=-1, q_begin=0, q_end=None, expect_status=0,
                oracle_trans=None, modes=("i32", "u16", "mask")):
    """Builds on the GPU in the requested output modes and compares every word
    and entry with the oracle (bit-exact)."""
    Q = trans.shape[0]
    want_mask, want_next, _ = fsm_oracle.index_build(trans if oracle_trans is None else oracle_trans,
                                                     accept, vb, vo, dead, eos, q_begin=q_begin,
                                                     q_end=q_end, threads=THREADS)
    for mode in modes:
        if mode == "u16" and Q > 65535:
            continue
        sd = fg.FSM_STATE_U16 if mode == "u16" else fg.FSM_STATE_I32
        idx = gpu_index(trans, accept, vb, vo, dead, eos, sd, mode != "mask", q_begin, q_end)
        got_mask = mask_np(idx)
        assert got_mask.shape == want_mask.shape
        bad = np.argwhere(got_mask != want_mask)
        assert bad.size == 0, (mode, "mask", bad[:5], len(bad))
        if mode != "mask":
            got_next = next_np(idx)
            bad = np.argwhere(got_next != want_next)
            assert bad.size == 0, (mode, "next", bad[:5], len(bad))
        status = int(idx.status.item())
        assert status == expect_status, (mode, status)
    return want_mask, want_next
