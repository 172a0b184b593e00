"""Multi-process checks of the sharding logic on CPU (gloo, world size 2): state
slabs of the index and batch slices of the decode step, each computed by one
rank, reassemble to the unsharded result.  The per-rank compute here is the CPU
oracle; on GPUs the same partition feeds fsm_index_build_rows / guided_mask_step."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from fsm_inputs import make_config, step_logits_numpy
        from oracle import fsm_oracle
        from paper_2307_09702_b200 import sharding
        w = make_config(1)
        d = w.dfa
        # ---- index rows sharded by state slab
        q0, q1 = sharding.state_slab(d.Q, rank, world)
        m, n, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                         w.eos_id, q_begin=q0, q_end=q1)
        full_mask = sharding.all_gather_rows(torch.from_numpy(m.view(np.int32)), d.Q)
        full_next = sharding.all_gather_rows(torch.from_numpy(n), d.Q)
        rm, rn, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead,
                                           w.eos_id)
        assert (full_mask.numpy().view(np.uint32) == rm).all()
        assert (full_next.numpy() == rn).all()
        # ---- decode step sharded by batch rows (index replicated)
        B = 5
        w.B = B
        x = step_logits_numpy(w, 0)
        states = (np.arange(B) % (d.Q - 1)).astype(np.int32)
        b0, b1 = sharding.batch_slice(B, rank, world)
        st, fin = states[b0:b1].copy(), np.zeros(b1 - b0, np.uint8)
        tok, _ = fsm_oracle.mask_step(np.ascontiguousarray(x[b0:b1]), st, fin, rm, rn, d.dead, w.eos_id)
        all_tok = sharding.all_gather_rows(torch.from_numpy(tok), B).numpy()
        all_st = sharding.all_gather_rows(torch.from_numpy(st), B).numpy()
        st_ref, fin_ref = states.copy(), np.zeros(B, np.uint8)
        tok_ref, _ = fsm_oracle.mask_step(x, st_ref, fin_ref, rm, rn, d.dead, w.eos_id)
        assert (all_tok == tok_ref).all() and (all_st == st_ref).all()
        # ---- equal slabs gathered in place (the layout of the sharded benchmark)
        per = -(-d.Q // world)
        full = torch.full((world * per, n.shape[1]), -5, dtype=torch.int32)
        e0, e1 = sharding.equal_slab(d.Q, rank, world)
        full[e0:e1] = torch.from_numpy(rn[e0:e1])
        whole = sharding.all_gather_slabs_in_place(full, d.Q)
        assert whole.shape[0] == d.Q and (whole.numpy() == rn).all()
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_contiguous_shards_cover_everything():
    sys.path.insert(0, ROOT)
    from paper_2307_09702_b200 import sharding
    for n in (0, 1, 5, 8, 1001, 20001):
        for world in (1, 2, 3, 8):
            s = sharding.contiguous_shards(n, world)
            assert s[0][0] == 0 and s[-1][1] == n and len(s) == world
            assert all(a[1] == b[0] for a, b in zip(s, s[1:]))
            sizes = [e - b for b, e in s]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.contiguous_shards(5, 0)
    for n in (0, 1, 5, 8, 1001, 20001):
        for world in (1, 2, 3, 8):
            slabs = [sharding.equal_slab(n, r, world) for r in range(world)]
            per = -(-n // world)
            assert slabs[0][0] == 0 and slabs[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(slabs, slabs[1:]))
            assert all(b == min(n, r * per) and e - b <= per for r, (b, e) in enumerate(slabs))


def test_state_slabs_and_batch_slices_reassemble_with_gloo(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
