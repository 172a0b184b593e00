"""Index files on the GPU: what fsm_index_save writes is the oracle's index in the documented
layout (read back here with numpy, without the library), fsm_index_load restores it bit for
bit into fresh device arrays, and damaged or foreign files are refused."""
import hashlib
import struct

import numpy as np
import pytest
import torch

from fsm_inputs import bpe_like_vocab, make_config, random_class_dfa
from oracle import fsm_oracle
from test_index_io_host import splitmix_checksum

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from paper_2307_09702_b200.binding import FSM_ERR_FORMAT, FSM_ERR_IO
    from gpu_util import THREADS, gpu_index, mask_np, next_np
    from test_gpu_csr import build_csr


def read_index_file(path):
    """Parses a file from the header comment alone."""
    raw = open(path, "rb").read()
    assert raw[:8] == b"FSMGIDX1"
    version, form, Q, N, sd, dead, eos, zero = struct.unpack("<IiiiiiiI", raw[8:40])
    nnz, payload_bytes, check = struct.unpack("<qQQ", raw[40:64])
    assert version == 1 and zero == 0 and raw[96:128] == bytes(32)
    payload = raw[128:]
    assert len(payload) == payload_bytes and splitmix_checksum(payload) == check
    W = (N + 31) // 32
    at = 0

    def take(dtype, count):
        nonlocal at
        a = np.frombuffer(payload, dtype=dtype, count=count, offset=at)
        at += (a.nbytes + 7) // 8 * 8
        return a
    out = {"form": form, "Q": Q, "N": N, "state_dtype": sd, "dead": dead, "eos": eos, "nnz": nnz,
           "digest": raw[64:96], "mask": take("<u4", Q * W).reshape(Q, W)}
    if form == 0:
        out["next"] = take("<u2" if sd == 1 else "<i4", Q * N).reshape(Q, N)
    elif form == 2:
        out["offsets"], out["tokens"], out["csr_next"] = take("<i8", Q + 1), take("<i4", nnz), take("<i4", nnz)
    assert at == len(payload)
    return out


def input_digest_by_hashlib(trans, accept, vb, vo, dead, eos):
    Q, N = trans.shape[0], len(vo) - 1
    h = hashlib.sha256()
    h.update(struct.pack("<iiiiq", Q, N, dead, eos, int(vo[-1])))
    for a, dt in ((trans, np.int32), (accept, np.uint8), (vo, np.int32), (vb[: int(vo[-1])], np.uint8)):
        h.update(np.ascontiguousarray(a, dtype=dt).tobytes())
    return h.digest()


def problem(kind):
    if kind == "config1":
        w = make_config(1)
        return w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id
    if kind == "config2":
        w = make_config(2)
        return w.dfa.trans, w.dfa.accept, w.vocab_bytes, w.vocab_offsets, w.dfa.dead, w.eos_id
    # 300 states x 20,001 tokens: a 24 MB table, which crosses the 16 MiB staging pieces, and a
    # table whose byte count is not a multiple of 8 in the 16-bit form
    d, _ = random_class_dfa(300, n_live=299, n_classes=40, live_classes_per_state=9)
    vb, vo = bpe_like_vocab(7, 20_001, zero_length_ids=(20_000,))
    return d.trans, d.accept, vb, vo, d.dead, 20_000


@pytest.mark.parametrize("kind", ["config1", "config2", "staged"])
@pytest.mark.parametrize("mode", ["i32", "u16", "mask"])
def test_dense_round_trip_equals_the_oracle(tmp_path, kind, mode):
    trans, accept, vb, vo, dead, eos = problem(kind)
    want_mask, want_next, _ = fsm_oracle.index_build(trans, accept, vb, vo, dead, eos, threads=THREADS)
    sd = fg.FSM_STATE_U16 if mode == "u16" else fg.FSM_STATE_I32
    idx = gpu_index(trans, accept, vb, vo, dead, eos, sd, mode != "mask")
    digest = idx.input_digest()
    assert digest == input_digest_by_hashlib(trans, accept, vb, vo, dead, eos)
    path = str(tmp_path / "index.fsmidx")
    idx.save(path)
    f = read_index_file(path)
    assert (f["form"], f["Q"], f["N"], f["dead"], f["eos"], f["nnz"]) == \
        (1 if mode == "mask" else 0, trans.shape[0], len(vo) - 1, dead, eos, 0)
    assert f["digest"] == digest and f["state_dtype"] == (1 if mode == "u16" else 0)
    assert (f["mask"] == want_mask).all()
    if mode != "mask":
        assert (f["next"].astype(np.int32) == want_next).all()
    import os
    assert os.path.getsize(path) == fg.fsm_index_serialized_bytes(idx._desc(digest))
    # a fresh object for the same inputs, arrays poisoned, filled from the file
    fresh = fg.GuidedIndex(trans, accept, vb, vo, dead, eos, sd, mode != "mask")
    fresh.allowed_mask.fill_(0x55555555)
    if fresh.next_state is not None:
        fresh.next_state.view(torch.uint8).fill_(0xEE)
    fresh.load(path)
    assert (mask_np(fresh) == want_mask).all()
    if mode != "mask":
        assert (next_np(fresh) == want_next).all()


def test_compressed_rows_round_trip_equals_the_oracle(tmp_path):
    for kind in ("config2", "staged"):
        trans, accept, vb, vo, dead, eos = problem(kind)
        Q, N = trans.shape[0], len(vo) - 1
        want_mask, want_off, want_tok, want_next = fsm_oracle.index_csr(trans, accept, vb, vo, dead, eos,
                                                                        threads=THREADS)
        nnz = int(want_off[-1])
        mask, off, tok, nxt, status = build_csr(trans, accept, vb, vo, dead, eos, nnz)
        assert status == 0
        d = fg.index_desc(fg.FSM_INDEX_CSR, Q, N, dead, eos, 0, nnz, b"\7" * 32, mask, None, off, tok, nxt)
        path = str(tmp_path / f"{kind}.fsmidx")
        assert fg.fsm_index_save(path, d) == 0
        f = read_index_file(path)
        assert f["form"] == 2 and f["nnz"] == nnz and f["digest"] == b"\7" * 32
        assert (f["mask"] == want_mask).all() and (f["offsets"] == want_off).all()
        assert (f["tokens"] == want_tok).all() and (f["csr_next"] == want_next).all()
        peek = fg.IndexDesc()
        assert fg.fsm_index_peek(path, peek) == 0 and peek.nnz == nnz and peek.Q == Q
        dev = mask.device
        m2, o2 = torch.full_like(mask, 3), torch.full_like(off, -3)
        t2, n2 = torch.full((nnz,), -3, dtype=torch.int32, device=dev), torch.full((nnz,), -3, dtype=torch.int32, device=dev)
        d2 = fg.index_desc(fg.FSM_INDEX_CSR, Q, N, dead, eos, 0, nnz, None, m2, None, o2, t2, n2)   # any digest
        assert fg.fsm_index_load(path, d2) == 0
        torch.cuda.synchronize()
        assert (m2.cpu().numpy().view(np.uint32) == want_mask).all() and (o2.cpu().numpy() == want_off).all()
        assert (t2.cpu().numpy() == want_tok).all() and (n2.cpu().numpy() == want_next).all()


def test_damaged_truncated_and_foreign_files_are_refused(tmp_path):
    trans, accept, vb, vo, dead, eos = problem("config2")
    idx = gpu_index(trans, accept, vb, vo, dead, eos, fg.FSM_STATE_U16)
    path = str(tmp_path / "index.fsmidx")
    idx.save(path)
    raw = bytearray(open(path, "rb").read())

    def poisoned():
        o = fg.GuidedIndex(trans, accept, vb, vo, dead, eos, fg.FSM_STATE_U16)
        o.allowed_mask.fill_(0x55555555)
        return o
    # truncated: refused from the header, nothing written
    cut = str(tmp_path / "cut")
    open(cut, "wb").write(raw[: len(raw) // 2])
    o = poisoned()
    with pytest.raises(fg.FsmError) as e:
        o.load(cut)
    assert e.value.code == FSM_ERR_IO
    torch.cuda.synchronize()
    assert (o.allowed_mask == 0x55555555).all()
    # one payload bit flipped: the checksum catches it
    bad = bytearray(raw)
    bad[128 + 4000] ^= 0x10
    flipped = str(tmp_path / "flipped")
    open(flipped, "wb").write(bad)
    with pytest.raises(fg.FsmError) as e:
        poisoned().load(flipped)
    assert e.value.code == FSM_ERR_FORMAT
    # a file for other inputs (another EOS id changes the digest and the header)
    other = fg.GuidedIndex(trans, accept, vb, vo, dead, eos - 1, fg.FSM_STATE_U16)
    other.allowed_mask.fill_(0x55555555)
    with pytest.raises(fg.FsmError) as e:
        other.load(path)
    assert e.value.code == FSM_ERR_FORMAT
    torch.cuda.synchronize()
    assert (other.allowed_mask == 0x55555555).all()
    # same header, other inputs: only the digest differs
    t2 = trans.copy()
    t2[0, 65] = 0 if trans[0, 65] != 0 else 1
    changed = fg.GuidedIndex(t2, accept, vb, vo, dead, eos, fg.FSM_STATE_U16)
    with pytest.raises(fg.FsmError) as e:
        changed.load(path)
    assert e.value.code == FSM_ERR_FORMAT
    # another table dtype
    with pytest.raises(fg.FsmError) as e:
        fg.GuidedIndex(trans, accept, vb, vo, dead, eos, fg.FSM_STATE_I32).load(path)
    assert e.value.code == FSM_ERR_FORMAT
    # an unwritable path
    with pytest.raises(fg.FsmError) as e:
        idx.save(str(tmp_path / "no_such_dir" / "x"))
    assert e.value.code == FSM_ERR_IO
    # the good file still loads
    poisoned().load(path)
