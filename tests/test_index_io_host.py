"""Host side of the index files: the SHA-256 and checksum routines against independent
definitions, the documented header layout, and the refusals that need no GPU."""
import hashlib
import os
import struct

import numpy as np
import pytest


@pytest.fixture(scope="module")
def fg():
    from paper_2307_09702_b200 import build as b
    b.build()
    import paper_2307_09702_b200 as fg
    return fg


def splitmix_checksum(data: bytes, first: int = 0) -> int:
    """The header's definition, restated with numpy."""
    w = np.frombuffer(data, dtype="<u8").copy()
    i = np.arange(first + 1, first + 1 + len(w), dtype=np.uint64)
    with np.errstate(over="ignore"):
        x = w + i * np.uint64(0x9E3779B97F4A7C15)
        x = (x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        x = (x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        x = x ^ (x >> np.uint64(31))
        return int(x.sum(dtype=np.uint64))


def write_index_file(path, form, Q, N, state_dtype, dead, eos, nnz, digest, arrays):
    """Writes an index file from the header comment alone (independent of the library)."""
    payload = b""
    for a in arrays:
        b = np.ascontiguousarray(a).tobytes()
        payload += b + b"\0" * ((-len(b)) % 8)
    h = b"FSMGIDX1" + struct.pack("<IiiiiiiI", 1, form, Q, N, state_dtype, dead, eos, 0)
    h += struct.pack("<qQQ", nnz, len(payload), splitmix_checksum(payload)) + bytes(digest) + b"\0" * 32
    assert len(h) == 128
    with open(path, "wb") as f:
        f.write(h + payload)
    return len(h) + len(payload)


def test_sha256_against_the_standard_and_hashlib(fg):
    # FIPS 180-4 example: SHA-256("abc")
    assert fg.fsm_sha256(b"abc").hex() == "ba7816bf8f01cfea414140de5dae2223b00361a396177a9cb410ff61f20015ad"
    rng = np.random.default_rng(0)
    for n in (0, 1, 55, 56, 57, 63, 64, 65, 119, 120, 1000, 65_536, 1_000_003):
        data = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
        assert fg.fsm_sha256(data) == hashlib.sha256(data).digest(), n


def test_checksum_follows_its_definition_and_sees_order(fg):
    rng = np.random.default_rng(1)
    data = rng.integers(0, 256, size=8 * 1000, dtype=np.uint8).tobytes()
    assert fg.fsm_checksum64(data) == splitmix_checksum(data)
    assert fg.fsm_checksum64(data, 77) == splitmix_checksum(data, 77)
    # pieces add up: the sum over a file can be taken piece by piece
    a, b = data[:2400], data[2400:]
    assert (fg.fsm_checksum64(a) + fg.fsm_checksum64(b, 300)) % 2**64 == fg.fsm_checksum64(data)
    swapped = data[8:16] + data[:8] + data[16:]
    assert fg.fsm_checksum64(swapped) != fg.fsm_checksum64(data)
    assert fg.fsm_checksum64(b"\0" * 8) != fg.fsm_checksum64(b"\0" * 16)


def test_serialized_size(fg):
    Q, N = 7, 100
    W = 4
    d = fg.index_desc(fg.FSM_INDEX_DENSE, Q, N, 6, -1, fg.FSM_STATE_I32)
    assert fg.fsm_index_serialized_bytes(d) == 128 + Q * W * 4 + Q * N * 4
    d = fg.index_desc(fg.FSM_INDEX_DENSE, Q, 101, 6, 3, fg.FSM_STATE_U16)
    assert fg.fsm_index_serialized_bytes(d) == 128 + Q * 4 * 4 + (Q * 101 * 2 + 7) // 8 * 8
    d = fg.index_desc(fg.FSM_INDEX_BITMASK, Q, N, 6, -1)
    assert fg.fsm_index_serialized_bytes(d) == 128 + Q * W * 4
    d = fg.index_desc(fg.FSM_INDEX_CSR, Q, N, 6, -1, 0, 55)
    assert fg.fsm_index_serialized_bytes(d) == 128 + Q * W * 4 + (Q + 1) * 8 + 2 * ((55 * 4 + 7) // 8 * 8)
    for bad in (fg.index_desc(7, Q, N, 6, -1), fg.index_desc(0, 0, N, 0, -1), fg.index_desc(0, Q, N, Q, -1),
                fg.index_desc(0, Q, N, 6, N), fg.index_desc(0, 70_000, N, 6, -1, fg.FSM_STATE_U16),
                fg.index_desc(fg.FSM_INDEX_CSR, Q, N, 6, -1, 0, Q * N + 1),
                fg.index_desc(fg.FSM_INDEX_BITMASK, Q, N, 6, -1, 0, 5)):
        assert fg.fsm_index_serialized_bytes(bad) == 0


def test_peek_reads_a_file_written_from_the_documented_layout(fg, tmp_path):
    Q, N = 5, 70
    W = 3
    rng = np.random.default_rng(2)
    mask = rng.integers(0, 2**32, size=(Q, W), dtype=np.uint32)
    nxt = rng.integers(0, Q, size=(Q, N)).astype(np.uint16)
    digest = hashlib.sha256(b"inputs").digest()
    path = str(tmp_path / "a.fsmidx")
    size = write_index_file(path, 0, Q, N, 1, 4, 9, 0, digest, [mask, nxt])
    want = fg.index_desc(fg.FSM_INDEX_DENSE, Q, N, 4, 9, fg.FSM_STATE_U16)
    assert size == fg.fsm_index_serialized_bytes(want)
    got = fg.IndexDesc()
    got.allowed_mask = 0x1234
    assert fg.fsm_index_peek(path, got) == 0
    assert (got.form, got.Q, got.N, got.state_dtype, got.dead_state, got.eos_id, got.nnz) == (0, Q, N, 1, 4, 9, 0)
    assert bytes(got.input_digest) == digest and got.allowed_mask == 0x1234
    # CSR header
    path2 = str(tmp_path / "b.fsmidx")
    write_index_file(path2, 2, Q, N, 0, 4, -1, 3, digest, [mask, np.arange(Q + 1, dtype=np.int64),
                                                          np.arange(3, dtype=np.int32), np.zeros(3, np.int32)])
    assert fg.fsm_index_peek(path2, got) == 0 and got.form == 2 and got.nnz == 3 and got.eos_id == -1


def test_refusals_that_need_no_device(fg, tmp_path):
    from paper_2307_09702_b200.binding import FSM_ERR_FORMAT, FSM_ERR_IO
    d = fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 70, 4, -1, allowed_mask=0x1000)
    missing = str(tmp_path / "nothing_here")
    assert fg.fsm_index_peek(missing, fg.IndexDesc()) == FSM_ERR_IO
    assert fg.fsm_index_load(missing, d, stream=0) == FSM_ERR_IO
    assert "FSM_ERR_IO" in fg.fsm_status_string(FSM_ERR_IO)
    assert "FSM_ERR_FORMAT" in fg.fsm_status_string(FSM_ERR_FORMAT)
    junk = str(tmp_path / "junk")
    open(junk, "wb").write(os.urandom(300))
    assert fg.fsm_index_peek(junk, fg.IndexDesc()) == FSM_ERR_FORMAT
    assert fg.fsm_index_load(junk, d, stream=0) == FSM_ERR_FORMAT
    short = str(tmp_path / "short")
    open(short, "wb").write(b"FSMGIDX1" + b"\0" * 20)
    assert fg.fsm_index_peek(short, fg.IndexDesc()) == FSM_ERR_IO
    # a well-formed file for another problem, and a truncated one: refused from the header
    mask = np.zeros((5, 3), np.uint32)
    good = str(tmp_path / "good")
    write_index_file(good, 1, 5, 70, 0, 4, -1, 0, bytes(32), [mask])
    assert fg.fsm_index_peek(good, fg.IndexDesc()) == 0
    for other in (fg.index_desc(fg.FSM_INDEX_BITMASK, 6, 70, 4, -1, allowed_mask=0x1000),
                  fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 71, 4, -1, allowed_mask=0x1000),
                  fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 70, 3, -1, allowed_mask=0x1000),
                  fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 70, 4, 2, allowed_mask=0x1000),
                  fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 70, 4, -1, input_digest=b"\1" * 32, allowed_mask=0x1000)):
        assert fg.fsm_index_load(good, other, stream=0) == FSM_ERR_FORMAT
    data = open(good, "rb").read()
    cut = str(tmp_path / "cut")
    open(cut, "wb").write(data[:-8])
    assert fg.fsm_index_peek(cut, fg.IndexDesc()) == FSM_ERR_IO
    assert fg.fsm_index_load(cut, d, stream=0) == FSM_ERR_IO
    longer = str(tmp_path / "longer")
    open(longer, "wb").write(data + b"\0" * 8)
    assert fg.fsm_index_load(longer, d, stream=0) == FSM_ERR_FORMAT
    # descriptor errors come before the file is opened
    assert fg.fsm_index_load(good, fg.index_desc(fg.FSM_INDEX_BITMASK, 5, 70, 4, -1), stream=0) == -1
    assert fg.fsm_index_save(str(tmp_path / "x"), fg.index_desc(fg.FSM_INDEX_DENSE, 5, 70, 4, -1, allowed_mask=1), stream=0) == -1
