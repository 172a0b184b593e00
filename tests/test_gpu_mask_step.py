"""GPU parity of guided_mask_step and guided_sample_step against the CPU oracle:
masked logits, chosen tokens, states and finished flags are compared bit for bit
(tolerance 0; the sampled token is a pure function of logits, seed and draw number)."""
import numpy as np
import pytest
import torch

from fsm_inputs import f32_to_bf16_bits, make_config, start_states
from oracle import fsm_oracle

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    import paper_2307_09702_b200 as fg
    from gpu_util import THREADS, gpu_index, mask_np, next_np


@pytest.fixture(autouse=True)
def _reset_knobs():
    yield
    for key in (1, 2, 3, 4):
        fg.fsm_debug_set(key, 0)


def random_index(rng, Q, N, allowed_frac=0.25):
    W = (N + 31) // 32
    bits = rng.random((Q, W * 32)) < allowed_frac
    bits[:, N:] = False
    bits[Q - 1] = False
    mask = np.packbits(bits, axis=1, bitorder="little").view(np.uint32)
    nxt = rng.integers(0, Q - 1, size=(Q, N)).astype(np.int32)
    nxt[~bits[:, :N]] = Q - 1
    return np.ascontiguousarray(mask), nxt


def run_case(rng, Q, N, B, dtype, mode, k=0, stride_pad=0, state_dtype=0, eos=5, coarse=True,
             sample=None, special=None):
    """``sample`` = (inv_temperature, seed, draw) runs the categorical draw instead of argmax;
    ``special(x, mask, states)`` may rewrite the fp32 logits before they are converted."""
    mask, nxt = random_index(rng, Q, N)
    mask[3] = 0
    x = rng.standard_normal((B, N)).astype(np.float32) * 2
    if coarse:
        x = np.round(x, 1)                     # many exact ties
    x[0, : min(N, 6)] = [-0.0, 0.0, -np.inf, 0.0, -0.0, 0.0][: min(N, 6)]
    states = rng.integers(0, Q - 1, size=B).astype(np.int32)
    finished = np.zeros(B, np.uint8)
    if B > 4:
        states[2] = 3            # live state with an empty row
        states[3] = Q - 1        # dead state
        finished[4] = 1
        finished[1] = 2
    if B > 6 and eos >= 0:
        mask[states[6], eos >> 5] |= np.uint32(1 << (eos & 31))
        x[6, eos] = 1000.0
    if special is not None:
        special(x, mask, states)
    host_logits = f32_to_bf16_bits(x) if dtype == "bf16" else x
    st_o, fin_o = states.copy(), finished.copy()
    if sample is None:
        tok_o, out_o = fsm_oracle.mask_step(host_logits, st_o, fin_o, mask, nxt, Q - 1, eos,
                                            write_logits=(mode != "select"), threads=THREADS)
    else:
        tok_o, out_o = fsm_oracle.sample_step(host_logits, st_o, fin_o, mask, nxt, Q - 1, eos,
                                              sample[0], sample[1], sample[2],
                                              write_logits=(mode != "select"), threads=THREADS)

    dev = torch.device("cuda")
    stride = N + stride_pad
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    buf = torch.zeros((B, stride), dtype=tdt, device=dev)
    hl = torch.from_numpy(host_logits.view(np.int16) if dtype == "bf16" else host_logits)
    view = buf.view(torch.int16) if dtype == "bf16" else buf
    view[:, :N] = hl.to(dev)
    pad_before = view[:, N:].clone()
    d_mask = torch.from_numpy(mask.view(np.int32)).to(dev)
    if state_dtype == 1:
        d_next = torch.from_numpy(nxt.astype(np.uint16).view(np.int16)).to(dev).view(torch.uint16)
    else:
        d_next = torch.from_numpy(nxt).to(dev)
    d_states = torch.from_numpy(states).to(dev)
    d_fin = torch.from_numpy(finished).to(dev)
    d_tok = torch.full((B,), -77, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if mode == "inplace":
        out = buf
    elif mode == "outofplace":
        out = torch.full_like(buf, 7.0)
    else:
        out = None
    fg.fsm_debug_set(2, k)
    ldt = fg.FSM_LOGITS_BF16 if dtype == "bf16" else fg.FSM_LOGITS_F32
    if sample is None:
        rc = fg.guided_mask_step(buf, out, ldt, stride, d_states, d_fin, d_tok, d_mask, d_next,
                                 state_dtype, Q, N, B, Q - 1, eos, status)
    else:
        rc = fg.guided_sample_step(buf, out, ldt, stride, d_states, d_fin, d_tok, d_mask, d_next,
                                   state_dtype, Q, N, B, Q - 1, eos, sample[0], sample[1],
                                   sample[2], status)
    assert rc == 0, fg.fsm_status_string(rc)
    torch.cuda.synchronize()
    assert (d_tok.cpu().numpy() == tok_o).all(), (d_tok.cpu().numpy(), tok_o)
    assert (d_states.cpu().numpy() == st_o).all()
    assert (d_fin.cpu().numpy() == fin_o).all()
    assert int(status.item()) == 0
    if out is not None:
        oview = out.view(torch.int16) if dtype == "bf16" else out.view(torch.int32)
        got = oview[:, :N].cpu().numpy()
        want = out_o.view(np.int16) if dtype == "bf16" else out_o.view(np.int32)
        live = finished == 0
        assert (got[live] == want[live]).all()
        if mode == "inplace":                     # finished rows and row padding untouched
            assert (got[~live] == want[~live]).all()
            assert (view[:, N:] == pad_before).all()
        else:                                     # ... and still hold the fill value 7.0
            seven = 0x40E0 if dtype == "bf16" else 0x40E00000
            assert (got[~live] == seven).all()
            assert (oview[:, N:] == seven).all()
    return tok_o


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["inplace", "outofplace", "select"])
def test_step_modes(dtype, mode):
    run_case(np.random.default_rng(1), Q=11, N=5000, B=9, dtype=dtype, mode=mode)


@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_cluster_sizes(k):
    run_case(np.random.default_rng(k), Q=11, N=40000, B=7, dtype="bf16", mode="inplace", k=k)
    run_case(np.random.default_rng(k), Q=11, N=20000, B=7, dtype="f32", mode="select", k=k)


@pytest.mark.parametrize("N,pad", [(1, 7), (7, 1), (33, 7), (1000, 0), (1003, 5), (1000, 8), (4097, 7)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ragged_rows_and_narrow_alignment(N, pad, dtype):
    """Rows that are only 16-byte aligned, and lengths that leave a partial vector."""
    if dtype == "f32":
        pad = (-N) % 4 if (N + pad) % 4 else pad
    else:
        pad = pad if (N + pad) % 8 == 0 else (-N) % 8
    run_case(np.random.default_rng(N), Q=6, N=N, B=8, dtype=dtype, mode="inplace", stride_pad=pad, eos=0)
    run_case(np.random.default_rng(N), Q=6, N=N, B=8, dtype=dtype, mode="outofplace", stride_pad=pad, eos=-1)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["inplace", "outofplace", "select"])
def test_sample_step_modes(dtype, mode):
    toks = [run_case(np.random.default_rng(1), Q=11, N=5000, B=9, dtype=dtype, mode=mode,
                     sample=(1.0, 0x0123456789ABCDEF, draw)) for draw in (0, 1, 2**40 + 7)]
    assert any((toks[0] != t).any() for t in toks[1:])      # a new draw number, a new draw


@pytest.mark.parametrize("inv_t", [0.25, 1.0, 10.0])
@pytest.mark.parametrize("k", [1, 2, 4, 8])
def test_sample_step_cluster_sizes_and_temperatures(k, inv_t):
    run_case(np.random.default_rng(k), Q=11, N=40000, B=7, dtype="bf16", mode="inplace", k=k,
             sample=(inv_t, 99 + k, 5), coarse=False)
    run_case(np.random.default_rng(k), Q=11, N=20000, B=7, dtype="f32", mode="select", k=k,
             sample=(inv_t, 99 + k, 6), coarse=False)


@pytest.mark.parametrize("N,pad", [(1, 7), (7, 1), (33, 7), (1003, 5), (4097, 7)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_sample_step_ragged_rows(N, pad, dtype):
    if dtype == "f32":
        pad = (-N) % 4 if (N + pad) % 4 else pad
    else:
        pad = pad if (N + pad) % 8 == 0 else (-N) % 8
    run_case(np.random.default_rng(N), Q=6, N=N, B=8, dtype=dtype, mode="inplace", stride_pad=pad,
             eos=0, sample=(2.0, 7, 3))


def test_sample_step_rejects_bad_temperature():
    z = torch.zeros(8, dtype=torch.int32, device="cuda")
    x = torch.zeros((1, 8), device="cuda")
    f = torch.zeros(1, dtype=torch.uint8, device="cuda")
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        assert fg.guided_sample_step(x, x, fg.FSM_LOGITS_F32, 8, z, f, z, z, z, 0, 2, 8, 1, 1, -1,
                                     bad, 1, 1) == -6


def test_sample_workload_5_shape_steps_match_oracle():
    """Workload 5's shape (256 x 128,256 bf16 logits, workload 3's index), temperature 0.1
    as in the paper's runs: 3 steps in lock step with the oracle."""
    w = make_config(5)
    d = w.dfa
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    mask, nxt = mask_np(idx), next_np(idx)
    st = start_states(w)
    st_o, fin_o = st.copy(), np.zeros(w.B, np.uint8)
    d_st = torch.from_numpy(st).cuda()
    d_fin = torch.zeros(w.B, dtype=torch.uint8, device="cuda")
    d_tok = torch.zeros(w.B, dtype=torch.int32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(w.seed)
    for step in range(3):
        x = (torch.randn((w.B, w.N), generator=g, device="cuda") * w.logits_sigma).to(torch.bfloat16)
        host = x.view(torch.int16).cpu().numpy().view(np.uint16)
        tok_o, out_o = fsm_oracle.sample_step(host, st_o, fin_o, mask, nxt, d.dead, w.eos_id, 10.0,
                                              w.seed, step, threads=THREADS)
        idx.sample(x, d_st, d_fin, d_tok, 10.0, w.seed, step)
        torch.cuda.synchronize()
        assert (d_tok.cpu().numpy() == tok_o).all()
        assert (d_st.cpu().numpy() == st_o).all() and (d_fin.cpu().numpy() == fin_o).all()
        assert (x.view(torch.int16).cpu().numpy().view(np.uint16) == out_o).all()


def _tiny_values(dtype):
    """Positive values below, at and just above the subnormal boundary, exactly
    representable in ``dtype`` (bf16 keeps 8 significant bits of the fp32 pattern)."""
    if dtype == "bf16":
        bits = [0x00010000, 0x00030000, 0x007F0000, 0x00800000, 0x00810000]
    else:
        bits = [0x00000001, 0x00012345, 0x007FFFFF, 0x00800000, 0x00800001]
    return np.array(bits, dtype=np.uint32).view(np.float32)


def _subnormal_rows(dtype):
    """Rewrites rows 0, 5, 7 and 8 so that the comparison among the allowed logits is decided
    by subnormals, signed zeros and the smallest normal number, with ties among them; a
    comparison that flushed subnormals to zero would pick other tokens."""
    tiny = _tiny_values(dtype)

    def special(x, mask, states):
        B, N = x.shape
        rng = np.random.default_rng(B * 31 + N)

        def allowed_ids(row):
            q = states[row]
            bits = np.unpackbits(mask[q].view(np.uint8), bitorder="little")[:N]
            ids = np.flatnonzero(bits)
            assert len(ids) >= 8, "the seeded case gives these rows a non-empty state"
            return ids

        # row 0: every allowed logit in {-tiny, -0, +0, +tiny}; the largest subnormal appears
        # several times, zeros sit at lower ids
        ids = allowed_ids(0)
        vals = np.concatenate([tiny[:3], -tiny[:3], [0.0, -0.0]]).astype(np.float32)
        x[0, ids] = rng.choice(vals, size=len(ids))
        x[0, ids[:2]] = [0.0, -0.0]
        x[0, ids[len(ids) // 2]] = tiny[2]
        x[0, ids[-1]] = tiny[2]
        # row 5: all allowed logits are negative subnormals or -0.0 after some +0.0-free prefix:
        # the maximum is a signed zero, which must not tie with a flushed subnormal before it
        ids = allowed_ids(5)
        x[5, ids] = -rng.choice(tiny[:3], size=len(ids))
        x[5, ids[len(ids) // 3]] = -0.0
        x[5, ids[2 * len(ids) // 3]] = 0.0
        # row 7: smallest normal against the largest subnormal, both repeated
        ids = allowed_ids(7)
        x[7, ids] = rng.choice(np.array([tiny[2], -tiny[3], tiny[1], 0.0], dtype=np.float32), size=len(ids))
        x[7, ids[len(ids) // 2]] = tiny[3]
        x[7, ids[-2]] = tiny[3]
        # row 8: smallest subnormal alone above zeros
        ids = allowed_ids(8)
        x[8, ids] = rng.choice(np.array([0.0, -0.0, -tiny[0]], dtype=np.float32), size=len(ids))
        x[8, ids[-3]] = tiny[0]
    return special


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N,pad", [(5000, 0), (1003, 5)])
def test_subnormal_logits_compare_as_ieee_floats(dtype, N, pad):
    """Greedy selection among subnormals, signed zeros and the smallest normal (wide and
    narrow row alignment): bit-exact against the oracle."""
    if dtype == "f32":
        pad = (-N) % 4 if (N + pad) % 4 else pad
    else:
        pad = pad if (N + pad) % 8 == 0 else (-N) % 8
    for mode in ("inplace", "select"):
        tok = run_case(np.random.default_rng(3), Q=11, N=N, B=9, dtype=dtype, mode=mode,
                       stride_pad=pad, special=_subnormal_rows(dtype))
        assert (tok[[0, 5, 7, 8]] >= 0).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("k", [1, 4])
def test_subnormal_logits_in_the_categorical_draw(dtype, k):
    """With a huge inverse temperature a subnormal logit moves the score; the product must be
    formed from the unflushed value."""
    tiny = _tiny_values(dtype)

    def special(x, mask, states):
        rng = np.random.default_rng(17)
        x[:] = rng.choice(np.concatenate([tiny[:3], -tiny[:3], [0.0, -0.0]]).astype(np.float32),
                          size=x.shape)

    for inv_t in (1.0e38, 3.0e37):
        run_case(np.random.default_rng(k), Q=11, N=6000, B=9, dtype=dtype, mode="inplace", k=k,
                 sample=(inv_t, 4242, 9), coarse=False, special=special)


def test_u16_next_state_and_smooth_logits():
    run_case(np.random.default_rng(5), Q=300, N=9000, B=33, dtype="bf16", mode="inplace",
             state_dtype=1, coarse=False)


def test_bad_state_is_flagged_and_row_stuck():
    dev = torch.device("cuda")
    rng = np.random.default_rng(0)
    Q, N, B = 5, 640, 2
    mask, nxt = random_index(rng, Q, N)
    logits = torch.randn((B, N), device=dev)
    states = torch.tensor([77, 1], dtype=torch.int32, device=dev)
    fin = torch.zeros(B, dtype=torch.uint8, device=dev)
    tok = torch.zeros(B, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rc = fg.guided_mask_step(logits, logits, 0, N, states, fin, tok, torch.from_numpy(mask.view(np.int32)).to(dev),
                             torch.from_numpy(nxt).to(dev), 0, Q, N, B, Q - 1, -1, status)
    assert rc == 0
    torch.cuda.synchronize()
    assert int(status.item()) == 4 and fin.tolist() == [2, 0] and tok[0].item() == -1
    assert torch.isneginf(logits[0]).all()


def test_tiny_workload_decode_20_steps():
    """Workload 1: full index build, then 20 greedy masked steps at B = 1, fp32."""
    w = make_config(1)
    d = w.dfa
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    o_mask, o_next, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets,
                                               d.dead, w.eos_id)
    dev = torch.device("cuda")
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    fin = torch.zeros(1, dtype=torch.uint8, device=dev)
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    st_o, fin_o = np.zeros(1, np.int32), np.zeros(1, np.uint8)
    g = torch.Generator(device="cpu").manual_seed(w.seed)
    for step in range(w.steps):
        x = torch.randn((1, w.N), generator=g)
        if step == 15:
            x[0, w.eos_id] = 100.0
        xd = x.to(dev)
        idx.step(xd, st, fin, tok)
        tok_o, out_o = fsm_oracle.mask_step(x.numpy(), st_o, fin_o, o_mask, o_next, d.dead, w.eos_id)
        torch.cuda.synchronize()
        assert tok.item() == tok_o[0] and st.item() == st_o[0] and fin.item() == fin_o[0]
        if fin_o[0] == 0:
            assert (xd.cpu().numpy().view(np.int32) == out_o.view(np.int32)).all()


def test_workload_5_lockstep_1000_steps():
    """B = 256 bf16 rows over the workload-3 index for 1,000 steps: tokens, states
    and finished flags are compared every step, the full masked logits every step
    for the first 20 and every 50th step after that."""
    w = make_config(5)
    d = w.dfa
    idx = gpu_index(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets, d.dead, w.eos_id)
    o_mask, o_next = mask_np(idx), next_np(idx)      # index parity is covered by test_gpu_index
    ref_mask, ref_next, _ = fsm_oracle.index_build(d.trans, d.accept, w.vocab_bytes, w.vocab_offsets,
                                                   d.dead, w.eos_id, threads=THREADS)
    assert (o_mask == ref_mask).all() and (o_next == ref_next).all()
    o_mask, o_next = ref_mask, ref_next
    dev = torch.device("cuda")
    st0 = start_states(w)
    st = torch.from_numpy(st0).to(dev)
    fin = torch.zeros(w.B, dtype=torch.uint8, device=dev)
    tok = torch.zeros(w.B, dtype=torch.int32, device=dev)
    st_o, fin_o = st0.copy(), np.zeros(w.B, np.uint8)
    g = torch.Generator(device=dev)
    sigma = w.logits_sigma
    n_finished_seen = 0
    for step in range(w.steps):
        g.manual_seed(w.seed * 1000 + step)
        x = (torch.randn((w.B, w.N), generator=g, device=dev) * sigma).to(torch.bfloat16)
        if step % 97 == 5:      # let EOS win in a few rows now and then
            x[step % w.B, w.eos_id] = 60.0
        host = x.view(torch.int16).cpu().numpy().view(np.uint16)
        full = step < 20 or step % 50 == 0
        idx.step(x, st, fin, tok)
        tok_o, out_o = fsm_oracle.mask_step(host, st_o, fin_o, o_mask, o_next, d.dead, w.eos_id,
                                            write_logits=full, threads=THREADS)
        torch.cuda.synchronize()
        assert (tok.cpu().numpy() == tok_o).all(), step
        assert (st.cpu().numpy() == st_o).all(), step
        assert (fin.cpu().numpy() == fin_o).all(), step
        if full:
            assert (x.view(torch.int16).cpu().numpy().view(np.uint16) == out_o).all(), step
        n_finished_seen = int((fin_o != 0).sum())
    assert 0 < n_finished_seen < w.B
