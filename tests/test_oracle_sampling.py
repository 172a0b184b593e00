"""Pins of the sampling oracle (paper Algorithm 2 with the categorical draw): the
counter-based generator against its published known answers, the fp32 logarithm
against the mathematical one, the Gumbel variates against their closed-form moments,
and the sampled frequencies against softmax(masked logits / temperature)."""
import math
import os

import numpy as np
import pytest

from oracle import fsm_oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for r in rows:
        words = [int(x, 16) for x in r]
        assert fsm_oracle.philox4x32_10(words[0:4], words[4:6]) == words[6:10]


def test_philox_is_a_bijection_of_the_counter_on_a_sample():
    """Distinct counters give distinct blocks (a keyed permutation), and the words look
    uniform: mean of 4,000 words within 5 sigma of 2^31."""
    seen, words = set(), []
    for i in range(1000):
        out = tuple(fsm_oracle.philox4x32_10([i, 3, 0, 0], [17, 5]))
        assert out not in seen
        seen.add(out)
        words += out
    mean = np.mean(words)
    assert abs(mean - 2**31) < 5 * (2**32 / math.sqrt(12)) / math.sqrt(len(words))


def test_fp32_logarithm_against_math_log():
    xs = np.exp(np.linspace(math.log(2.0**-24), math.log(40.0), 4001))
    for x in xs:
        x32 = float(np.float32(x))
        got = fsm_oracle.ln_f32(x32)
        want = math.log(x32)
        assert abs(got - want) <= 2.5e-7 * max(1.0, abs(want)), (x32, got, want)
    assert fsm_oracle.ln_f32(1.0) == 0.0
    assert fsm_oracle.ln_f32(2.0) == float(np.float32(0.693147182))
    assert fsm_oracle.ln_f32(float(np.float32(1 - 2.0**-24))) < 0.0     # -ln u stays positive


def test_gumbel_variates_definition_and_moments():
    rng = np.random.default_rng(3)
    bits = rng.integers(0, 2**32, size=20000, dtype=np.uint64)
    g = np.array([fsm_oracle.gumbel_f32(int(b)) for b in bits])
    u = (2 * (bits >> 9) + 1).astype(np.float64) * 2.0**-24
    assert ((u > 0) & (u < 1)).all()
    want = -np.log(-np.log(u))
    assert np.max(np.abs(g - want) / np.maximum(1.0, np.abs(want))) < 2e-6
    # standard Gumbel: mean = Euler's constant, variance = pi^2 / 6
    assert abs(g.mean() - 0.5772156649) < 5 * math.sqrt(math.pi**2 / 6 / len(g))
    assert abs(g.var() - math.pi**2 / 6) < 0.08
    # extreme words stay finite
    assert math.isfinite(fsm_oracle.gumbel_f32(0)) and math.isfinite(fsm_oracle.gumbel_f32(2**32 - 1))


def _tiny_index(N=8, allowed=(0, 2, 3, 5, 7)):
    mask = np.zeros((2, 1), dtype=np.uint32)
    for v in allowed:
        mask[0, 0] |= np.uint32(1 << v)
    nxt = np.full((2, N), 1, dtype=np.int32)
    nxt[0, list(allowed)] = 0
    return mask, nxt


@pytest.mark.parametrize("inv_t", [1.0, 0.5, 3.0])
def test_sampled_frequencies_follow_the_masked_softmax(inv_t):
    """Categorical(softmax(m . alpha / T)): 100,000 draws on 8 tokens, 5 allowed."""
    N, allowed = 8, (0, 2, 3, 5, 7)
    mask, nxt = _tiny_index(N, allowed)
    x = np.array([0.3, 9.0, -1.2, 0.9, 9.0, 0.0, 9.0, 1.5], dtype=np.float32)
    B, draws = 1000, 100
    logits = np.tile(x, (B, 1))
    counts = np.zeros(N)
    for d in range(draws):
        st, fin = np.zeros(B, np.int32), np.zeros(B, np.uint8)
        tok, out = fsm_oracle.sample_step(logits, st, fin, mask, nxt, 1, -1, inv_t, 4242, d)
        counts += np.bincount(tok, minlength=N)
        assert np.isneginf(out[:, [1, 4, 6]]).all() and (out[:, list(allowed)] == x[list(allowed)]).all()
    assert counts[[1, 4, 6]].sum() == 0                     # masked tokens are never drawn
    z = np.array([x[v] * inv_t for v in allowed], dtype=np.float64)
    p = np.exp(z - z.max())
    p /= p.sum()
    n = B * draws
    for v, pv in zip(allowed, p):
        assert abs(counts[v] / n - pv) < 5 * math.sqrt(pv * (1 - pv) / n) + 1e-4, (v, counts[v] / n, pv)


def test_low_temperature_is_greedy_and_rows_draw_independently():
    N, allowed = 8, (0, 2, 3, 5, 7)
    mask, nxt = _tiny_index(N, allowed)
    x = np.array([0.3, 9.0, -1.2, 0.9, 9.0, 0.0, 9.0, 1.5], dtype=np.float32)
    logits = np.tile(x, (64, 1))
    st, fin = np.zeros(64, np.int32), np.zeros(64, np.uint8)
    tok, _ = fsm_oracle.sample_step(logits, st, fin, mask, nxt, 1, -1, 1000.0, 1, 0)
    assert (tok == 7).all()                                 # the largest allowed logit
    st[:] = 0
    tok, _ = fsm_oracle.sample_step(logits, st, fin, mask, nxt, 1, -1, 1.0, 1, 0)
    assert len(set(tok.tolist())) > 1                       # the batch row enters the counter
    tok2, _ = fsm_oracle.sample_step(logits, st.copy() * 0, fin, mask, nxt, 1, -1, 1.0, 1, 0)
    assert (tok == tok2).all()                              # same seed and draw: same tokens
    tok3, _ = fsm_oracle.sample_step(logits, st.copy() * 0, fin, mask, nxt, 1, -1, 1.0, 2, 0)
    assert (tok != tok3).any()                              # another seed: another draw


def test_sample_step_bookkeeping_matches_the_greedy_step():
    """EOS, stuck rows, finished rows: same rules as the greedy step."""
    N = 8
    mask, nxt = _tiny_index(N, (4,))
    mask = np.vstack([mask, np.zeros((1, 1), np.uint32)])   # state 2: empty row
    nxt = np.vstack([nxt, np.full((1, N), 1, np.int32)])
    logits = np.zeros((4, N), dtype=np.float32)
    st = np.array([0, 2, 0, 0], dtype=np.int32)
    fin = np.array([0, 0, 1, 0], dtype=np.uint8)
    tok, out = fsm_oracle.sample_step(logits, st, fin, mask, nxt, 1, 4, 1.0, 9, 9)
    assert tok.tolist() == [4, -1, -1, 4]
    assert fin.tolist() == [1, 2, 1, 1] and st.tolist() == [0, 2, 0, 0]
    assert np.isneginf(out[1]).all() and (out[2] == 0).all()
