/*
 * TEST INFRASTRUCTURE - CPU oracle for FSM vocabulary indexing and the masked
 * greedy decode step.  Plain, slow, scalar; written from the paper's
 * definitions.  It shares no code with the CUDA library and must never be
 * linked into, imported by or called from the product path: only the tests,
 * the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows (paper: "Efficient Guided Generation for Large Language
 * Models", arXiv 2307.09702):
 *   - Definition 1: the automaton (Q, Sigma, delta, q0, F) with integer states;
 *     here delta is a dense table over the 256 byte values and one designated
 *     absorbing state `dead` stands for "delta(q, b) is undefined".
 *   - Algorithm 3 (find_sub_sequences): walk a vocabulary string through delta
 *     from a start state, abandoning the walk at the first undefined transition.
 *   - Algorithm 4 (map_states_to_vocab): token v joins sigma(q) for every start
 *     state q whose walk survives.  F is never consulted for ordinary tokens.
 *   - Section 3 / Section 4 example ("f" -> (0,1), (1,2), (2,2)): a state
 *     sequence is the start state followed by the state after each character, so
 *     its last element is the state the automaton is in after the token; that is
 *     the tracked state of Section 3 ("FSM states can then be tracked").
 *   - Algorithm 2: per step, mask the logits with m(sigma(state)), pick a token,
 *     stop on EOS, otherwise append and continue.  Selection here is the greedy
 *     rule of Section 2.1 (highest-probability token).
 *
 * Readings where the paper is silent (each is also a line of the design notes):
 *   - sigma is stored as a packed bitmask, bit (v & 31) of word (v >> 5) of row q,
 *     padding bits zero; the end state of each walk is stored in a dense table,
 *     with `dead` where the token is not allowed.
 *   - EOS has no byte string.  It is allowed exactly in accepting states (F) and
 *     keeps the state.  Zero-length tokens other than EOS are never allowed.
 *   - The dead state's own row is empty whatever its table row holds.
 *   - m (.) alpha on logits: disallowed entries become -inf, allowed entries are
 *     passed through bit for bit.
 *   - Ties in the maximum go to the lowest token id; comparison is IEEE float
 *     comparison (so -0.0 == +0.0); the maximum is over allowed tokens only.
 *   - A row with no allowed token finishes as "stuck" (2); a row that picks EOS
 *     finishes (1); finished rows are left untouched and report token -1.
 *
 * Sampling (oracle_sample_step) is Algorithm 2 as printed: the token is drawn from
 * Categorical(softmax(masked logits / temperature)).  The draw is the Gumbel-max
 * form of that distribution - argmax over the allowed tokens of
 * logit / temperature + G, G = -ln(-ln(u)) - so that, with the random bits fixed by
 * a counter-based generator, the result is a pure function of its inputs:
 *   - bits: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers:
 *     as easy as 1, 2, 3", SC'11), key = the two halves of the 64-bit seed,
 *     counter = (token id / 4, batch row, low and high half of the 64-bit draw
 *     number); token v takes output word v % 4;
 *   - u = (2 * (bits >> 9) + 1) * 2^-24, an odd multiple of 2^-24 strictly inside
 *     (0, 1), exact in fp32;
 *   - ln in fp32, every operation rounded to nearest: x = m * 2^e with m in
 *     (sqrt(1/2), sqrt(2)], s = (m - 1) / (m + 1), ln m = 2 s (1 + s^2/3 + s^4/5 +
 *     s^6/7 + s^8/9) evaluated by Horner's rule with fused multiply-adds, ln x =
 *     fma(e, ln 2, ln m)  (the textbook atanh series; truncation error below 2e-9);
 *   - score = fma(logit, 1/temperature, G) in fp32; largest score wins, ties go to
 *     the lowest token id.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_RANGE (-2)

/* delta*(q, bytes of v) with Algorithm 3's abandonment: returns `dead` as soon
 * as one transition leads there.  *lookups counts evaluations of delta. */
static int32_t walk_token(const int32_t *trans, int32_t dead, int32_t q,
                          const uint8_t *bytes, int32_t len, int64_t *lookups)
{
    int32_t s = q;
    for (int32_t i = 0; i < len; ++i) {
        s = trans[(size_t)s * 256 + bytes[i]];
        ++*lookups;
        if (s == dead)
            break;
    }
    return s;
}

/*
 * Index rows q_begin <= q < q_end.
 *   allowed_mask: [(q_end - q_begin) * W] words, W = ceil(N / 32)
 *   next_state:   [(q_end - q_begin) * N] or NULL
 *   lookups:      optional; total delta evaluations an abandoning walk makes
 *   threads:      > 1 splits the state loop with OpenMP (timing convenience only)
 */
int oracle_index_build(const int32_t *trans, const uint8_t *accept,
                       const uint8_t *vocab_bytes, const int32_t *vocab_offsets,
                       int32_t Q, int32_t N, int32_t dead, int32_t eos_id,
                       int32_t q_begin, int32_t q_end,
                       uint32_t *allowed_mask, int32_t *next_state,
                       int64_t *lookups, int32_t threads)
{
    if (!trans || !accept || !vocab_offsets || !allowed_mask || Q <= 0 || N <= 0)
        return ORACLE_ERR_ARG;
    if (dead < 0 || dead >= Q || q_begin < 0 || q_end > Q || q_begin > q_end)
        return ORACLE_ERR_RANGE;
    const int64_t W = ((int64_t)N + 31) / 32;
    int64_t total = 0;
    (void)threads;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : total) num_threads(threads > 1 ? threads : 1)
    for (int32_t q = q_begin; q < q_end; ++q) {
        uint32_t *mrow = allowed_mask + (size_t)(q - q_begin) * W;
        int32_t *nrow = next_state ? next_state + (size_t)(q - q_begin) * N : NULL;
        memset(mrow, 0, (size_t)W * sizeof(uint32_t));
        for (int32_t v = 0; v < N; ++v) {
            int32_t len = vocab_offsets[v + 1] - vocab_offsets[v];
            int32_t s;
            if (v == eos_id)
                s = (q != dead && accept[q]) ? q : dead;
            else if (q == dead || len == 0)
                s = dead;
            else
                s = walk_token(trans, dead, q, vocab_bytes + vocab_offsets[v], len, &total);
            if (s != dead)
                mrow[v >> 5] |= (uint32_t)1 << (v & 31);
            if (nrow)
                nrow[v] = s;
        }
    }
    if (lookups)
        *lookups = total;
    return ORACLE_OK;
}

static float bf16_to_float(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * One masked greedy step over B rows (Algorithm 2 with argmax selection).
 *   dtype: 0 = fp32 logits, 1 = bf16 logits (bit patterns in uint16)
 *   logits_out: may equal logits_in, or be NULL (select only)
 *   next_state: int32 [Q * N]
 */
int oracle_mask_step(const void *logits_in, void *logits_out, int32_t dtype,
                     int64_t row_stride, int32_t *states, uint8_t *finished,
                     int32_t *tokens_out, const uint32_t *allowed_mask,
                     const int32_t *next_state, int32_t Q, int32_t N, int32_t B,
                     int32_t dead, int32_t eos_id, int32_t threads)
{
    if (!logits_in || !states || !finished || !tokens_out || !allowed_mask || !next_state)
        return ORACLE_ERR_ARG;
    if (Q <= 0 || N <= 0 || B < 0 || row_stride < N || (dtype != 0 && dtype != 1))
        return ORACLE_ERR_ARG;
    const int64_t W = ((int64_t)N + 31) / 32;
    int bad = 0;
    (void)threads;
    (void)dead;
#pragma omp parallel for schedule(static) num_threads(threads > 1 ? threads : 1)
    for (int32_t i = 0; i < B; ++i) {
        if (finished[i]) {
            tokens_out[i] = -1;
            continue;
        }
        int32_t q = states[i];
        if (q < 0 || q >= Q) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        const uint32_t *mrow = allowed_mask + (size_t)q * W;
        int32_t best = -1;
        float best_val = 0.0f;
        for (int32_t v = 0; v < N; ++v) {
            size_t at = (size_t)i * row_stride + v;
            int allowed = (mrow[v >> 5] >> (v & 31)) & 1;
            float x;
            if (dtype == 0) {
                uint32_t bits = ((const uint32_t *)logits_in)[at];
                memcpy(&x, &bits, sizeof x);
                if (logits_out)
                    ((uint32_t *)logits_out)[at] = allowed ? bits : 0xFF800000u;
            } else {
                uint16_t bits = ((const uint16_t *)logits_in)[at];
                x = bf16_to_float(bits);
                if (logits_out)
                    ((uint16_t *)logits_out)[at] = allowed ? bits : (uint16_t)0xFF80u;
            }
            if (allowed && (best < 0 || x > best_val)) {
                best = v;
                best_val = x;
            }
        }
        if (best < 0) {
            finished[i] = 2;
            tokens_out[i] = -1;
        } else if (best == eos_id) {
            finished[i] = 1;
            tokens_out[i] = best;
        } else {
            tokens_out[i] = best;
            states[i] = next_state[(size_t)q * N + best];
        }
    }
    return bad ? ORACLE_ERR_RANGE : ORACLE_OK;
}


/* ------------------------------------------------------------------------------------
 * Sampling step (Algorithm 2 with the categorical draw), see the header comment.
 */

/* Philox4x32-10: ten rounds of two 32x32->64 multiplications whose high halves are
 * XORed with the other counter words and the round key; the key grows by the two
 * Weyl constants after every round. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0;
        c1 = n1;
        c2 = n2;
        c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

/* ln x for a positive normal fp32 x, in fp32 operations rounded to nearest. */
float oracle_ln_f32(float x)
{
    uint32_t b;
    memcpy(&b, &x, sizeof b);
    int32_t e = (int32_t)(b >> 23) - 127;
    uint32_t mb = (b & 0x007FFFFFu) | 0x3F800000u;
    float m;
    memcpy(&m, &mb, sizeof m);          /* m in [1, 2) */
    if (m > 1.41421354f) {              /* fold into (sqrt(1/2), sqrt(2)] */
        m = m * 0.5f;
        e += 1;
    }
    const float s = (m - 1.0f) / (m + 1.0f);
    const float z = s * s;
    float p = fmaf(z, 1.0f / 9.0f, 1.0f / 7.0f);
    p = fmaf(z, p, 1.0f / 5.0f);
    p = fmaf(z, p, 1.0f / 3.0f);
    p = fmaf(z, p, 1.0f);
    const float lnm = (s + s) * p;
    return fmaf((float)e, 0.693147182f, lnm);
}

/* Standard Gumbel variate from 32 random bits. */
float oracle_gumbel_f32(uint32_t bits)
{
    const float u = (float)(2u * (bits >> 9) + 1u) * 5.9604644775390625e-08f; /* 2^-24 */
    const float y = -oracle_ln_f32(u);  /* Exp(1) variate, > 0 */
    return -oracle_ln_f32(y);
}

int oracle_sample_step(const void *logits_in, void *logits_out, int32_t dtype,
                       int64_t row_stride, int32_t *states, uint8_t *finished,
                       int32_t *tokens_out, const uint32_t *allowed_mask,
                       const int32_t *next_state, int32_t Q, int32_t N, int32_t B,
                       int32_t dead, int32_t eos_id, float inv_temperature, uint64_t seed,
                       uint64_t draw, int32_t threads)
{
    if (!logits_in || !states || !finished || !tokens_out || !allowed_mask || !next_state)
        return ORACLE_ERR_ARG;
    if (Q <= 0 || N <= 0 || B < 0 || row_stride < N || (dtype != 0 && dtype != 1))
        return ORACLE_ERR_ARG;
    const int64_t W = ((int64_t)N + 31) / 32;
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    int bad = 0;
    (void)dead;
#pragma omp parallel for schedule(static) num_threads(threads > 1 ? threads : 1)
    for (int32_t i = 0; i < B; ++i) {
        if (finished[i]) {
            tokens_out[i] = -1;
            continue;
        }
        int32_t q = states[i];
        if (q < 0 || q >= Q) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        const uint32_t *mrow = allowed_mask + (size_t)q * W;
        int32_t best = -1;
        float best_score = 0.0f;
        for (int32_t v = 0; v < N; ++v) {
            size_t at = (size_t)i * row_stride + v;
            int allowed = (mrow[v >> 5] >> (v & 31)) & 1;
            float x;
            if (dtype == 0) {
                uint32_t bits = ((const uint32_t *)logits_in)[at];
                memcpy(&x, &bits, sizeof x);
                if (logits_out)
                    ((uint32_t *)logits_out)[at] = allowed ? bits : 0xFF800000u;
            } else {
                uint16_t bits = ((const uint16_t *)logits_in)[at];
                x = bf16_to_float(bits);
                if (logits_out)
                    ((uint16_t *)logits_out)[at] = allowed ? bits : (uint16_t)0xFF80u;
            }
            if (!allowed)
                continue;
            const uint32_t ctr[4] = {(uint32_t)v >> 2, (uint32_t)i, (uint32_t)draw,
                                     (uint32_t)(draw >> 32)};
            uint32_t r[4];
            oracle_philox4x32_10(ctr, key, r);
            const float score = fmaf(x, inv_temperature, oracle_gumbel_f32(r[v & 3]));
            if (best < 0 || score > best_score) {
                best = v;
                best_score = score;
            }
        }
        if (best < 0) {
            finished[i] = 2;
            tokens_out[i] = -1;
        } else if (best == eos_id) {
            finished[i] = 1;
            tokens_out[i] = best;
        } else {
            tokens_out[i] = best;
            states[i] = next_state[(size_t)q * N + best];
        }
    }
    return bad ? ORACLE_ERR_RANGE : ORACLE_OK;
}
