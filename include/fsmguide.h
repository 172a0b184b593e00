/*
 * fsmguide - FSM vocabulary indexing and masked greedy decoding on NVIDIA B200
 * (sm_100a), after "Efficient Guided Generation for Large Language Models"
 * (arXiv 2307.09702).
 *
 * C ABI.  Unless an argument is marked HOST, every array pointer is a DEVICE
 * pointer owned by the caller; the library neither allocates nor frees device
 * memory and never aborts.  The build and decode calls never synchronise the
 * stream: all their work is enqueued on `cuda_stream` (a cudaStream_t passed as
 * void*, NULL = the default stream) and may still be running when a call
 * returns.  The index-file calls and fsm_profile_read block, and say so.
 *
 * Return value: FSM_OK, or a negative FSM_ERR_* code.  Errors that can be
 * detected from the scalar arguments and pointer values are returned before
 * anything is enqueued.  Faults in the *contents* of device arrays cannot be
 * seen from the host without a synchronisation; kernels neutralise them (see
 * each argument) and OR a FSM_FLAG_* bit into `*status_word`, a device int32
 * the caller zeroes beforehand and may read after synchronising.  `status_word`
 * may be NULL.
 */
#ifndef FSMGUIDE_H
#define FSMGUIDE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FSM_OK 0
#define FSM_ERR_NULL (-1)      /* a required pointer is NULL */
#define FSM_ERR_SHAPE (-2)     /* a size is non-positive or inconsistent */
#define FSM_ERR_ALIGN (-3)     /* a pointer or stride breaks the stated alignment */
#define FSM_ERR_DTYPE (-4)     /* unknown dtype code, or FSM_STATE_U16 with Q > 65535 */
#define FSM_ERR_WORKSPACE (-5) /* workspace missing or smaller than the query says */
#define FSM_ERR_RANGE (-6)     /* dead_state, eos_id or a row range is out of range */
#define FSM_ERR_CUDA (-7)      /* a CUDA runtime call failed (launch, attribute) */
#define FSM_ERR_DEVICE (-8)    /* no device of compute capability 10.x is current */
#define FSM_ERR_IO (-9)        /* an index file cannot be opened, read or written, or is shorter
                                  than its header says */
#define FSM_ERR_FORMAT (-10)   /* not an index file of this version, a file for another problem
                                  (sizes, dtype, dead/EOS ids or input digest differ from what
                                  the caller expects), or its contents fail their checksum */

/* Bits of *status_word (device int32). */
#define FSM_FLAG_TRANS_RANGE 1   /* a transition outside [0,Q) was read; treated as dead */
#define FSM_FLAG_OFFSETS 2       /* vocab_offsets not non-decreasing / out of bounds; token
                                    treated as empty */
#define FSM_FLAG_STATE_RANGE 4   /* states[i] outside [0,Q); row finished as stuck */
#define FSM_FLAG_CLASS_SPLIT 8   /* informational: two byte columns hashed alike but differ;
                                    the build took the uncompressed path (still exact) */
#define FSM_FLAG_WAIT_TIMEOUT 16 /* a bounded wait on an on-chip copy gave up; output invalid */
#define FSM_FLAG_CSR_OVERFLOW 32 /* fsm_index_build_csr: more allowed pairs than `capacity`;
                                    row_offsets is complete, entries beyond capacity are missing */
#define FSM_FLAG_INDEX 64        /* range-checked library only (built with -DFSM_CHECKED, file
                                    name ending in _checked): an index computed from data was
                                    outside its array; the access was skipped, output invalid */

typedef enum { FSM_STATE_I32 = 0, FSM_STATE_U16 = 1 } fsm_state_dtype;
typedef enum { FSM_LOGITS_F32 = 0, FSM_LOGITS_BF16 = 1 } fsm_logits_dtype;

/* Text for a return code ("FSM_OK", "FSM_ERR_NULL: ...").  HOST string, static. */
const char* fsm_status_string(int status);

/* FSM_OK if the current device has compute capability 10.x, else FSM_ERR_DEVICE
 * (FSM_ERR_CUDA if the runtime cannot be queried). */
int fsm_device_check(void);

/* Bytes of device scratch fsm_index_build needs for an automaton of Q states and a
 * vocabulary of N tokens whose byte strings total vocab_nbytes.  0 on bad sizes.
 * Pure host arithmetic; needs no device. */
size_t fsm_index_workspace_bytes(int32_t Q, int32_t N, int64_t vocab_nbytes);

/*
 * Vocabulary index construction (paper Section 3, Algorithms 3 and 4).
 *
 * For every state q in [0,Q) and every token v in [0,N) the token's bytes are
 * walked through delta from q (Algorithm 3); the walk is abandoned at the first
 * transition into `dead_state`, the designated absorbing state that stands for
 * "delta undefined".  A token whose walk survives belongs to sigma(q)
 * (Algorithm 4) and the state the walk ends in is recorded, so that the FSM
 * state can be carried from token to token (Section 3).  Accepting states are
 * not consulted for ordinary tokens.
 *
 *   dfa_trans      int32 [Q*256], row-major: dfa_trans[q*256 + b] = delta(q, b)
 *                  (Definition 1, over the 256 byte values).  Values outside [0,Q)
 *                  count as dead and raise FSM_FLAG_TRANS_RANGE.  The dead state's
 *                  own row is never consulted.
 *   accept         uint8 [Q], non-zero = state in F.
 *   vocab_bytes    uint8 [vocab_offsets[N]], token byte strings back to back.
 *   vocab_offsets  int32 [N+1], vocab_offsets[0] = 0, non-decreasing.  Tokens may
 *                  have any length; a zero-length token is never allowed.
 *   vocab_nbytes   HOST scalar equal to vocab_offsets[N] (used for bounds only).
 *   Q, N           number of states (dead included), number of tokens.
 *   dead_state     in [0,Q).
 *   eos_id         token id of EOS, or -1.  EOS has no byte string: it is allowed
 *                  exactly in accepting states and leads back to the same state.
 *   allowed_mask   out uint32 [Q*W], W = ceil(N/32).  Bit (v & 31) of word
 *                  q*W + (v >> 5) is 1 iff v is in sigma(q).  Every word is written;
 *                  bits for v >= N are 0.  4-byte aligned.
 *   next_state     out [Q*N] of `state_dtype`: the end state of the walk, or
 *                  dead_state where the token is not allowed.  NULL = bitmask only.
 *                  Aligned to its element size.
 *   state_dtype    FSM_STATE_I32, or FSM_STATE_U16 (requires Q <= 65535).
 *   workspace      device scratch, 256-byte aligned, at least
 *                  fsm_index_workspace_bytes(Q, N, vocab_nbytes) bytes (the compressed
 *                  table, the token records, the bit planes of the one-byte tokens:
 *                  about 7 MB for 1,001 states and 128,256 tokens; for Q < 256 also
 *                  Q * N 16-bit entries, from which fsm_index_build_csr cuts its rows).
 *                  Contents on entry are irrelevant; concurrent calls need separate
 *                  workspaces.
 *   status_word    device int32 or NULL.
 *
 * fsm_index_build_rows builds only rows q_begin <= q < q_end, written to
 * allowed_mask[(q - q_begin)*W ..] and next_state[(q - q_begin)*N ..]; it is the
 * unit of work when the states are sharded over several GPUs.
 */
int fsm_index_build(const int32_t* dfa_trans, const uint8_t* accept,
                    const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                    int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                    int32_t eos_id, uint32_t* allowed_mask, void* next_state,
                    int32_t state_dtype, void* workspace, size_t workspace_bytes,
                    int32_t* status_word, void* cuda_stream);

int fsm_index_build_rows(const int32_t* dfa_trans, const uint8_t* accept,
                         const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                         int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                         int32_t eos_id, int32_t q_begin, int32_t q_end,
                         uint32_t* allowed_mask, void* next_state, int32_t state_dtype,
                         void* workspace, size_t workspace_bytes, int32_t* status_word,
                         void* cuda_stream);

/*
 * The index in the paper's own form (Section 3, Algorithm 4: sigma maps a state to the
 * *set* of allowed tokens), as compressed rows.  Most (state, token) pairs are not
 * allowed (the paper notes that the map's memory grows with the number of states only),
 * so this form is a small fraction of the dense next-state table.
 *
 *   allowed_mask   out, as fsm_index_build.
 *   row_offsets    out, int64 [Q+1], 8-byte aligned: row q's entries are
 *                  row_offsets[q] .. row_offsets[q+1]-1; row_offsets[Q] is the number of
 *                  allowed pairs.
 *   csr_tokens     out, int32 [capacity]: the allowed token ids of each row, increasing.
 *   csr_next       out, int32 [capacity]: the state each of them leads to (for EOS: the
 *                  state itself).
 *   capacity       entries the two arrays hold.  If the index has more, the first
 *                  `capacity` entries are written, FSM_FLAG_CSR_OVERFLOW is raised and
 *                  row_offsets (always complete) tells the size needed.
 * Other arguments, workspace and status word as fsm_index_build.
 */
int fsm_index_build_csr(const int32_t* dfa_trans, const uint8_t* accept,
                        const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                        int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                        int32_t eos_id, uint32_t* allowed_mask, int64_t* row_offsets,
                        int32_t* csr_tokens, int32_t* csr_next, int64_t capacity,
                        void* workspace, size_t workspace_bytes, int32_t* status_word,
                        void* cuda_stream);

/*
 * Index build without caller-provided scratch.  The paper has no counterpart:
 * this entry point exists for callers that cannot obtain device scratch memory
 * themselves - a plug-in running inside a host application that has handed the
 * whole device to its own memory pool, a serving loop in which cudaMalloc (and
 * the implicit device synchronisation it brings) is forbidden, or a process
 * that must not grow its footprint after start-up.
 *
 * It computes exactly what fsm_index_build computes (same arguments, same
 * outputs, same status flags), but takes its scratch from a fixed array of
 * FSM_STATIC_SCRATCH_BYTES that lives inside the library's device image: every
 * GPU on which the library is loaded holds those bytes until the process
 * exits.  The call allocates and frees nothing.
 *
 *   - Size limit: the array holds the compressed transition table and the class
 *     records of the tokens; it has no room for the scratch of the faster
 *     work-avoiding walks, so this entry point always uses the dense walk (same
 *     results, lower throughput).  The build is refused with FSM_ERR_WORKSPACE,
 *     before anything is enqueued, when that scratch (about 270 KB + 528 bytes per
 *     state + 20 bytes per token) exceeds FSM_STATIC_SCRATCH_BYTES - as a guide: about
 *     1,000 states with 55,000 tokens, or 2,000 states with 30,000 tokens.  Larger
 *     problems need fsm_index_build and a workspace.
 *   - First call on each device: the library looks up the device address of its
 *     scratch array (the device must be current).  Make that first call outside
 *     any stream capture.
 *   - The array is shared by every call on that device and still holds the
 *     previous call's intermediates; the build overwrites every part it reads,
 *     so nothing has to be cleared in between.  Two calls whose kernels may run
 *     at the same time on one device (different streams or threads) race on the
 *     array: serialise them.
 */
#define FSM_STATIC_SCRATCH_BYTES (2u << 20)
int fsm_index_build_static(const int32_t* dfa_trans, const uint8_t* accept,
                           const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                           int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                           int32_t eos_id, uint32_t* allowed_mask, void* next_state,
                           int32_t state_dtype, int32_t* status_word, void* cuda_stream);

/*
 * One step of guided greedy decoding for a batch (paper Algorithm 2, with the
 * greedy selection rule of Section 2.1 in place of the categorical draw).
 *
 * For every row i with finished[i] == 0, with q = states[i]:
 *   mask    logits_out[i][v] = logits_in[i][v] (bit for bit) if v is in sigma(q),
 *           else -inf  (the boolean mask m of Section 2.2 applied to the logits);
 *   select  tok = the allowed token with the largest logit, compared as IEEE
 *           floats (so -0.0 == +0.0); ties go to the lowest token id; NaN logits
 *           are outside the contract;
 *   advance if no token is allowed: finished[i] = 2, tokens_out[i] = -1;
 *           else if tok == eos_id:  finished[i] = 1, tokens_out[i] = tok;
 *           else tokens_out[i] = tok and states[i] = next_state[q*N + tok].
 * Rows with finished[i] != 0 are left untouched (their logits_out row is not
 * written) and report tokens_out[i] = -1.
 *
 *   logits_in    [B*row_stride] of `logits_dtype`, 16-byte aligned; row i starts
 *                at element i*row_stride.  row_stride >= N and row_stride*sizeof
 *                (element) a multiple of 16.
 *   logits_out   same layout; may equal logits_in (in place) or be NULL (select and
 *                advance only).  Partial overlap is not allowed.
 *   states       int32 [B], in/out.  A value outside [0,Q) finishes the row as stuck
 *                and raises FSM_FLAG_STATE_RANGE.
 *   finished     uint8 [B], in/out: 0 live, 1 finished by EOS, 2 stuck.
 *   tokens_out   int32 [B], out.
 *   allowed_mask, next_state, state_dtype, Q, N, dead_state, eos_id
 *                the index as fsm_index_build wrote it (all Q rows).
 *   B            batch rows, >= 0 (0 is a no-op).
 */
int guided_mask_step(const void* logits_in, void* logits_out, int32_t logits_dtype,
                     int64_t row_stride, int32_t* states, uint8_t* finished,
                     int32_t* tokens_out, const uint32_t* allowed_mask,
                     const void* next_state, int32_t state_dtype, int32_t Q, int32_t N,
                     int32_t B, int32_t dead_state, int32_t eos_id, int32_t* status_word,
                     void* cuda_stream);

/*
 * One step of guided decoding with the categorical draw of paper Algorithm 2
 * ("Sample s ~ Categorical(alpha~)"): as guided_mask_step, except that the token is
 * drawn from the softmax of the masked logits divided by the temperature
 * (Section 2.1 calls this multinomial sampling; the paper's runs use temperature 0.1).
 *
 * The draw is the Gumbel-max form of that distribution, so that the step is a pure
 * function of its arguments:
 *   tok = argmax over v in sigma(q) of fma(logit[v], inv_temperature, G(v)), ties to
 *         the lowest id, with G(v) = -ln(-ln(u(v))) a standard Gumbel variate;
 *   u(v) = (2*(r >> 9) + 1) * 2^-24 with r the 32-bit word v % 4 of
 *         Philox4x32-10(key = (seed low, seed high),
 *                       counter = (v / 4, batch row, draw low, draw high))
 *         (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
 *         SC'11);
 *   ln is evaluated in fp32 with explicitly rounded operations: x = m 2^e, m in
 *         (sqrt(1/2), sqrt(2)], s = (m-1)/(m+1), ln m = 2s(1 + s^2/3 + s^4/5 + s^6/7 +
 *         s^8/9) by Horner's rule with fused multiply-adds, ln x = fma(e, ln 2, ln m).
 * Logits are widened to fp32 exactly.  Rows, masking, EOS, stuck rows, finished rows,
 * the state update and every other argument are as in guided_mask_step.
 *
 *   inv_temperature  1 / temperature as fp32, > 0 and finite (FSM_ERR_RANGE otherwise).
 *   seed, draw       64-bit key and draw number: use a new `draw` for every step (the
 *                    step index), the same `seed` for a sequence of steps.
 */
int guided_sample_step(const void* logits_in, void* logits_out, int32_t logits_dtype,
                       int64_t row_stride, int32_t* states, uint8_t* finished,
                       int32_t* tokens_out, const uint32_t* allowed_mask,
                       const void* next_state, int32_t state_dtype, int32_t Q, int32_t N,
                       int32_t B, int32_t dead_state, int32_t eos_id, float inv_temperature,
                       uint64_t seed, uint64_t draw, int32_t* status_word, void* cuda_stream);

/*
 * The decode step on the compressed-row index of fsm_index_build_csr: guided_mask_step
 * (sample == 0) or guided_sample_step (sample != 0; inv_temperature, seed and draw as
 * there), except that the next state of the chosen token is found by binary search among
 * the row's tokens instead of in a dense table.  Same masking, selection and bookkeeping,
 * same results.  `capacity` is the number of entries csr_tokens and csr_next hold, as given
 * to fsm_index_build_csr: nothing beyond it is read.  A chosen token whose entry is missing
 * (index built with too small a capacity, FSM_FLAG_CSR_OVERFLOW) sends the row to the dead
 * state.
 */
int guided_step_csr(const void* logits_in, void* logits_out, int32_t logits_dtype,
                    int64_t row_stride, int32_t* states, uint8_t* finished, int32_t* tokens_out,
                    const uint32_t* allowed_mask, const int64_t* row_offsets,
                    const int32_t* csr_tokens, const int32_t* csr_next, int64_t capacity,
                    int32_t Q, int32_t N, int32_t B, int32_t dead_state, int32_t eos_id,
                    int32_t sample,
                    float inv_temperature, uint64_t seed, uint64_t draw, int32_t* status_word,
                    void* cuda_stream);

/*
 * Merging of identical index rows (paper Section 3: the index maps a state to its
 * set of allowed tokens; Section 5: it is built from automata that are not
 * reduced, so different states can carry the same row).
 *
 *   row_alias[q] = the smallest state whose row equals state q's, where "row" is
 *   the bitmask row and, when next_state is given, also the next-state row (only
 *   then can two states share one stored row of both arrays).  With next_state
 *   NULL two states alias exactly when they allow the same set of tokens.
 *
 *   allowed_mask  [Q*W] as built, 4-byte aligned
 *   next_state    [Q*N] of state_dtype as built, or NULL
 *   row_alias     out, int32 [Q]; row_alias[q] <= q, row_alias[row_alias[q]] == row_alias[q]
 *   n_unique      out, device int32: the number of distinct rows (states with row_alias[q] == q)
 *   workspace     device scratch, 256-byte aligned, at least
 *                 fsm_row_alias_workspace_bytes(Q) bytes (a few dozen bytes per state)
 *
 * Rows are grouped by a 64-bit hash and every merge is verified by comparing the
 * two rows entry by entry, so the result does not depend on the hash (with
 * FSM_DEBUG_WEAK_HASH set every row hashes alike and the result is the same).
 * Three launches on `cuda_stream`; reads each row once, and rows that have an
 * equal-hash partner a second time.
 */
size_t fsm_row_alias_workspace_bytes(int32_t Q);
int fsm_index_row_alias(const uint32_t* allowed_mask, const void* next_state, int32_t state_dtype,
                        int32_t Q, int32_t N, int32_t* row_alias, int32_t* n_unique,
                        void* workspace, size_t workspace_bytes, int32_t* status_word,
                        void* cuda_stream);

/*
 * Index files (paper Section 3.2: the index is computed once per (automaton,
 * vocabulary) pair and reused; the paper's example session switches such a
 * cache off to time the build).  A built index - the bitmask with either the
 * dense next-state table, no table, or the compressed rows - is written to one
 * flat little-endian file and read back into device arrays the caller owns.
 *
 * File layout: a 128-byte header
 *     bytes  0..7    "FSMGIDX1"
 *            8..11   uint32 version (1)
 *           12..15   int32  form          FSM_INDEX_DENSE | FSM_INDEX_BITMASK | FSM_INDEX_CSR
 *           16..19   int32  Q
 *           20..23   int32  N
 *           24..27   int32  state_dtype   FSM_STATE_* of the dense table (0 otherwise)
 *           28..31   int32  dead_state
 *           32..35   int32  eos_id
 *           36..39   (zero)
 *           40..47   int64  nnz           entries of the compressed rows (0 otherwise)
 *           48..55   uint64 payload_bytes
 *           56..63   uint64 payload_check (see fsm_checksum64)
 *           64..95   input_digest         32 bytes chosen by the caller, meant to be the
 *                                         SHA-256 of the build's inputs (fsm_index_input_digest)
 *           96..127  (zero)
 * followed by the payload, arrays back to back, each padded with zeros to a
 * multiple of 8 bytes: allowed_mask [Q*W] uint32; then for FSM_INDEX_DENSE
 * next_state [Q*N] of state_dtype; for FSM_INDEX_CSR row_offsets [Q+1] int64,
 * csr_tokens [nnz] int32, csr_next [nnz] int32.
 *
 * The three calls below are HOST-side: they block (they synchronise
 * `cuda_stream` and wait for their own copies), stage the arrays through two
 * pinned host buffers of 16 MiB that they allocate and free, and issue one
 * cudaMemcpyAsync per staged piece.  `path` is a HOST string.  The array
 * pointers in the descriptor are DEVICE pointers; arrays the form does not use
 * are ignored.
 */
#define FSM_INDEX_DENSE 0   /* bitmask + next-state table */
#define FSM_INDEX_BITMASK 1 /* bitmask only */
#define FSM_INDEX_CSR 2     /* bitmask + compressed rows */

typedef struct fsm_index_desc {
    int32_t form;
    int32_t Q, N;
    int32_t state_dtype; /* FSM_INDEX_DENSE: FSM_STATE_I32 or FSM_STATE_U16 */
    int32_t dead_state, eos_id;
    int64_t nnz;         /* FSM_INDEX_CSR: entries of csr_tokens / csr_next (= row_offsets[Q]) */
    uint8_t input_digest[32];
    uint32_t* allowed_mask; /* [Q*W] */
    void* next_state;       /* [Q*N] of state_dtype */
    int64_t* row_offsets;   /* [Q+1] */
    int32_t* csr_tokens;    /* [nnz] */
    int32_t* csr_next;      /* [nnz] */
} fsm_index_desc;

/* Size in bytes of the file fsm_index_save writes for `desc` (sizes and form
 * only; pointers are not looked at), or 0 when the descriptor is inconsistent. */
size_t fsm_index_serialized_bytes(const fsm_index_desc* desc);

/* Writes the index to `path` (replacing the file).  FSM_ERR_NULL / FSM_ERR_SHAPE /
 * FSM_ERR_DTYPE / FSM_ERR_RANGE for a bad descriptor, FSM_ERR_IO when the file cannot
 * be written, FSM_ERR_CUDA when a copy fails. */
int fsm_index_save(const char* path, const fsm_index_desc* desc, void* cuda_stream);

/* Reads the header of `path` into the scalar fields and input_digest of `*desc`
 * (pointers are left alone), so that a caller can size its arrays.  Touches no
 * device.  FSM_ERR_IO / FSM_ERR_FORMAT as above. */
int fsm_index_peek(const char* path, fsm_index_desc* desc);

/* Reads the index at `path` into the device arrays of `desc`.  Every scalar
 * field of `desc` and its input_digest must equal the file's (an all-zero
 * digest in `desc` accepts any): FSM_ERR_FORMAT otherwise, before any array is
 * touched.  A file shorter than its header says gives FSM_ERR_IO; a payload
 * that fails its checksum gives FSM_ERR_FORMAT after the arrays have been
 * written - their contents are then invalid. */
int fsm_index_load(const char* path, const fsm_index_desc* desc, void* cuda_stream);

/* SHA-256 (FIPS 180-4) of `nbytes` HOST bytes into out32 (HOST, 32 bytes). */
int fsm_sha256(const void* data, size_t nbytes, uint8_t* out32);

/* The payload checksum of the index files, over HOST bytes (nbytes a multiple
 * of 8): the wrap-around sum over 8-byte little-endian words w_i of
 * mix(w_i + (i+1) * 0x9E3779B97F4A7C15), mix being the splitmix64 finaliser.
 * Order-sensitive, cheap, not cryptographic: it catches truncation, bit rot
 * and swapped blocks, nothing adversarial. */
uint64_t fsm_checksum64(const void* data, size_t nbytes, uint64_t first_word_index);

/* SHA-256 of the inputs of an index build, for the header's input_digest: the
 * digest of the concatenation of the scalars (Q, N, dead_state, eos_id as int32,
 * vocab_nbytes as int64, little-endian) and the DEVICE arrays dfa_trans [Q*256]
 * int32, accept [Q] uint8, vocab_offsets [N+1] int32, vocab_bytes [vocab_nbytes].
 * Blocks (copies the arrays to the host); out32 is a HOST pointer. */
int fsm_index_input_digest(const int32_t* dfa_trans, const uint8_t* accept,
                           const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                           int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                           int32_t eos_id, uint8_t* out32, void* cuda_stream);

/*
 * Tuning and test hooks (no counterpart in the paper).  Sets a process-wide knob
 * and returns the previous value, or FSM_ERR_RANGE for an unknown key.  Not
 * thread-safe against concurrent library calls.
 */
#define FSM_DEBUG_WEAK_HASH 1       /* non-zero: hash every transition column alike, so that
                                       byte-class verification fails and the exact
                                       uncompressed path is exercised */
#define FSM_TUNE_MASK_CLUSTER 2     /* CTAs per logits row in guided_mask_step: 1,2,4,8; 0 = auto */
#define FSM_TUNE_WALK_CTAS 3        /* CTAs of the preparation and walk kernels; 0 = one per SM */
#define FSM_TUNE_SMEM_TABLE_BYTES 4 /* cap on the shared-memory table tile; 0 = device maximum */
#define FSM_PROFILE_WALK 5          /* non-zero: record a CUDA event pair around the walk
                                       kernel of every index build (see fsm_profile_read) */
#define FSM_TUNE_WALK_ALGO 6        /* 0 = automatic (a build of at least one row per SM: 2
                                       with a next-state table, 3 without; a smaller one: 1),
                                       1 = dense warp-tile walk, 2 = row-wise fill-and-patch
                                       walk, 3 = bucket walk (bitmask-only builds; builds with
                                       a next-state table take 2).  Same results in every
                                       case */
#define FSM_DEBUG_WAIT_PROBE 7      /* n > 0: once its table has arrived, a walk kernel waits
                                       (at most n polls) for a completion that nothing will
                                       ever signal, then takes its give-up path: it raises
                                       FSM_FLAG_WAIT_TIMEOUT and returns.  For tests of that
                                       path; the build's output is invalid while it is set */
int fsm_debug_set(int32_t key, int32_t value);

/*
 * Instrumentation (no counterpart in the paper).  While FSM_PROFILE_WALK is set,
 * each index build brackets its walk kernel (the launch that produces the
 * bitmask and the next-state table) with a pair of CUDA events on the build's
 * stream; nothing is skipped or reordered.  fsm_profile_read synchronises on
 * the recorded events, writes their elapsed times in milliseconds, oldest
 * first, to the HOST array ms_out (at most `capacity` values), forgets them and
 * returns how many it wrote (or FSM_ERR_CUDA).  At most 4096 launches are kept
 * between reads; later ones are not recorded.  Call it from the thread that
 * issued the builds, with their device current.
 */
int fsm_profile_read(float* ms_out, int32_t capacity);

#ifdef __cplusplus
}
#endif
#endif /* FSMGUIDE_H */
