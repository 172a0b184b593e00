// Vocabulary index construction (paper Section 3, Algorithms 3 and 4) for sm_100a.
//
// Four launches on the caller's stream, no host synchronisation:
//   1. hash_columns    one pass over delta: a 64-bit hash of each of the 256 byte columns
//   2. derive_classes  bytes with equal column hashes share a byte class
//   3. prepare_inputs  (a) class-compressed table [Q x Cs] with exact verification that
//                      every byte's column equals its class representative's column,
//                      (b) token bytes translated to class ids in 16-byte records
//   4. walk            every (state, token) pair: one warp owns 32 consecutive tokens
//                      (lane = token) and a run of 32 states; the table (or the tile of
//                      start states) is staged in shared memory by bulk async copy; a
//                      warp ballot gives the bitmask word, the end states go out as one
//                      coalesced store per state.
// If verification in 3(a) fails (a 64-bit hash collision) the walk reads the
// uncompressed table instead, so the result is exact in every case.
#include "fsm_common.cuh"

namespace fsm {
namespace {

constexpr int kHashBlocks = 128;
constexpr int kMaxCs = 264;            // 256 classes + the null class, rounded up to 8
constexpr int kWalkThreads = 1024;
constexpr int kWalkWarps = kWalkThreads / 32;
constexpr int kChunk = 32;             // states per warp task
constexpr int kInlineBytes = 16;       // token bytes kept in registers
constexpr uint32_t kBulkChunk = 32768; // bytes per bulk copy instruction
constexpr int kBatch = 4;              // 32-token chunks in flight per warp (sparse walk)

struct IndexMeta {
    int32_t C;        // number of byte classes (the null class has id C)
    int32_t Cs;       // row stride of the compressed table, entries
    int32_t any_bad;  // set when a byte's column differs from its representative's
    int32_t pad;
};

struct Workspace {
    IndexMeta* meta;
    uint8_t* cls;        // [256] byte -> class
    uint8_t* class_rep;  // [256] class -> representative byte
    uint64_t* partial;   // [kHashBlocks][256]
    void* table;         // [Q][kMaxCs] of TabT (row stride Cs once known)
    uint4* tok_cls;      // [G*32] first 16 class ids of each token
    uint8_t* tok_len;    // [G*32] min(length, 17)
    uint4* srec;         // [N] tokens sorted by first-byte class: {min(len,17), class of byte 1..15}
    int32_t* sid;        // [N] token id, same order as srec
    int32_t* gcount;     // [256] tokens per first-byte class
    int32_t* gcursor;    // [256] placement cursors of the counting sort
    int32_t* gstart;     // [257] first sorted position of each class
    size_t bytes;
};

size_t table_elem_bytes(int32_t Q) { return Q <= 65535 ? 2 : 4; }

Workspace carve(void* base, int32_t Q, int32_t N) {
    Workspace w;
    uint8_t* p = static_cast<uint8_t*>(base);
    size_t off = 0;
    auto take = [&](size_t n) {
        uint8_t* r = p ? p + off : nullptr;
        off += align_up(n, 256);
        return r;
    };
    const size_t G = (static_cast<size_t>(N) + 31) / 32;
    w.meta = reinterpret_cast<IndexMeta*>(take(sizeof(IndexMeta)));
    w.cls = take(256);
    w.class_rep = take(256);
    w.partial = reinterpret_cast<uint64_t*>(take(sizeof(uint64_t) * kHashBlocks * 256));
    w.table = take(static_cast<size_t>(Q) * kMaxCs * table_elem_bytes(Q));
    w.tok_cls = reinterpret_cast<uint4*>(take(G * 32 * sizeof(uint4)));
    w.tok_len = take(G * 32);
    w.srec = reinterpret_cast<uint4*>(take(static_cast<size_t>(N) * sizeof(uint4)));
    w.sid = reinterpret_cast<int32_t*>(take(static_cast<size_t>(N) * sizeof(int32_t)));
    w.gcount = reinterpret_cast<int32_t*>(take(256 * sizeof(int32_t)));
    w.gcursor = reinterpret_cast<int32_t*>(take(256 * sizeof(int32_t)));
    w.gstart = reinterpret_cast<int32_t*>(take(257 * sizeof(int32_t)));
    w.bytes = off;
    return w;
}

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

__device__ __forceinline__ uint32_t clamp_state(int32_t v, int32_t Q, int32_t dead) {
    return (static_cast<uint32_t>(v) >= static_cast<uint32_t>(Q)) ? dead : v;
}

// ---------------------------------------------------------------------------- 1
// Thread b owns byte column b; a block strides over rows.  The per-column hash is
// a wrap-around sum of mixed (row, value) pairs, so equal columns hash alike and
// partial sums from different blocks simply add.
__global__ void __launch_bounds__(256) hash_columns(const int32_t* __restrict__ trans, int32_t Q,
                                                   int32_t dead, uint64_t* __restrict__ partial,
                                                   int weak, int32_t* status) {
    const int b = threadIdx.x;
    uint64_t h = 0;
    bool bad = false;
    for (int q = blockIdx.x; q < Q; q += gridDim.x) {
        if (q == dead) continue;
        int32_t v = trans[static_cast<size_t>(q) * 256 + b];
        bad |= static_cast<uint32_t>(v) >= static_cast<uint32_t>(Q);
        h += mix64((static_cast<uint64_t>(q) << 32) | static_cast<uint32_t>(v));
    }
    partial[blockIdx.x * 256 + b] = weak ? 0 : h;
    if (__syncthreads_or(bad) && threadIdx.x == 0) raise_flag(status, FSM_FLAG_TRANS_RANGE);
}

// ---------------------------------------------------------------------------- 2
// One block.  Bytes whose column hashes are equal form a class, represented by the
// smallest such byte; class ids are the ranks of the representatives.  Equal hashes
// are found through a small open-addressing table in shared memory.
__global__ void __launch_bounds__(256) derive_classes(const uint64_t* __restrict__ partial,
                                                     int nblocks, IndexMeta* meta,
                                                     uint8_t* cls, uint8_t* class_rep,
                                                     int32_t* gcount, int32_t* gcursor) {
    constexpr int kSlots = 1024;
    gcount[threadIdx.x] = 0;
    gcursor[threadIdx.x] = 0;
    __shared__ unsigned long long keys[kSlots];
    __shared__ int min_byte[kSlots];
    __shared__ uint32_t rep_bits[8];
    constexpr unsigned long long kEmpty = ~0ull;
    const int b = threadIdx.x;
    uint64_t sum = 0;
#pragma unroll 8
    for (int k = 0; k < nblocks; ++k) sum += partial[k * 256 + b];
    // kEmpty marks a free slot; folding that one value onto its neighbour can only merge
    // two classes, which the exact verification of the next kernel would catch.
    const unsigned long long key = (sum == kEmpty) ? sum - 1 : sum;
    for (int i = b; i < kSlots; i += 256) {
        keys[i] = kEmpty;
        min_byte[i] = 256;
    }
    __syncthreads();
    // at most 256 distinct keys in 1024 slots: linear probing ends within kSlots steps
    int slot = static_cast<int>((key ^ (key >> 29)) & (kSlots - 1));
    for (int probe = 0; probe < kSlots; ++probe) {
        const unsigned long long was = atomicCAS(&keys[slot], kEmpty, key);
        if (was == kEmpty || was == key) break;
        slot = (slot + 1) & (kSlots - 1);
    }
    atomicMin(&min_byte[slot], b);
    __syncthreads();
    const int r = min_byte[slot];
    const bool is_rep = (r == b);
    const uint32_t m = __ballot_sync(kFullWarp, is_rep);
    if ((b & 31) == 0) rep_bits[b >> 5] = m;
    __syncthreads();
    int id = __popc(rep_bits[r >> 5] & ((1u << (r & 31)) - 1u));
    for (int w = 0; w < (r >> 5); ++w) id += __popc(rep_bits[w]);
    cls[b] = static_cast<uint8_t>(id);
    if (is_rep) class_rep[id] = static_cast<uint8_t>(b);
    if (b == 0) {
        int C = 0;
        for (int w = 0; w < 8; ++w) C += __popc(rep_bits[w]);
        meta->C = C;
        meta->Cs = (C + 1 + 7) & ~7;
        // 256 distinct columns leave no byte value for the null class: such a table
        // is walked uncompressed.
        meta->any_bad = (C > 255) ? 1 : 0;
        meta->pad = 0;
    }
}

// Bounds-checked view of one token for the token-side preparation kernels.
struct TokenInfo {
    int64_t start;
    int len;    // min(length, kInlineBytes + 1); 0 = not bucketed (empty, EOS, bad offsets)
    int first;  // class of the first byte
};

__device__ __forceinline__ TokenInfo token_info(const uint8_t* __restrict__ vocab_bytes,
                                                const int32_t* __restrict__ vocab_offsets,
                                                int64_t vocab_nbytes, int32_t N, int32_t eos_id,
                                                const uint8_t* s_cls, int64_t v, bool* bad) {
    TokenInfo t = {0, 0, 0};
    if (v < N && v != eos_id) {
        const int64_t o0 = vocab_offsets[v], o1 = vocab_offsets[v + 1];
        if (o0 < 0 || o1 < o0 || o1 > vocab_nbytes) {
            *bad = true;
        } else if (o1 > o0) {
            t.start = o0;
            t.len = static_cast<int>(min(o1 - o0, static_cast<int64_t>(kInlineBytes + 1)));
            t.first = s_cls[vocab_bytes[o0]];
        }
    }
    return t;
}

// ---------------------------------------------------------------------------- 3
// Blocks [0, row_blocks) compress and verify table rows; the remaining blocks
// translate tokens.  Column C of the compressed table (the null class) and the
// padding columns lead to the dead state, as does the whole row of the dead state.
template <typename TabT>
__global__ void __launch_bounds__(256)
prepare_inputs(const int32_t* __restrict__ trans, const uint8_t* __restrict__ vocab_bytes,
               const int32_t* __restrict__ vocab_offsets, int64_t vocab_nbytes, int32_t Q,
               int32_t N, int32_t dead, int32_t eos_id, int row_blocks, IndexMeta* meta,
               const uint8_t* __restrict__ cls, const uint8_t* __restrict__ class_rep,
               TabT* __restrict__ table, uint4* __restrict__ tok_cls,
               uint8_t* __restrict__ tok_len, int32_t* __restrict__ gcount, int32_t* status) {
    const int C = meta->C, Cs = meta->Cs;
    if (static_cast<int>(blockIdx.x) < row_blocks) {
        __shared__ int32_t row[256];
        __shared__ uint8_t s_cls[256], s_rep[256];
        s_cls[threadIdx.x] = cls[threadIdx.x];
        s_rep[threadIdx.x] = class_rep[threadIdx.x];
        bool bad = false;
        for (int q = blockIdx.x; q < Q; q += row_blocks) {
            __syncthreads();
            row[threadIdx.x] = clamp_state(trans[static_cast<size_t>(q) * 256 + threadIdx.x], Q, dead);
            __syncthreads();
            if (q != dead) bad |= row[threadIdx.x] != row[s_rep[s_cls[threadIdx.x]]];
            for (int c = threadIdx.x; c < Cs; c += 256) {
                int32_t v = (q == dead || c >= C) ? dead : row[s_rep[c]];
                table[static_cast<size_t>(q) * Cs + c] = static_cast<TabT>(v);
            }
        }
        if (__syncthreads_or(bad) && threadIdx.x == 0) {
            atomicExch(&meta->any_bad, 1);
            raise_flag(status, FSM_FLAG_CLASS_SPLIT);
        }
    } else if (gcount != nullptr) {
        // sparse walk: count the tokens of each first-byte class (placement: sort_tokens)
        __shared__ int hist[256];
        __shared__ uint8_t s_cls[256];
        hist[threadIdx.x] = 0;
        s_cls[threadIdx.x] = cls[threadIdx.x];
        __syncthreads();
        bool bad = false;
        const int64_t v = static_cast<int64_t>(blockIdx.x - row_blocks) * 256 + threadIdx.x;
        const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
        if (t.len > 0) atomicAdd(&hist[t.first], 1);
        if (__syncthreads_or(bad) && threadIdx.x == 0) raise_flag(status, FSM_FLAG_OFFSETS);
        if (hist[threadIdx.x] > 0) atomicAdd(&gcount[threadIdx.x], hist[threadIdx.x]);
    } else {
        // dense walk: 16-byte class records in token order
        const int64_t slots = (static_cast<int64_t>(N) + 31) / 32 * 32;
        const int64_t v = static_cast<int64_t>(blockIdx.x - row_blocks) * 256 + threadIdx.x;
        if (v >= slots) return;
        uint32_t w[4] = {static_cast<uint32_t>(C), 0, 0, 0};  // an empty token reads the null class
        int len = 0;
        if (v < N && v != eos_id) {
            const int64_t o0 = vocab_offsets[v], o1 = vocab_offsets[v + 1];
            if (o0 < 0 || o1 < o0 || o1 > vocab_nbytes) {
                raise_flag(status, FSM_FLAG_OFFSETS);
            } else {
                len = static_cast<int>(min(o1 - o0, static_cast<int64_t>(kInlineBytes + 1)));
                const int n = min(len, kInlineBytes);
                if (n > 0) w[0] = 0;
                for (int i = 0; i < n; ++i)
                    w[i >> 2] |= static_cast<uint32_t>(cls[vocab_bytes[o0 + i]]) << ((i & 3) * 8);
            }
        }
        tok_cls[v] = make_uint4(w[0], w[1], w[2], w[3]);
        tok_len[v] = static_cast<uint8_t>(len);
    }
}

// ---------------------------------------------------------------------------- 4
struct WalkParams {
    const void* table;
    const uint4* tok_cls;
    const uint8_t* tok_len;
    const IndexMeta* meta;
    const int32_t* trans;
    const uint8_t* accept;
    const uint8_t* vocab_bytes;
    const int32_t* vocab_offsets;
    int64_t vocab_nbytes;
    int32_t Q, N, G, dead, eos_id, q_begin, q_end;
    uint32_t smem_cap;  // bytes of dynamic shared memory available for the table tile
    const uint4* srec;
    const int32_t* sid;
    const int32_t* gstart;
    uint32_t* mask;
    void* next;
    int32_t* status;
};

__device__ __forceinline__ uint32_t tok_byte(const uint4& t, int i) {
    const uint32_t w = (i >> 2) == 0 ? t.x : (i >> 2) == 1 ? t.y : (i >> 2) == 2 ? t.z : t.w;
    return (w >> ((i & 3) * 8)) & 0xFFu;
}

// Walks bytes [from, len) of token v through the uncompressed table.
__device__ __noinline__ uint32_t raw_walk_impl(const int32_t* __restrict__ trans,
                                               const uint8_t* __restrict__ vocab_bytes, int32_t Q,
                                               int32_t dead, uint32_t s, int64_t o0, int64_t o1,
                                               int from) {
    for (int64_t i = o0 + from; i < o1 && s != static_cast<uint32_t>(dead); ++i)
        s = clamp_state(trans[static_cast<size_t>(s) * 256 + vocab_bytes[i]], Q, dead);
    return s;
}

__device__ __forceinline__ uint32_t raw_walk(const WalkParams& p, uint32_t s, int64_t o0,
                                             int64_t o1, int from) {
    return raw_walk_impl(p.trans, p.vocab_bytes, p.Q, p.dead, s, o0, o1, from);
}

template <typename OutT, bool HAS_OUT>
__device__ __forceinline__ void emit(const WalkParams& p, int q, int g, int v, int lane, uint32_t s) {
    const size_t r = static_cast<size_t>(q - p.q_begin);
    if (HAS_OUT && v < p.N) static_cast<OutT*>(p.next)[r * p.N + v] = static_cast<OutT>(s);
    const uint32_t word = __ballot_sync(kFullWarp, s != static_cast<uint32_t>(p.dead));
    if (lane == 0) p.mask[r * p.G + g] = word;
}

// Bytes 1.. of one token walked from state s, all 32 lanes in lock step.  `go` says
// whether this lane still has a live walk with bytes left.  The loop is warp-uniform
// (one vote per byte) and its body has no branches: lanes that are done keep their
// state through a select.  Every state value is a valid table row (out-of-range
// entries were replaced by `dead` when the table was compressed), so the shared-memory
// lookup needs no guard; the global-memory lookup is predicated to save traffic.
template <typename TabT, bool FULL>
__device__ __forceinline__ uint32_t walk_rest(const TabT* __restrict__ tab, uint32_t Cs,
                                              uint32_t dead, const uint4& tk, int len, uint32_t s,
                                              bool& go) {
#pragma unroll
    for (int i = 1; i < kInlineBytes; ++i) {
        if (!__any_sync(kFullWarp, go)) break;
        const uint32_t c = tok_byte(tk, i);
        uint32_t ns;
        if (FULL) {
            ns = tab[s * Cs + c];
        } else {
            ns = s;
            if (go) ns = __ldg(tab + static_cast<size_t>(s) * Cs + c);
        }
        s = go ? ns : s;
        go = go && (ns != dead) && (i + 1 < len);
    }
    return s;
}

// One warp task: tokens 32g .. 32g+31 (lane = token) from states q0 .. q0+nq-1.
// `first` points at row q0 of the shared-memory tile; `tab` is the table used for
// the second and later bytes (the same tile when FULL, else global memory).
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL, bool HAS_EOS>
__device__ __forceinline__ void walk_task(const WalkParams& p, const TabT* __restrict__ first,
                                          const TabT* __restrict__ tab, int Cs, int q0, int nq,
                                          int g, int lane) {
    const int v = g * 32 + lane;
    const uint4 tk = p.tok_cls[v];
    const int len = p.tok_len[v];
    const uint32_t dead = p.dead;
    const bool multi = len > 1;
    const bool eos_lane = HAS_EOS && (v == p.eos_id);
    const bool store_ok = HAS_OUT && (v < p.N);
    const TabT* f = first + (tk.x & 0xFFu);
    const size_t r0 = static_cast<size_t>(q0 - p.q_begin);
    OutT* outp = HAS_OUT ? static_cast<OutT*>(p.next) + r0 * p.N + v : nullptr;
    uint32_t* mp = p.mask + r0 * p.G + g;
    for (int j = 0; j < nq; ++j) {
        uint32_t s = *f;
        bool go = multi && (s != dead);
        s = walk_rest<TabT, FULL>(tab, Cs, dead, tk, len, s, go);
        if (go)  // longer than the inline record and still alive: finish on the raw bytes
            s = raw_walk(p, s, p.vocab_offsets[v], p.vocab_offsets[v + 1], kInlineBytes);
        if (HAS_EOS) {
            const int q = q0 + j;
            if (eos_lane) s = (q != p.dead && p.accept[q]) ? q : dead;
        }
        if (store_ok) *outp = static_cast<OutT>(s);
        const uint32_t word = __ballot_sync(kFullWarp, s != dead);
        if (lane == 0) *mp = word;
        f += Cs;
        if (HAS_OUT) outp += p.N;
        mp += p.G;
    }
}

// Same task on the uncompressed table (exact fallback after a class split).
template <typename OutT, bool HAS_OUT>
__device__ __forceinline__ void walk_task_raw(const WalkParams& p, int q0, int nq, int g, int lane) {
    const int v = g * 32 + lane;
    int64_t o0 = 0, o1 = 0;
    if (v < p.N && v != p.eos_id) {
        o0 = p.vocab_offsets[v];
        o1 = p.vocab_offsets[v + 1];
        if (o0 < 0 || o1 < o0 || o1 > p.vocab_nbytes) o0 = o1 = 0;
    }
    for (int j = 0; j < nq; ++j) {
        const int q = q0 + j;
        uint32_t s = p.dead;
        if (o1 > o0 && q != p.dead) s = raw_walk(p, q, o0, o1, 0);
        if (v == p.eos_id) s = (q != p.dead && p.accept[q]) ? q : p.dead;
        emit<OutT, HAS_OUT>(p, q, g, v, lane, s);
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    TabT* tile = reinterpret_cast<TabT*>(smem_raw);
    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int Cs = p.meta->Cs;
    const bool raw = p.meta->any_bad != 0;
    const uint32_t row_bytes = Cs * sizeof(TabT);
    const int nrows = p.q_end - p.q_begin;
    const bool full = static_cast<uint64_t>(p.Q) * row_bytes <= p.smem_cap;
    const int cap_rows = max(kChunk, static_cast<int>(p.smem_cap / row_bytes) / kChunk * kChunk);
    const int ntiles = full ? 1 : (nrows + cap_rows - 1) / cap_rows;
    const int lane = threadIdx.x & 31;
    const int64_t wg = static_cast<int64_t>(blockIdx.x) * kWalkWarps + (threadIdx.x >> 5);
    const int64_t TW = static_cast<int64_t>(gridDim.x) * kWalkWarps;

    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    uint32_t parity = 0;
    for (int ti = 0; ti < ntiles; ++ti) {
        const int t_q0 = full ? 0 : p.q_begin + ti * cap_rows;          // first staged row
        const int t_rows = full ? p.Q : min(cap_rows, p.q_end - t_q0);  // staged rows
        const int w_q0 = full ? p.q_begin : t_q0;                       // first start state
        const int w_rows = full ? nrows : t_rows;
        if (!raw) {
            if (ti > 0) __syncthreads();  // every warp is done with the previous tile
            if (threadIdx.x == 0) {
                const uint32_t bytes = static_cast<uint32_t>(t_rows) * row_bytes;
                const uint8_t* src =
                    reinterpret_cast<const uint8_t*>(gtab) + static_cast<size_t>(t_q0) * row_bytes;
                mbar_expect_tx(&bar, bytes);
                for (uint32_t o = 0; o < bytes; o += kBulkChunk)
                    bulk_copy_g2s(smem_raw + o, src + o, min(kBulkChunk, bytes - o), &bar);
            }
            bool ok = mbar_wait_bounded(&bar, parity);
            if (!ok) ok = mbar_wait_bounded(&bar, parity);  // drain before giving up
            parity ^= 1;
            if (!__syncthreads_and(ok)) {
                if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
                return;
            }
        }
        const int nchunks = (w_rows + kChunk - 1) / kChunk;
        const int64_t ntasks = static_cast<int64_t>(nchunks) * p.G;
        for (int64_t t = wg; t < ntasks; t += TW) {
            const int chunk = static_cast<int>(t / p.G);
            const int g = static_cast<int>(t - static_cast<int64_t>(chunk) * p.G);
            const int q0 = w_q0 + chunk * kChunk;
            const int nq = min(kChunk, w_q0 + w_rows - q0);
            if (raw) {
                walk_task_raw<OutT, HAS_OUT>(p, q0, nq, g, lane);
            } else {
                const TabT* first = tile + static_cast<size_t>(q0 - t_q0) * Cs;
                const bool has_eos = (p.eos_id >= 0) && ((p.eos_id >> 5) == g);
                if (has_eos) {  // rare: one group in the whole vocabulary
                    if (full)
                        walk_task<TabT, OutT, HAS_OUT, true, true>(p, first, tile, Cs, q0, nq, g, lane);
                    else
                        walk_task<TabT, OutT, HAS_OUT, false, true>(p, first, gtab, Cs, q0, nq, g, lane);
                } else if (full) {
                    walk_task<TabT, OutT, HAS_OUT, true, false>(p, first, tile, Cs, q0, nq, g, lane);
                } else {
                    walk_task<TabT, OutT, HAS_OUT, false, false>(p, first, gtab, Cs, q0, nq, g, lane);
                }
            }
        }
    }
}


// ---------------------------------------------------------------------------- 3b
// Token order for the work-avoiding walk: all non-empty tokens sorted by the class of
// their first byte (a counting sort over at most 256 classes).  The per-class counts
// come from prepare_inputs' token blocks; this kernel places the records.  A record
// keeps the length and the classes of bytes 1..15 - the first byte's class is the
// bucket - and `sid` the token id, in the same order.
__global__ void __launch_bounds__(256)
sort_tokens(const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
            int64_t vocab_nbytes, int32_t N, int32_t eos_id, const uint8_t* __restrict__ cls,
            const int32_t* __restrict__ gcount, int32_t* __restrict__ gcursor,
            int32_t* __restrict__ gstart, uint4* __restrict__ srec, int32_t* __restrict__ sid) {
    __shared__ int lhist[256];
    __shared__ int lbase[256];
    __shared__ int gst[257];
    __shared__ uint8_t s_cls[256];
    s_cls[threadIdx.x] = cls[threadIdx.x];
    lhist[threadIdx.x] = 0;
    if (threadIdx.x < 32) {  // exclusive prefix over the 256 class counts, 8 per lane
        int local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            local[i] = sum;
            sum += gcount[threadIdx.x * 8 + i];
        }
        int incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullWarp, incl, off);
            if (static_cast<int>(threadIdx.x) >= off) incl += o;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) gst[threadIdx.x * 8 + i] = incl - sum + local[i];
        if (threadIdx.x == 31) gst[256] = incl;
    }
    __syncthreads();
    if (blockIdx.x == 0) {
        gstart[threadIdx.x] = gst[threadIdx.x];
        if (threadIdx.x == 0) gstart[256] = gst[256];
    }
    bool bad = false;
    const int64_t v = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
    const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
    int rank = 0;
    if (t.len > 0) rank = atomicAdd(&lhist[t.first], 1);
    __syncthreads();
    if (lhist[threadIdx.x] > 0) lbase[threadIdx.x] = atomicAdd(&gcursor[threadIdx.x], lhist[threadIdx.x]);
    __syncthreads();
    if (t.len > 0) {
        uint32_t w[4] = {static_cast<uint32_t>(t.len), 0, 0, 0};
        const int nb = min(t.len, kInlineBytes);
        for (int i = 1; i < nb; ++i)
            w[i >> 2] |= static_cast<uint32_t>(s_cls[vocab_bytes[t.start + i]]) << ((i & 3) * 8);
        const int pos = gst[t.first] + lbase[t.first] + rank;
        srec[pos] = make_uint4(w[0], w[1], w[2], w[3]);
        sid[pos] = static_cast<int32_t>(v);
    }
}

// ---------------------------------------------------------------------------- 4b
// Work-avoiding walk.  One persistent CTA per SM; the compressed table is staged in
// shared memory once (bulk async copy) when it fits.  A CTA's unit of work is one index
// row (one state q):
//   fill     the row of the next-state table is set to `dead` and the bitmask row to 0
//            with streaming 16-byte stores - this settles every token whose first byte
//            q cannot read, with no table lookup at all;
//   buckets  one lookup per byte class tells which first-byte buckets are readable;
//   walk     only the tokens of those buckets are walked (lane = token, 32-token chunks,
//            several chunks in flight per warp); survivors store their end state into
//            the row and OR their bit into the bitmask row.  The row was written
//            microseconds earlier by the same CTA, so these stores merge in L2 and each
//            line still reaches HBM once.
// Every (state, token) pair gets its entry; results are identical to the dense walk.
struct LiveBucket {
    uint32_t s1;  // state after the first byte
    int32_t start;
    int32_t count;
};

constexpr int kMaxLive = 256;

template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void sparse_row(const WalkParams& p, const TabT* __restrict__ tab,
                                           int C, int Cs, bool raw, LiveBucket* live,
                                           int32_t* cpre, int* counts, const int32_t* s_gstart,
                                           int r) {
    const uint32_t dead = p.dead;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = p.q_begin + r;
    OutT* nrow = HAS_OUT ? static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N : nullptr;
    uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G;
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (FULL) return tab[s * static_cast<uint32_t>(Cs) + c];
        return __ldg(tab + static_cast<size_t>(s) * Cs + c);
    };

    // ---- fill (head and tail element-wise, the aligned middle as 16-byte vectors)
    if (HAS_OUT) {
        constexpr int kVecElems = 16 / sizeof(OutT);
        const uintptr_t addr = reinterpret_cast<uintptr_t>(nrow);
        int head = static_cast<int>(((16 - (addr & 15)) & 15) / sizeof(OutT));
        if (head > p.N) head = p.N;
        const int nvec = (p.N - head) / kVecElems;
        const uint32_t d = sizeof(OutT) == 2 ? (dead | (dead << 16)) : dead;
        const uint4 dead16 = make_uint4(d, d, d, d);
        uint4* mid = reinterpret_cast<uint4*>(nrow + head);
        for (int i = threadIdx.x; i < nvec; i += kWalkThreads) mid[i] = dead16;
        for (int i = threadIdx.x; i < head; i += kWalkThreads) nrow[i] = static_cast<OutT>(dead);
        for (int i = head + nvec * kVecElems + threadIdx.x; i < p.N; i += kWalkThreads)
            nrow[i] = static_cast<OutT>(dead);
    }
    for (int i = threadIdx.x; i < p.G; i += kWalkThreads) mrow[i] = 0;

    // ---- readable buckets of this state
    if (warp == 0 && !raw) {
        int cnt = 0, chunks = 0;
        for (int c0 = 0; c0 < C; c0 += 32) {
            const int c = c0 + lane;
            uint32_t s1 = dead;
            int start = 0, num = 0;
            if (c < C) {
                s1 = lookup(q, c);
                start = s_gstart[c];
                num = s_gstart[c + 1] - start;
            }
            const bool is_live = (s1 != dead) && (num > 0);
            const uint32_t m = __ballot_sync(kFullWarp, is_live);
            const int nch = is_live ? (num + 31) >> 5 : 0;
            int incl = nch;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(kFullWarp, incl, off);
                if (lane >= off) incl += o;
            }
            if (is_live) {
                const int pos = cnt + __popc(m & ((1u << lane) - 1u));
                LiveBucket b;
                b.s1 = s1;
                b.start = start;
                b.count = num;
                live[pos] = b;
                cpre[pos] = chunks + incl - nch;
            }
            cnt += __popc(m);
            chunks += __shfl_sync(kFullWarp, incl, 31);
        }
        if (lane == 0) {
            counts[0] = cnt;
            counts[1] = chunks;
            cpre[cnt] = chunks;
        }
    }
    __syncthreads();  // also orders the fill before the scattered stores below

    if (!raw) {
        const int M = counts[1];
        int b = 0;
        for (int g0 = warp; g0 < M; g0 += kWalkWarps * kBatch) {
            // issue the loads of kBatch chunks, then walk them one after the other
            uint4 rec[kBatch];
            int32_t id[kBatch];  // -1 = lane has no token in this chunk
            uint32_t s1[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int g = g0 + k * kWalkWarps;
                rec[k] = make_uint4(0, 0, 0, 0);
                id[k] = -1;
                s1[k] = dead;
                if (g < M) {
                    while (g >= cpre[b + 1]) ++b;
                    const LiveBucket lb = live[b];
                    const int i = (g - cpre[b]) * 32 + lane;
                    s1[k] = lb.s1;
                    if (i < lb.count) {
                        rec[k] = __ldg(p.srec + lb.start + i);
                        id[k] = __ldg(p.sid + lb.start + i);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int len = rec[k].x & 0xFFu;
                bool go = len > 1;
                uint32_t st = walk_rest<TabT, FULL>(tab, Cs, dead, rec[k], len, s1[k], go);
                if (go)  // longer than the inline record: finish on the raw bytes
                    st = raw_walk(p, st, p.vocab_offsets[id[k]], p.vocab_offsets[id[k] + 1],
                                  kInlineBytes);
                if (id[k] >= 0 && st != dead) {
                    if (HAS_OUT) nrow[id[k]] = static_cast<OutT>(st);
                    atomicOr(&mrow[id[k] >> 5], 1u << (id[k] & 31));
                }
            }
        }
    } else if (q != p.dead) {
        for (int v = threadIdx.x; v < p.N; v += kWalkThreads) {
            if (v == p.eos_id) continue;
            const int64_t o0 = p.vocab_offsets[v], o1 = p.vocab_offsets[v + 1];
            if (o0 < 0 || o1 <= o0 || o1 > p.vocab_nbytes) continue;
            const uint32_t s = raw_walk(p, q, o0, o1, 0);
            if (s != dead) {
                if (HAS_OUT) nrow[v] = static_cast<OutT>(s);
                atomicOr(&mrow[v >> 5], 1u << (v & 31));
            }
        }
    }
    if (threadIdx.x == 0 && p.eos_id >= 0 && q != p.dead && p.accept[q]) {
        if (HAS_OUT) nrow[p.eos_id] = static_cast<OutT>(q);
        atomicOr(&mrow[p.eos_id >> 5], 1u << (p.eos_id & 31));
    }
    __syncthreads();  // the bucket list is rebuilt by the next row
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk_sparse(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ LiveBucket live[kMaxLive];
    __shared__ int32_t cpre[kMaxLive + 4];
    __shared__ int32_t s_gstart[260];
    __shared__ int counts[2];
    TabT* stab = reinterpret_cast<TabT*>(smem_raw);

    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int C = p.meta->C, Cs = p.meta->Cs;
    const bool raw = p.meta->any_bad != 0;
    const uint64_t table_bytes = static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT);
    const bool full = !raw && table_bytes <= p.smem_cap;

    for (int i = threadIdx.x; i < 257; i += kWalkThreads) s_gstart[i] = p.gstart[i];
    if (full) {
        if (threadIdx.x == 0) {
            mbar_init(&bar, 1);
            fence_mbar_init();
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            const uint32_t bytes = static_cast<uint32_t>(table_bytes);
            mbar_expect_tx(&bar, bytes);
            for (uint32_t o = 0; o < bytes; o += kBulkChunk)
                bulk_copy_g2s(smem_raw + o, reinterpret_cast<const uint8_t*>(gtab) + o,
                              min(kBulkChunk, bytes - o), &bar);
        }
        bool ok = mbar_wait_bounded(&bar, 0);
        if (!ok) ok = mbar_wait_bounded(&bar, 0);  // drain before giving up
        if (!__syncthreads_and(ok)) {
            if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
            return;
        }
    } else {
        __syncthreads();
    }

    const int nrows = p.q_end - p.q_begin;
    for (int r = blockIdx.x; r < nrows; r += gridDim.x) {
        if (full)
            sparse_row<TabT, OutT, HAS_OUT, true>(p, stab, C, Cs, raw, live, cpre, counts, s_gstart, r);
        else
            sparse_row<TabT, OutT, HAS_OUT, false>(p, gtab, C, Cs, raw, live, cpre, counts, s_gstart, r);
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_sparse(const WalkParams& p, int grid, cudaStream_t stream) {
    auto kernel = walk_sparse<TabT, OutT, HAS_OUT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    kernel<<<grid, kWalkThreads, p.smem_cap, stream>>>(p);
    return cudaGetLastError();
}

template <typename TabT>
cudaError_t launch_sparse_for(const WalkParams& p, int grid, int32_t state_dtype, bool has_out,
                              cudaStream_t stream) {
    if (!has_out) return launch_sparse<TabT, int32_t, false>(p, grid, stream);
    if (state_dtype == FSM_STATE_U16) return launch_sparse<TabT, uint16_t, true>(p, grid, stream);
    return launch_sparse<TabT, int32_t, true>(p, grid, stream);
}

template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_walk(const WalkParams& p, int grid, cudaStream_t stream) {
    auto kernel = walk<TabT, OutT, HAS_OUT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    kernel<<<grid, kWalkThreads, p.smem_cap, stream>>>(p);
    return cudaGetLastError();
}

template <typename TabT>
cudaError_t launch_walk_for(const WalkParams& p, int grid, int32_t state_dtype, bool has_out,
                            cudaStream_t stream) {
    if (!has_out) return launch_walk<TabT, int32_t, false>(p, grid, stream);
    if (state_dtype == FSM_STATE_U16) return launch_walk<TabT, uint16_t, true>(p, grid, stream);
    return launch_walk<TabT, int32_t, true>(p, grid, stream);
}

}  // namespace
}  // namespace fsm

extern "C" size_t fsm_index_workspace_bytes(int32_t Q, int32_t N, int64_t vocab_nbytes) {
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0) return 0;
    return fsm::carve(nullptr, Q, N).bytes;
}

extern "C" int fsm_index_build_rows(const int32_t* dfa_trans, const uint8_t* accept,
                                    const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                    int64_t vocab_nbytes, int32_t Q, int32_t N,
                                    int32_t dead_state, int32_t eos_id, int32_t q_begin,
                                    int32_t q_end, uint32_t* allowed_mask, void* next_state,
                                    int32_t state_dtype, void* workspace, size_t workspace_bytes,
                                    int32_t* status_word, void* cuda_stream) {
    using namespace fsm;
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0 || N > 0x7FFFFFE0) return FSM_ERR_SHAPE;
    if (!dfa_trans || !accept || !vocab_offsets || !allowed_mask) return FSM_ERR_NULL;
    if (!vocab_bytes && vocab_nbytes > 0) return FSM_ERR_NULL;
    if (state_dtype != FSM_STATE_I32 && state_dtype != FSM_STATE_U16) return FSM_ERR_DTYPE;
    if (state_dtype == FSM_STATE_U16 && Q > 65535) return FSM_ERR_DTYPE;
    if (dead_state < 0 || dead_state >= Q) return FSM_ERR_RANGE;
    if (eos_id < -1 || eos_id >= N) return FSM_ERR_RANGE;
    if (q_begin < 0 || q_end > Q || q_begin > q_end) return FSM_ERR_RANGE;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(dfa_trans, 4) || misaligned(vocab_offsets, 4) || misaligned(allowed_mask, 4) ||
        misaligned(status_word, 4))
        return FSM_ERR_ALIGN;
    if (next_state && misaligned(next_state, state_dtype == FSM_STATE_U16 ? 2 : 4))
        return FSM_ERR_ALIGN;
    const size_t need = fsm_index_workspace_bytes(Q, N, vocab_nbytes);
    if (!workspace || workspace_bytes < need) return FSM_ERR_WORKSPACE;
    if (misaligned(workspace, 256)) return FSM_ERR_ALIGN;
    if (q_begin == q_end) return FSM_OK;

    const DeviceInfo& dev = device_info();
    if (!dev.ok) return FSM_ERR_CUDA;
    if (dev.cc_major != 10) return FSM_ERR_DEVICE;
    const Tunables& tune = tunables();
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    Workspace ws = carve(workspace, Q, N);
    const bool wide = Q > 65535;

    const int hash_blocks = Q < kHashBlocks ? Q : kHashBlocks;
    hash_columns<<<hash_blocks, 256, 0, stream>>>(dfa_trans, Q, dead_state, ws.partial,
                                                  tune.weak_hash, status_word);
    derive_classes<<<1, 256, 0, stream>>>(ws.partial, hash_blocks, ws.meta, ws.cls, ws.class_rep,
                                          ws.gcount, ws.gcursor);
    const int G = (N + 31) / 32;
    const int row_blocks = Q < 2 * dev.sm_count ? Q : 2 * dev.sm_count;
    const bool bucketed = tune.walk_algo != 1;
    const int tok_blocks = (G * 32 + 255) / 256;  // dense: token records; sparse: class counts
    int32_t* count_into = bucketed ? ws.gcount : nullptr;
    if (wide)
        prepare_inputs<int32_t><<<row_blocks + tok_blocks, 256, 0, stream>>>(
            dfa_trans, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state, eos_id,
            row_blocks, ws.meta, ws.cls, ws.class_rep, static_cast<int32_t*>(ws.table),
            ws.tok_cls, ws.tok_len, count_into, status_word);
    else
        prepare_inputs<uint16_t><<<row_blocks + tok_blocks, 256, 0, stream>>>(
            dfa_trans, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state, eos_id,
            row_blocks, ws.meta, ws.cls, ws.class_rep, static_cast<uint16_t*>(ws.table),
            ws.tok_cls, ws.tok_len, count_into, status_word);
    if (bucketed)
        sort_tokens<<<(N + 255) / 256, 256, 0, stream>>>(vocab_bytes, vocab_offsets, vocab_nbytes, N,
                                                         eos_id, ws.cls, ws.gcount, ws.gcursor,
                                                         ws.gstart, ws.srec, ws.sid);
    if (cudaGetLastError() != cudaSuccess) return FSM_ERR_CUDA;

    WalkParams p;
    p.table = ws.table;
    p.tok_cls = ws.tok_cls;
    p.tok_len = ws.tok_len;
    p.meta = ws.meta;
    p.trans = dfa_trans;
    p.accept = accept;
    p.vocab_bytes = vocab_bytes;
    p.vocab_offsets = vocab_offsets;
    p.vocab_nbytes = vocab_nbytes;
    p.Q = Q;
    p.N = N;
    p.G = G;
    p.dead = dead_state;
    p.eos_id = eos_id;
    p.q_begin = q_begin;
    p.q_end = q_end;
    p.mask = allowed_mask;
    p.next = next_state;
    p.status = status_word;
    p.srec = ws.srec;
    p.sid = ws.sid;
    p.gstart = ws.gstart;
    int cap = dev.smem_optin - 1024;  // static shared memory and alignment slack
    if (tune.smem_table_cap > 0 && tune.smem_table_cap < cap) cap = tune.smem_table_cap;
    if (bucketed) {
        cap -= 8 * 1024;  // static shared memory of walk_sparse (bucket list)
        if (cap < 1024) cap = 1024;
        p.smem_cap = static_cast<uint32_t>(cap) / 128 * 128;
        int64_t grid = dev.sm_count;
        if (tune.walk_ctas > 0) grid = tune.walk_ctas;
        if (grid > q_end - q_begin) grid = q_end - q_begin;
        const int prof = profile_begin(stream);
        cudaError_t e = wide ? launch_sparse_for<int32_t>(p, static_cast<int>(grid), state_dtype,
                                                           next_state != nullptr, stream)
                             : launch_sparse_for<uint16_t>(p, static_cast<int>(grid), state_dtype,
                                                            next_state != nullptr, stream);
        profile_end(prof, stream);
        return e == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
    }
    const int min_cap = kChunk * kMaxCs * 4;
    if (cap < min_cap) cap = min_cap;
    p.smem_cap = static_cast<uint32_t>(cap) / 128 * 128;

    const int64_t tasks = static_cast<int64_t>((q_end - q_begin + kChunk - 1) / kChunk) * G;
    int64_t grid = (tasks + kWalkWarps - 1) / kWalkWarps;
    if (grid > dev.sm_count) grid = dev.sm_count;
    if (tune.walk_ctas > 0) grid = tune.walk_ctas;
    const int prof = profile_begin(stream);
    cudaError_t e = wide ? launch_walk_for<int32_t>(p, static_cast<int>(grid), state_dtype,
                                                   next_state != nullptr, stream)
                         : launch_walk_for<uint16_t>(p, static_cast<int>(grid), state_dtype,
                                                    next_state != nullptr, stream);
    profile_end(prof, stream);
    return e == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
}

extern "C" int fsm_index_build(const int32_t* dfa_trans, const uint8_t* accept,
                               const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                               int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                               int32_t eos_id, uint32_t* allowed_mask, void* next_state,
                               int32_t state_dtype, void* workspace, size_t workspace_bytes,
                               int32_t* status_word, void* cuda_stream) {
    return fsm_index_build_rows(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                                dead_state, eos_id, 0, Q, allowed_mask, next_state, state_dtype,
                                workspace, workspace_bytes, status_word, cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant: the scratch of the four kernels above lives in this array inside the
// library's device image instead of in a caller-provided workspace.  In host code the name
// `g_static_scratch` is only a handle for the runtime, not a device address: the address the
// kernels need comes from cudaGetSymbolAddress, looked up once per device.
namespace fsm {
namespace {
static __device__ __align__(256) unsigned char g_static_scratch[FSM_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, or nullptr on failure.
void* static_scratch_address() {
    constexpr int kMaxDevices = 64;
    static void* cached[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (cached[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        cached[dev] = ptr;
    }
    return cached[dev];
}
}  // namespace
}  // namespace fsm

extern "C" int fsm_index_build_static(const int32_t* dfa_trans, const uint8_t* accept,
                                      const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                      int64_t vocab_nbytes, int32_t Q, int32_t N,
                                      int32_t dead_state, int32_t eos_id, uint32_t* allowed_mask,
                                      void* next_state, int32_t state_dtype, int32_t* status_word,
                                      void* cuda_stream) {
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0) return FSM_ERR_SHAPE;
    const size_t need = fsm_index_workspace_bytes(Q, N, vocab_nbytes);
    if (need == 0 || need > FSM_STATIC_SCRATCH_BYTES) return FSM_ERR_WORKSPACE;
    if (!fsm::device_info().ok) return FSM_ERR_CUDA;
    void* scratch = fsm::static_scratch_address();
    if (scratch == nullptr) return FSM_ERR_CUDA;
    // Every part of the scratch that the build reads is written earlier in the same build,
    // so the previous call's leftovers need no clearing.
    return fsm_index_build_rows(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                                dead_state, eos_id, 0, Q, allowed_mask, next_state, state_dtype,
                                scratch, FSM_STATIC_SCRATCH_BYTES, status_word, cuda_stream);
}
