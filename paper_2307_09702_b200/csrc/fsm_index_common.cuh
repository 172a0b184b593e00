// Shared definitions of the index-build kernels (paper Section 3, Algorithms 3 and 4).
#pragma once

#include "fsm_common.cuh"

namespace fsm {
namespace {

constexpr int kHashBlocks = 32;
constexpr int kMaxCs = 264;             // bound on the row stride (256 classes + the null class)
constexpr int kWalkThreads = 1024;
constexpr int kWalkWarps = kWalkThreads / 32;
constexpr int kChunk = 32;              // states per warp task (dense walk)
constexpr int kSmallChunk = 8;          // the same for builds of few tasks
constexpr int kInlineBytes = 16;        // token bytes kept in a 16-byte record (dense walk)
constexpr int kSortedInline = 12;       // token bytes covered by a sorted record (its last word is the id)
constexpr uint32_t kBulkChunk = 32768;  // bytes per bulk copy instruction (table staging)
constexpr int kKeyStride = 129;         // second-level keys per first-byte class (two-level sort)
constexpr int kKeys = kKeyStride * kKeyStride;
constexpr int kTwoLevelMaxC = 127;      // more classes than this: one-level buckets only
constexpr int kCsrDenseRows = 256;      // smaller automata: compressed rows cut out of a dense table
constexpr int kStaticSmemSlack = 3072;   // static shared memory of the walk kernels, with margin

struct IndexMeta {
    int32_t C;          // number of byte classes (the null class has id C)
    int32_t Cs;         // row stride of the compressed table, entries
    int32_t any_bad;    // set when the compressed table cannot be used (exact fallback)
    int32_t two_level;  // tokens are bucketed by (class of byte 0, class of byte 1)
};

struct Workspace {
    IndexMeta* meta;
    uint8_t* cls;        // [256] byte -> class
    uint64_t* partial;   // [kHashBlocks][256] column hash partial sums
    void* table;         // [Q][Cs] of TabT
    // dense walk: token records in token order (aliases the sorted records)
    uint4* tok_cls;      // [G*32] first 16 class ids of each token
    uint8_t* tok_len;    // [G*32] min(length, 17)
    // work-avoiding walks: tokens sorted by bucket key
    uint4* srec;         // [N] {min(len,13), classes of bytes 1..11, token id}
    int32_t* gstart;     // [257] first sorted position of each first-byte class
    int32_t* row_ctr;    // [1] rows handed out by the row-wise walk beyond the first one per CTA
    int32_t* count2;     // [kKeys] tokens per (first class, second key)
    int32_t* cursor2;    // [kKeys] placement cursors
    int32_t* start2;     // [kKeys] first sorted position of each (first class, second key)
    // bucket walk: bit planes of the one-byte tokens by class, live classes of every state
    uint32_t* planes;    // [256][plane_stride(W)] bit v of plane c: token v is the one byte of class c
    uint8_t* tok_c1;     // [N rounded up to 1024] class of a one-byte token, else the null class
    uint32_t* live;      // [Q][8] bit c: state reads class c
    int32_t* row_count;  // [Q] allowed tokens per row (compressed-row build)
    uint16_t* tok_head;  // [N] first byte | min(length, 255) << 8 of every token
    int32_t* row_order;  // [Q] rows of the row-wise walk, most candidate tokens first
    int32_t* win_order;  // [G] windows of 32 sorted tokens of the bucket walk, most keys first
    uint16_t* csr_dense; // [Q][N] end states of an automaton of fewer than kCsrDenseRows states
                         // (compressed-row build: the rows are cut out of the dense table)
    size_t bytes;        // everything above
    size_t dense_bytes;  // the leading part that the dense walk needs
};

inline size_t table_elem_bytes(int32_t Q) { return Q <= 65535 ? 2 : 4; }

// Words between the bit planes of two classes: the row length rounded up so that every
// plane starts on a 16-byte boundary.
__host__ __device__ constexpr int plane_stride(int W) { return (W + 3) & ~3; }

// Row stride of the compressed table in entries: room for C classes and the null class,
// and an odd number of 32-bit words, so that the same column of 32 different rows lies
// in 32 different shared-memory banks (lanes that hold different states and look up one
// class do not conflict).
template <typename TabT>
__host__ __device__ constexpr int table_row_stride(int C) {
    return sizeof(TabT) == 2 ? ((C + 1 + 1) / 4 * 4 + 2) : ((C + 1) | 1);
}

inline Workspace carve(void* base, int32_t Q, int32_t N) {
    Workspace w;
    uint8_t* p = static_cast<uint8_t*>(base);
    size_t off = 0;
    auto take = [&](size_t n) {
        uint8_t* r = p ? p + off : nullptr;
        off += align_up(n, 256);
        return r;
    };
    const size_t G32 = (static_cast<size_t>(N) + 31) / 32 * 32;
    w.meta = reinterpret_cast<IndexMeta*>(take(sizeof(IndexMeta)));
    w.cls = take(256);
    w.partial = reinterpret_cast<uint64_t*>(take(sizeof(uint64_t) * kHashBlocks * 256));
    w.table = take(static_cast<size_t>(Q) * kMaxCs * table_elem_bytes(Q));
    const size_t dense_bytes = G32 * sizeof(uint4) + G32;
    uint8_t* tokens = take(dense_bytes);  // (the sorted records, N * 16 bytes, fit as well)
    w.tok_cls = reinterpret_cast<uint4*>(tokens);
    w.tok_len = tokens ? tokens + G32 * sizeof(uint4) : nullptr;
    w.srec = reinterpret_cast<uint4*>(tokens);
    w.gstart = reinterpret_cast<int32_t*>(take(257 * sizeof(int32_t)));
    w.row_ctr = reinterpret_cast<int32_t*>(take(sizeof(int32_t)));
    w.count2 = reinterpret_cast<int32_t*>(take(kKeys * sizeof(int32_t)));
    w.cursor2 = reinterpret_cast<int32_t*>(take(kKeys * sizeof(int32_t)));
    w.start2 = reinterpret_cast<int32_t*>(take(kKeys * sizeof(int32_t)));
    w.dense_bytes = off;
    w.planes = reinterpret_cast<uint32_t*>(take(256 * static_cast<size_t>(plane_stride(static_cast<int>(G32 / 32))) * sizeof(uint32_t)));
    w.tok_c1 = take((static_cast<size_t>(N) + 1023) / 1024 * 1024);
    w.live = reinterpret_cast<uint32_t*>(take(static_cast<size_t>(Q) * 8 * sizeof(uint32_t)));
    w.row_count = reinterpret_cast<int32_t*>(take(static_cast<size_t>(Q) * sizeof(int32_t)));
    w.tok_head = reinterpret_cast<uint16_t*>(take(static_cast<size_t>(N) * sizeof(uint16_t)));
    w.row_order = reinterpret_cast<int32_t*>(take(static_cast<size_t>(Q) * sizeof(int32_t)));
    w.win_order = reinterpret_cast<int32_t*>(take(G32 / 32 * sizeof(int32_t)));
    w.csr_dense = reinterpret_cast<uint16_t*>(
        take(Q < kCsrDenseRows ? static_cast<size_t>(Q) * N * sizeof(uint16_t) : 0));
    w.bytes = off;
    return w;
}

struct WalkParams {
    const void* table;
    const IndexMeta* meta;
    const int32_t* trans;
    const uint8_t* accept;
    const uint8_t* vocab_bytes;
    const int32_t* vocab_offsets;
    int64_t vocab_nbytes;
    int32_t Q, N, G, dead, eos_id, q_begin, q_end;
    uint32_t smem_cap;  // bytes of dynamic shared memory requested at launch
    // dense walk
    const uint4* tok_cls;
    const uint8_t* tok_len;
    // work-avoiding walks
    const uint4* srec;
    const int32_t* gstart;
    const int32_t* count2;
    const int32_t* start2;
    int32_t* row_ctr;
    // bucket walk
    const uint32_t* planes;
    const uint8_t* tok_c1;
    const uint32_t* live;
    const int32_t* row_order;  // row-wise walk: rows in the order they are handed out, or null
    const int32_t* win_order;  // bucket walk: windows in the order they are handed out, or null
    int32_t chunk;             // dense walk: states per warp task (kChunk or kSmallChunk)
    int32_t wait_probe;        // > 0: polls of a wait that nothing ends (test of the give-up path)
    // outputs
    uint32_t* mask;
    void* next;
    int32_t* status;
};

#ifdef __CUDACC__
__device__ __forceinline__ uint64_t mix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

__device__ __forceinline__ uint32_t clamp_state(int32_t v, int32_t Q, int32_t dead) {
    return (static_cast<uint32_t>(v) >= static_cast<uint32_t>(Q)) ? dead : v;
}

// Bucket key of a token in the sorted order of the work-avoiding walks.
__device__ __forceinline__ int bucket_key(bool two_level, int first, int second_key) {
    return two_level ? first * kKeyStride + second_key : first;
}

// Bounds-checked view of one token for the token-side preparation kernels.  The raw part
// (offsets and first bytes) does not depend on the byte classes, so it can be fetched
// before they are known.
struct TokenRaw {
    int64_t start;
    int len;          // min(length, kInlineBytes + 1); 0 = not bucketed (empty, EOS, bad offsets)
    uint32_t b0, b1;  // first two bytes
};
struct TokenInfo {
    int64_t start;
    int len;
    int first;       // class of byte 0
    int second_key;  // 0 for one-byte tokens, else 1 + class of byte 1
};

__device__ __forceinline__ TokenRaw token_raw(const uint8_t* __restrict__ vocab_bytes,
                                              const int32_t* __restrict__ vocab_offsets,
                                              int64_t vocab_nbytes, int32_t N, int32_t eos_id,
                                              int64_t v, bool* bad) {
    TokenRaw t = {0, 0, 0, 0};
    if (v < N && v != eos_id) {
        const int64_t o0 = vocab_offsets[v], o1 = vocab_offsets[v + 1];
        if (o0 < 0 || o1 < o0 || o1 > vocab_nbytes) {
            *bad = true;
        } else if (o1 > o0) {
            t.start = o0;
            t.len = static_cast<int>(min(o1 - o0, static_cast<int64_t>(kInlineBytes + 1)));
            t.b0 = vocab_bytes[o0];
            if (t.len > 1) t.b1 = vocab_bytes[o0 + 1];
        }
    }
    return t;
}

__device__ __forceinline__ TokenInfo token_classify(const TokenRaw& r, const uint8_t* s_cls) {
    TokenInfo t = {r.start, r.len, 0, 0};
    if (r.len > 0) t.first = s_cls[r.b0];
    if (r.len > 1) t.second_key = 1 + s_cls[r.b1];
    return t;
}

__device__ __forceinline__ uint32_t tok_byte(const uint4& t, int i) {
    const uint32_t w = (i >> 2) == 0 ? t.x : (i >> 2) == 1 ? t.y : (i >> 2) == 2 ? t.z : t.w;
    return (w >> ((i & 3) * 8)) & 0xFFu;
}

// Walks bytes [from, o1 - o0) of a token through the uncompressed table.
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

// Bytes START .. END-1 of one token walked from state s, all 32 lanes in lock step.  `go`
// says whether this lane still has a live walk with bytes left.  The loop is
// warp-uniform (one vote per byte) and its body has no branches: lanes that are done
// keep their state through a select.  Every state value is a valid table row
// (out-of-range entries were replaced by `dead` when the table was compressed), so the
// shared-memory lookup needs no guard; the global-memory lookup is predicated to save
// traffic.  On return `go` is true only for tokens longer than the record covers.
// (`tab_n`: entries of the table, looked at by the range-checked build only.)
template <typename TabT, bool FULL, int START, int END = kInlineBytes>
__device__ __forceinline__ uint32_t walk_rest(const TabT* __restrict__ tab, uint32_t Cs,
                                              uint32_t dead, const uint4& tk, int len, uint32_t s,
                                              bool& go, uint32_t tab_n, int32_t* status) {
#pragma unroll
    for (int i = START; i < END; ++i) {
        if (!__any_sync(kFullWarp, go)) break;
        const uint32_t c = tok_byte(tk, i);
        uint32_t ns;
        if (FULL) {
            ns = idx_ok(s * Cs + c, tab_n, status) ? tab[s * Cs + c] : dead;
        } else {
            ns = s;
            if (go && idx_ok(static_cast<size_t>(s) * Cs + c, tab_n, status))
                ns = __ldg(tab + static_cast<size_t>(s) * Cs + c);
        }
        s = go ? ns : s;
        go = go && (ns != dead) && (i + 1 < len);
    }
    return s;
}
#endif  // __CUDACC__

}  // namespace
}  // namespace fsm
