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
constexpr int kSeg = 4096;             // tokens per vocabulary segment (bucketed walk)
constexpr int kSortThreads = 1024;     // threads of the per-segment counting sort
constexpr int kTeams = 4;              // independent 8-warp teams per CTA (bucketed walk)
constexpr int kTeamWarps = 8;
constexpr int kTeamThreads = kTeamWarps * 32;
constexpr int kBatch = 4;              // 32-token chunks in flight per warp
constexpr int kBStride = 264;          // bucket-start entries kept per segment (>= 257)

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
    uint4* srec;         // [nseg*kSeg] bucket-sorted token records: {min(len,17), class of byte 1..15}
    uint16_t* slid;      // [nseg*kSeg] token id within its segment, same order as srec
    uint16_t* bstart;    // [nseg*kBStride] first sorted position of each first-byte class
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
    const size_t nseg = (static_cast<size_t>(N) + kSeg - 1) / kSeg;
    w.srec = reinterpret_cast<uint4*>(take(nseg * kSeg * sizeof(uint4)));
    w.slid = reinterpret_cast<uint16_t*>(take(nseg * kSeg * sizeof(uint16_t)));
    w.bstart = reinterpret_cast<uint16_t*>(take(nseg * kBStride * sizeof(uint16_t)));
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
                                                     uint8_t* cls, uint8_t* class_rep) {
    constexpr int kSlots = 1024;
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
               uint8_t* __restrict__ tok_len, int32_t* status) {
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
    } else {
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
    const uint16_t* slid;
    const uint16_t* bstart;
    const uint8_t* cls;
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

// One warp task: tokens 32g .. 32g+31 (lane = token) from states q0 .. q0+nq-1.
// `first` points at row q0 of the shared-memory tile; `tab` is the table used for
// the second and later bytes (the same tile when FULL, else global memory).
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void walk_task(const WalkParams& p, const TabT* __restrict__ first,
                                          const TabT* __restrict__ tab, int Cs, int q0, int nq,
                                          int g, int lane) {
    const int v = g * 32 + lane;
    const uint4 tk = p.tok_cls[v];
    const int len = p.tok_len[v];
    const uint32_t dead = p.dead;
    const bool multi = len > 1;
    const bool has_eos = (p.eos_id >= 0) && ((p.eos_id >> 5) == g);
    const bool eos_lane = (v == p.eos_id);
    const TabT* f = first + (tk.x & 0xFFu);
    for (int j = 0; j < nq; ++j) {
        const int q = q0 + j;
        uint32_t s = f[static_cast<size_t>(j) * Cs];
        bool cont = multi && (s != dead);
        if (__any_sync(kFullWarp, cont)) {
#pragma unroll
            for (int i = 1; i < kInlineBytes; ++i) {
                if (cont) {
                    const uint32_t c = tok_byte(tk, i);
                    if (FULL)
                        s = tab[s * static_cast<uint32_t>(Cs) + c];
                    else
                        s = __ldg(tab + static_cast<size_t>(s) * Cs + c);
                    cont = (s != dead) && (i + 1 < len);
                }
                if (!__any_sync(kFullWarp, cont)) break;
            }
            if (cont) {  // longer than the inline record: finish on the raw bytes
                const int64_t o0 = p.vocab_offsets[v], o1 = p.vocab_offsets[v + 1];
                s = raw_walk(p, s, o0, o1, kInlineBytes);
            }
        }
        if (has_eos && eos_lane) s = (q != p.dead && p.accept[q]) ? q : dead;
        emit<OutT, HAS_OUT>(p, q, g, v, lane, s);
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
                if (full)
                    walk_task<TabT, OutT, HAS_OUT, true>(p, first, tile, Cs, q0, nq, g, lane);
                else
                    walk_task<TabT, OutT, HAS_OUT, false>(p, first, gtab, Cs, q0, nq, g, lane);
            }
        }
    }
}


// ---------------------------------------------------------------------------- 3b
// Bucketed layout for the work-avoiding walk: the vocabulary is cut into segments of
// kSeg consecutive token ids; inside a segment the non-empty tokens are grouped by the
// class of their first byte (counting sort in shared memory).  A record keeps the
// length and the classes of bytes 1..15; the first byte's class is the bucket.
__global__ void __launch_bounds__(kSortThreads)
bucket_tokens(const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
              int64_t vocab_nbytes, int32_t N, int32_t eos_id, const IndexMeta* meta,
              const uint8_t* __restrict__ cls, uint4* __restrict__ srec,
              uint16_t* __restrict__ slid, uint16_t* __restrict__ bstart, int32_t* status) {
    constexpr int kPer = kSeg / kSortThreads;
    __shared__ int hist[257];
    __shared__ int cursor[257];
    __shared__ uint8_t s_cls[256];
    const int seg = blockIdx.x;
    const int base = seg * kSeg;
    const int n = min(kSeg, N - base);
    if (threadIdx.x < 256) s_cls[threadIdx.x] = cls[threadIdx.x];
    for (int c = threadIdx.x; c < 257; c += kSortThreads) hist[c] = 0;
    __syncthreads();
    int64_t start[kPer];
    int length[kPer];  // 0 = not bucketed (empty, EOS, bad offsets, past the end)
    int first[kPer];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int t = threadIdx.x + k * kSortThreads;
        const int v = base + t;
        start[k] = 0;
        length[k] = 0;
        first[k] = 0;
        if (t < n && v != eos_id) {
            const int64_t o0 = vocab_offsets[v], o1 = vocab_offsets[v + 1];
            if (o0 < 0 || o1 < o0 || o1 > vocab_nbytes) {
                bad = true;
            } else if (o1 > o0) {
                start[k] = o0;
                length[k] = static_cast<int>(min(o1 - o0, static_cast<int64_t>(kInlineBytes + 1)));
                first[k] = s_cls[vocab_bytes[o0]];
                atomicAdd(&hist[first[k]], 1);
            }
        }
    }
    if (__syncthreads_or(bad) && threadIdx.x == 0) raise_flag(status, FSM_FLAG_OFFSETS);
    if (threadIdx.x < 32) {  // exclusive prefix over the 256 counters, 8 per lane
        int local[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            local[i] = sum;
            sum += hist[threadIdx.x * 8 + i];
        }
        int incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullWarp, incl, off);
            if (static_cast<int>(threadIdx.x) >= off) incl += o;
        }
        const int excl = incl - sum;
#pragma unroll
        for (int i = 0; i < 8; ++i) cursor[threadIdx.x * 8 + i] = excl + local[i];
        if (threadIdx.x == 31) cursor[256] = incl;
    }
    __syncthreads();
    for (int c = threadIdx.x; c < 257; c += kSortThreads)
        bstart[seg * kBStride + c] = static_cast<uint16_t>(cursor[c]);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        if (length[k] == 0) continue;
        uint32_t w[4] = {static_cast<uint32_t>(length[k]), 0, 0, 0};
        const int nb = min(length[k], kInlineBytes);
        for (int i = 1; i < nb; ++i)
            w[i >> 2] |= static_cast<uint32_t>(s_cls[vocab_bytes[start[k] + i]]) << ((i & 3) * 8);
        const int pos = atomicAdd(&cursor[first[k]], 1);
        srec[base + pos] = make_uint4(w[0], w[1], w[2], w[3]);
        slid[base + pos] = static_cast<uint16_t>(threadIdx.x + k * kSortThreads);
    }
}

// ---------------------------------------------------------------------------- 4b
// Work-avoiding walk.  One persistent CTA per SM; the compressed table is staged in
// shared memory once (bulk async copy) when it fits.  The CTA's 32 warps form four
// teams of eight; a team's unit of work is (state q, vocabulary segment).  The team
// fills the segment's slice of row q with `dead` in shared memory, finds the first-byte
// classes that q can read (one table lookup per class), walks only the tokens of those
// buckets (lane = token, several 32-token chunks in flight per warp), scatters the
// survivors' end states and bitmask bits into the slice, then streams the slice to
// global memory with coalesced 16-byte stores.  Every (state, token) pair still gets
// its entry; pairs whose first byte is unreadable are settled by the fill.
struct LiveBucket {
    uint32_t s1;      // state after the first byte
    uint16_t start;   // first sorted position of the bucket
    uint16_t count;
};

struct TeamScratch {
    LiveBucket live[256];
    uint16_t cpre[260];  // 32-token chunks before each live bucket; [n_live] = total
    int n_live;
    int n_chunks;
};

template <typename OutT, bool HAS_OUT>
__host__ __device__ constexpr size_t team_bytes() {
    return (HAS_OUT ? kSeg * sizeof(OutT) : 0) + kSeg / 8 + ((sizeof(TeamScratch) + 15) / 16) * 16;
}

__device__ __forceinline__ void team_sync(int team) {
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "n"(kTeamThreads) : "memory");
}

template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void bucketed_unit(const WalkParams& p, const TabT* __restrict__ tab,
                                              int C, int Cs, bool raw, OutT* row, uint32_t* mbits,
                                              TeamScratch* ts, int team, int r, int seg) {
    const uint32_t dead = p.dead;
    const int lane = threadIdx.x & 31;
    const int tw = (threadIdx.x >> 5) & (kTeamWarps - 1);
    const int tt = threadIdx.x & (kTeamThreads - 1);
    const int q = p.q_begin + r;
    const int base = seg * kSeg;
    const int n = min(kSeg, p.N - base);
    constexpr int kVecElems = 16 / sizeof(OutT);
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (FULL) return tab[s * static_cast<uint32_t>(Cs) + c];
        return __ldg(tab + static_cast<size_t>(s) * Cs + c);
    };

    // ---- fill
    if (HAS_OUT) {
        const uint32_t d = sizeof(OutT) == 2 ? (dead | (dead << 16)) : dead;
        const uint4 dead16 = make_uint4(d, d, d, d);
        for (int i = tt; i < kSeg / kVecElems; i += kTeamThreads)
            reinterpret_cast<uint4*>(row)[i] = dead16;
    }
    for (int i = tt; i < kSeg / 32; i += kTeamThreads) mbits[i] = 0;
    if (tw == 0 && !raw) {
        int cnt = 0, chunks = 0;
        const uint16_t* bs = p.bstart + static_cast<size_t>(seg) * kBStride;
        for (int c0 = 0; c0 < C; c0 += 32) {
            const int c = c0 + lane;
            uint32_t s1 = dead;
            int start = 0, num = 0;
            if (c < C) {
                s1 = lookup(q, c);
                start = bs[c];
                num = bs[c + 1] - start;
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
                b.start = static_cast<uint16_t>(start);
                b.count = static_cast<uint16_t>(num);
                ts->live[pos] = b;
                ts->cpre[pos] = static_cast<uint16_t>(chunks + incl - nch);
            }
            cnt += __popc(m);
            chunks += __shfl_sync(kFullWarp, incl, 31);
        }
        if (lane == 0) {
            ts->n_live = cnt;
            ts->n_chunks = chunks;
            ts->cpre[cnt] = static_cast<uint16_t>(chunks);
        }
    }
    team_sync(team);

    // ---- walk the live buckets, kBatch chunks in flight per warp
    if (!raw) {
        const int M = ts->n_chunks;
        int b = 0;
        for (int g0 = tw; g0 < M; g0 += kTeamWarps * kBatch) {
            uint4 rec[kBatch];
            uint32_t lid[kBatch], st[kBatch];
            bool cont[kBatch], act[kBatch];
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                const int g = g0 + k * kTeamWarps;
                rec[k] = make_uint4(0, 0, 0, 0);
                lid[k] = 0;
                st[k] = dead;
                act[k] = false;
                if (g < M) {
                    while (g >= ts->cpre[b + 1]) ++b;
                    const LiveBucket lb = ts->live[b];
                    const int i = (g - ts->cpre[b]) * 32 + lane;
                    st[k] = lb.s1;
                    if (i < lb.count) {
                        act[k] = true;
                        rec[k] = __ldg(p.srec + base + lb.start + i);
                        lid[k] = p.slid[base + lb.start + i];
                    }
                }
            }
            bool any_cont = false;
#pragma unroll
            for (int k = 0; k < kBatch; ++k) {
                cont[k] = (rec[k].x & 0xFFu) > 1;
                any_cont |= cont[k];
            }
            if (__any_sync(kFullWarp, any_cont)) {
#pragma unroll
                for (int j = 1; j < kInlineBytes; ++j) {
                    any_cont = false;
#pragma unroll
                    for (int k = 0; k < kBatch; ++k) {
                        if (cont[k]) {
                            st[k] = lookup(st[k], tok_byte(rec[k], j));
                            cont[k] = (st[k] != dead) && (j + 1 < static_cast<int>(rec[k].x & 0xFFu));
                        }
                        any_cont |= cont[k];
                    }
                    if (!__any_sync(kFullWarp, any_cont)) break;
                }
#pragma unroll
                for (int k = 0; k < kBatch; ++k)
                    if (cont[k]) {  // longer than the inline record: finish on the raw bytes
                        const int v = base + lid[k];
                        st[k] = raw_walk(p, st[k], p.vocab_offsets[v], p.vocab_offsets[v + 1],
                                         kInlineBytes);
                    }
            }
#pragma unroll
            for (int k = 0; k < kBatch; ++k)
                if (act[k] && st[k] != dead) {
                    if (HAS_OUT) row[lid[k]] = static_cast<OutT>(st[k]);
                    atomicOr(&mbits[lid[k] >> 5], 1u << (lid[k] & 31));
                }
        }
    } else {
        for (int t = tt; t < n; t += kTeamThreads) {
            const int v = base + t;
            if (v == p.eos_id || q == p.dead) continue;
            const int64_t o0 = p.vocab_offsets[v], o1 = p.vocab_offsets[v + 1];
            if (o0 < 0 || o1 <= o0 || o1 > p.vocab_nbytes) continue;
            const uint32_t s = raw_walk(p, q, o0, o1, 0);
            if (s != dead) {
                if (HAS_OUT) row[t] = static_cast<OutT>(s);
                atomicOr(&mbits[t >> 5], 1u << (t & 31));
            }
        }
    }
    if (tt == 0 && p.eos_id >= base && p.eos_id < base + n && q != p.dead && p.accept[q]) {
        const int e = p.eos_id - base;
        if (HAS_OUT) row[e] = static_cast<OutT>(q);
        atomicOr(&mbits[e >> 5], 1u << (e & 31));
    }
    team_sync(team);

    // ---- stream the slice out
    if (HAS_OUT) {
        OutT* dst = static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N + base;
        if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
            const int nvec = n / kVecElems;
            for (int i = tt; i < nvec; i += kTeamThreads)
                reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(row)[i];
            for (int i = nvec * kVecElems + tt; i < n; i += kTeamThreads) dst[i] = row[i];
        } else {
            for (int i = tt; i < n; i += kTeamThreads) dst[i] = row[i];
        }
    }
    uint32_t* mdst = p.mask + static_cast<size_t>(r) * p.G + (base >> 5);
    for (int i = tt; i < (n + 31) / 32; i += kTeamThreads) mdst[i] = mbits[i];
    team_sync(team);  // the slice is free for the next unit's fill
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk_bucketed(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    constexpr size_t kTeamBytes = team_bytes<OutT, HAS_OUT>();
    constexpr size_t kTeamArea = (kTeams * kTeamBytes + 127) / 128 * 128;
    const int team = threadIdx.x / kTeamThreads;
    uint8_t* mine = smem_raw + team * kTeamBytes;
    OutT* row = reinterpret_cast<OutT*>(mine);
    uint32_t* mbits = reinterpret_cast<uint32_t*>(mine + (HAS_OUT ? kSeg * sizeof(OutT) : 0));
    TeamScratch* ts = reinterpret_cast<TeamScratch*>(reinterpret_cast<uint8_t*>(mbits) + kSeg / 8);
    TabT* stab = reinterpret_cast<TabT*>(smem_raw + kTeamArea);

    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int C = p.meta->C, Cs = p.meta->Cs;
    const bool raw = p.meta->any_bad != 0;
    const uint64_t table_bytes = static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT);
    const bool full = !raw && p.smem_cap > kTeamArea && table_bytes <= p.smem_cap - kTeamArea;

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
                bulk_copy_g2s(reinterpret_cast<uint8_t*>(stab) + o,
                              reinterpret_cast<const uint8_t*>(gtab) + o,
                              min(kBulkChunk, bytes - o), &bar);
        }
        bool ok = mbar_wait_bounded(&bar, 0);
        if (!ok) ok = mbar_wait_bounded(&bar, 0);  // drain before giving up
        if (!__syncthreads_and(ok)) {
            if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
            return;
        }
    }

    const int nseg = (p.N + kSeg - 1) / kSeg;
    const int64_t units = static_cast<int64_t>(p.q_end - p.q_begin) * nseg;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kTeams;
    for (int64_t u = static_cast<int64_t>(blockIdx.x) * kTeams + team; u < units; u += stride) {
        const int r = static_cast<int>(u / nseg);
        const int seg = static_cast<int>(u - static_cast<int64_t>(r) * nseg);
        if (full)
            bucketed_unit<TabT, OutT, HAS_OUT, true>(p, stab, C, Cs, raw, row, mbits, ts, team, r, seg);
        else
            bucketed_unit<TabT, OutT, HAS_OUT, false>(p, gtab, C, Cs, raw, row, mbits, ts, team, r, seg);
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_bucketed(const WalkParams& p, int grid, cudaStream_t stream) {
    auto kernel = walk_bucketed<TabT, OutT, HAS_OUT>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    kernel<<<grid, kWalkThreads, p.smem_cap, stream>>>(p);
    return cudaGetLastError();
}

template <typename TabT>
cudaError_t launch_bucketed_for(const WalkParams& p, int grid, int32_t state_dtype, bool has_out,
                                cudaStream_t stream) {
    if (!has_out) return launch_bucketed<TabT, int32_t, false>(p, grid, stream);
    if (state_dtype == FSM_STATE_U16) return launch_bucketed<TabT, uint16_t, true>(p, grid, stream);
    return launch_bucketed<TabT, int32_t, true>(p, grid, stream);
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
    derive_classes<<<1, 256, 0, stream>>>(ws.partial, hash_blocks, ws.meta, ws.cls, ws.class_rep);
    const int G = (N + 31) / 32;
    const int row_blocks = Q < 2 * dev.sm_count ? Q : 2 * dev.sm_count;
    const bool bucketed = tune.walk_algo != 1;
    const int tok_blocks = bucketed ? 0 : (G * 32 + 255) / 256;  // token records of the dense walk
    if (wide)
        prepare_inputs<int32_t><<<row_blocks + tok_blocks, 256, 0, stream>>>(
            dfa_trans, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state, eos_id,
            row_blocks, ws.meta, ws.cls, ws.class_rep, static_cast<int32_t*>(ws.table),
            ws.tok_cls, ws.tok_len, status_word);
    else
        prepare_inputs<uint16_t><<<row_blocks + tok_blocks, 256, 0, stream>>>(
            dfa_trans, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N, dead_state, eos_id,
            row_blocks, ws.meta, ws.cls, ws.class_rep, static_cast<uint16_t*>(ws.table),
            ws.tok_cls, ws.tok_len, status_word);
    const int nseg = (N + kSeg - 1) / kSeg;
    if (bucketed)
        bucket_tokens<<<nseg, kSortThreads, 0, stream>>>(vocab_bytes, vocab_offsets, vocab_nbytes,
                                                          N, eos_id, ws.meta, ws.cls, ws.srec,
                                                          ws.slid, ws.bstart, status_word);
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
    p.slid = ws.slid;
    p.bstart = ws.bstart;
    p.cls = ws.cls;
    int cap = dev.smem_optin - 1024;  // static shared memory and alignment slack
    if (tune.smem_table_cap > 0 && tune.smem_table_cap < cap) cap = tune.smem_table_cap;
    if (bucketed) {
        const int min_cap = static_cast<int>(kTeams * team_bytes<int32_t, true>()) + 256;
        if (cap < min_cap) cap = min_cap;
        p.smem_cap = static_cast<uint32_t>(cap) / 128 * 128;
        const int64_t units = static_cast<int64_t>(q_end - q_begin) * nseg;
        int64_t grid = dev.sm_count;
        if (tune.walk_ctas > 0) grid = tune.walk_ctas;
        if (grid > (units + kTeams - 1) / kTeams) grid = (units + kTeams - 1) / kTeams;
        const int prof = profile_begin(stream);
        cudaError_t e = wide ? launch_bucketed_for<int32_t>(p, static_cast<int>(grid), state_dtype,
                                                           next_state != nullptr, stream)
                             : launch_bucketed_for<uint16_t>(p, static_cast<int>(grid), state_dtype,
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
