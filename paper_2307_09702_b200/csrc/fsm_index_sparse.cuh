// Work-avoiding walk of the index build.
//
// Most (state, token) walks die on their first or second byte.  Tokens are therefore
// kept sorted by bucket key - the class of byte 0 and (with few enough classes) the class
// of byte 1 - so that one table lookup settles a whole bucket.  One persistent CTA per
// SM works on one index row (one state q) at a time; the compressed table is staged in
// shared memory once (bulk async copy) when it fits, else lookups use the read-only cache.
//
//   enumerate warps take units (readable first class, block of 32 second keys) from a
//             shared counter; one lookup per key tells whether the bucket is readable;
//             readable buckets are cut into 32-token chunk descriptors in shared memory.
//   walk      warps pull chunks from the list; lane = token, starting at the first byte
//             the bucket key does not cover.  A surviving token appends (id within slice,
//             end state) to the list of its *slice* (1 KB of table-width states: 512
//             consecutive token ids with 16-bit table entries).  The lists live in a
//             per-CTA scratch in global memory that stays L2 resident; a list can hold a
//             whole slice, so nothing can overflow.
//   assemble  each warp takes slices in turn: it fills a 1 KB staging buffer in shared
//             memory with `dead`, writes the slice's survivors into it, reads it back,
//             derives the bitmask words from "state != dead" and stores the finished
//             slice of the next-state row with coalesced 16- or 32-byte stores.  Global
//             memory only sees full, write-once traffic for the outputs: the tokens
//             whose first byte q cannot read cost no lookup at all.
//
// Two CTA barriers per row.  Results are identical to the dense walk.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

// An assembly slice is 1 KB of table-width states: 512 token ids with 16-bit table
// entries, 256 with 32-bit entries.
constexpr int kStageBytes = 1024;
template <typename TabT> struct Slice {
    static constexpr int kShift = sizeof(TabT) == 2 ? 9 : 8;
    static constexpr int kTokens = 1 << kShift;
};
constexpr int kMaxSliceTokens = 512;
constexpr int kMaskWords = kMaxSliceTokens / 32;  // bitmask words of one slice
constexpr int kMaxSlices = 8192;          // vocabularies up to 2 M tokens (else the dense walk)
constexpr int kDescCap = 4096;            // chunk descriptors kept per row

// Survivor record: token id within its slice and end state.
template <typename TabT> struct Entry;
template <> struct Entry<uint16_t> {
    using type = uint32_t;
    __device__ static type pack(uint32_t lid, uint32_t s) { return (s << 16) | lid; }
    __device__ static uint32_t lid(type e) { return e & 0xFFFFu; }
    __device__ static uint32_t state(type e) { return e >> 16; }
};
template <> struct Entry<int32_t> {
    using type = unsigned long long;
    __device__ static type pack(uint32_t lid, uint32_t s) { return (static_cast<type>(s) << 32) | lid; }
    __device__ static uint32_t lid(type e) { return static_cast<uint32_t>(e); }
    __device__ static uint32_t state(type e) { return static_cast<uint32_t>(e >> 32); }
};

// Chunk descriptor: up to 32 tokens at sorted position `start`, all in `state` after
// the `depth` bytes their bucket key covers.
template <typename TabT> struct Desc;
template <> struct Desc<uint16_t> {
    using type = uint2;
    __device__ static type pack(int start, uint32_t state, int count, int depth) {
        return make_uint2(start, state | ((count - 1) << 16) | ((depth - 1) << 21));
    }
    __device__ static int start(type d) { return d.x; }
    __device__ static uint32_t state(type d) { return d.y & 0xFFFFu; }
    __device__ static int count(type d) { return ((d.y >> 16) & 31) + 1; }
    __device__ static int depth(type d) { return ((d.y >> 21) & 1) + 1; }
};
template <> struct Desc<int32_t> {
    using type = uint4;
    __device__ static type pack(int start, uint32_t state, int count, int depth) {
        return make_uint4(start, state, count, depth);
    }
    __device__ static int start(type d) { return d.x; }
    __device__ static uint32_t state(type d) { return d.y; }
    __device__ static int count(type d) { return d.z; }
    __device__ static int depth(type d) { return d.w; }
};

// Shared state of the row being walked.
template <typename TabT>
struct SurvivorSink {
    typename Entry<TabT>::type* lists;  // [nslices][slice tokens], this CTA's part of the scratch
    int* counts;                        // [nslices], shared memory
    typename Desc<TabT>::type* descs;   // [desc_cap] chunk descriptors, shared memory
    int desc_cap;
    int* ctrs;                          // shared: [0] unit counter, [1] descriptors written,
                                        //         [2] chunk counter, [3] descriptor overflow
};

// One chunk: up to 32 tokens of a bucket (lane = token).  chunk_load fetches the lane's
// record and token id; chunk_finish walks the rest of the token from state `s` (after
// the DEPTH bytes the bucket key covers) and appends a survivor to its slice's list.
// `with_rec` is false for a bucket of one-byte tokens: nothing of such a token is left to
// walk, so its record is not fetched.
__device__ __forceinline__ void chunk_load(const WalkParams& p, int pos, int count, int lane,
                                           bool with_rec, uint4& rec, int32_t& id) {
    rec = make_uint4(1, 0, 0, 0);  // length 1
    id = -1;
    if (lane < count) {
        if (with_rec) rec = __ldg(p.srec + pos + lane);
        id = __ldg(p.sid + pos + lane);
    }
}

template <typename TabT, bool FULL, int DEPTH>
__device__ __forceinline__ void chunk_finish(const WalkParams& p, const TabT* __restrict__ tab,
                                             uint32_t Cs, const SurvivorSink<TabT>& sink,
                                             const uint4& rec, int32_t id, uint32_t s) {
    const uint32_t dead = p.dead;
    const int len = rec.x & 0xFFu;
    bool go = len > DEPTH;
    uint32_t st = walk_rest<TabT, FULL, DEPTH>(tab, Cs, dead, rec, len, s, go);
    if (go)  // longer than the inline record and still alive: finish on the raw bytes
        st = raw_walk(p, st, p.vocab_offsets[id], p.vocab_offsets[id + 1], kInlineBytes);
    if (id >= 0 && st != dead) {
        constexpr int kTok = Slice<TabT>::kTokens;
        const int slice = id >> Slice<TabT>::kShift;
        const int at = atomicAdd(&sink.counts[slice], 1);  // < kTok: a token survives once
        sink.lists[static_cast<size_t>(slice) * kTok + at] = Entry<TabT>::pack(id & (kTok - 1), st);
    }
}

template <typename TabT, bool FULL>
__device__ __forceinline__ void chunk_finish_depth(const WalkParams& p, const TabT* __restrict__ tab,
                                                   uint32_t Cs, const SurvivorSink<TabT>& sink,
                                                   const uint4& rec, int32_t id, uint32_t s,
                                                   int depth) {
    if (depth == 2)
        chunk_finish<TabT, FULL, 2>(p, tab, Cs, sink, rec, id, s);
    else
        chunk_finish<TabT, FULL, 1>(p, tab, Cs, sink, rec, id, s);
}

// Visits every readable bucket of state q; warps take units (readable first class,
// block of 32 second keys) from a shared counter.  With ENUMERATE the chunks of the
// readable buckets are written to the descriptor list (and walked later, see
// walk_chunks); otherwise they are walked on the spot.
template <typename TabT, bool FULL, bool ENUMERATE>
__device__ __forceinline__ void walk_row(const WalkParams& p, const TabT* __restrict__ tab, int C,
                                         uint32_t Cs, bool two_level, const int32_t* s_gstart,
                                         const SurvivorSink<TabT>& sink, int q) {
    const uint32_t dead = p.dead;
    const int lane = threadIdx.x & 31;
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (FULL) return tab[s * Cs + c];
        return __ldg(tab + static_cast<size_t>(s) * Cs + c);
    };
    // readable, non-empty first-byte classes of state q
    uint32_t lm[8];
    int n_live = 0;
#pragma unroll
    for (int cb = 0; cb < 8; ++cb) {
        lm[cb] = 0;
        if (cb * 32 < C) {
            const int c = cb * 32 + lane;
            bool ok = false;
            if (c < C) ok = (lookup(q, c) != dead) && (s_gstart[c + 1] > s_gstart[c]);
            lm[cb] = __ballot_sync(kFullWarp, ok);
            n_live += __popc(lm[cb]);
        }
    }
    const int KB = two_level ? (C + 1 + 31) / 32 : 1;  // blocks of 32 second-level keys
    const int U = n_live * KB;
    while (true) {
        int j = 0;
        if (lane == 0) j = atomicAdd(&sink.ctrs[0], 1);
        j = __shfl_sync(kFullWarp, j, 0);
        if (j >= U) break;
        const int li = j / KB, kb = j - li * KB;
        int c0 = 0, rem = li;  // the li-th readable class
#pragma unroll
        for (int cb = 0; cb < 8; ++cb) {
            const int pc = __popc(lm[cb]);
            if (rem >= 0 && rem < pc) {
                c0 = cb * 32 + __fns(lm[cb], 0, rem + 1);
                rem = -1;
            } else if (rem >= 0) {
                rem -= pc;
            }
        }
        const uint32_t s1 = lookup(q, c0);
        // lane = second-level key: bucket size, position and state after its bytes
        int cnt = 0, start = 0;
        uint32_t s2 = dead;
        if (two_level) {
            const int key2 = kb * 32 + lane;
            if (key2 <= C) {
                cnt = __ldg(p.count2 + c0 * kKeyStride + key2);
                start = __ldg(p.start2 + c0 * kKeyStride + key2);
                s2 = (key2 == 0) ? s1 : lookup(s1, key2 - 1);
            }
        } else if (lane == 0) {
            start = s_gstart[c0];
            cnt = s_gstart[c0 + 1] - start;
            s2 = s1;
        }
        const bool alive = cnt > 0 && s2 != dead;
        if (ENUMERATE) {
            const int nch = alive ? (cnt + 31) >> 5 : 0;
            int incl = nch;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(kFullWarp, incl, off);
                if (lane >= off) incl += o;
            }
            const int total = __shfl_sync(kFullWarp, incl, 31);
            if (total == 0) continue;
            int base = 0;
            if (lane == 0) base = atomicAdd(&sink.ctrs[1], total);
            base = __shfl_sync(kFullWarp, base, 0);
            if (base + total > sink.desc_cap) {
                if (lane == 0) sink.ctrs[3] = 1;  // the row is redone without the list
                continue;
            }
            const int depth = (two_level && !(kb == 0 && lane == 0)) ? 2 : 1;
            for (int k = 0; k < nch; ++k)
                sink.descs[base + incl - nch + k] =
                    Desc<TabT>::pack(start + 32 * k, s2, min(32, cnt - 32 * k), depth);
        } else {
            uint32_t m = __ballot_sync(kFullWarp, alive);
            while (m) {
                const int l = __ffs(m) - 1;
                m &= m - 1;
                const int bstart = __shfl_sync(kFullWarp, start, l);
                const int bn = __shfl_sync(kFullWarp, cnt, l);
                const uint32_t bs = __shfl_sync(kFullWarp, s2, l);
                const int depth = (two_level && !(kb == 0 && l == 0)) ? 2 : 1;
                for (int i0 = 0; i0 < bn; i0 += 32) {
                    uint4 rec;
                    int32_t id;
                    chunk_load(p, bstart + i0, bn - i0, lane, true, rec, id);
                    chunk_finish_depth<TabT, FULL>(p, tab, Cs, sink, rec, id, bs, depth);
                }
            }
        }
    }
}

// Walks the chunks of the descriptor list; a warp takes kPull at a time and issues the
// loads of all of them before walking any.
constexpr int kPull = 2;

template <typename TabT, bool FULL>
__device__ __forceinline__ void walk_chunks(const WalkParams& p, const TabT* __restrict__ tab,
                                            uint32_t Cs, bool two_level,
                                            const SurvivorSink<TabT>& sink) {
    using D = Desc<TabT>;
    const int lane = threadIdx.x & 31;
    const int total = sink.ctrs[1];
    while (true) {
        int i = 0;
        if (lane == 0) i = atomicAdd(&sink.ctrs[2], kPull);
        i = __shfl_sync(kFullWarp, i, 0);
        if (i >= total) break;
        typename D::type d[kPull];
        uint4 rec[kPull];
        int32_t id[kPull];
#pragma unroll
        for (int k = 0; k < kPull; ++k) {
            const bool have = i + k < total;
            d[k] = sink.descs[have ? i + k : i];
            // with two-level keys a bucket of depth 1 holds the one-byte tokens
            chunk_load(p, D::start(d[k]), have ? D::count(d[k]) : 0, lane,
                       !(two_level && D::depth(d[k]) == 1), rec[k], id[k]);
        }
#pragma unroll
        for (int k = 0; k < kPull; ++k)
            if (i + k < total)
                chunk_finish_depth<TabT, FULL>(p, tab, Cs, sink, rec[k], id[k], D::state(d[k]),
                                               D::depth(d[k]));
    }
}

// Assembles and stores the slices of one row; warp w takes slices w, w+32, ...
// The slice is staged in table-entry width (1 KB per warp): filled with `dead`, then
// the survivors are written into it and OR their bits into the slice's bitmask words
// (shared memory).  Each lane then reads back two 16-byte vectors, widens the states if
// the output is wider than the table entries, and stores.
template <typename TabT, typename OutT, bool HAS_OUT>
__device__ __forceinline__ void assemble_row(const WalkParams& p, const SurvivorSink<TabT>& sink,
                                             TabT* stage, uint32_t* mwords, int nslices, int q,
                                             OutT* nrow, uint32_t* mrow) {
    using E = Entry<TabT>;
    constexpr int kTok = Slice<TabT>::kTokens;
    constexpr int kShift = Slice<TabT>::kShift;
    constexpr bool kWiden = sizeof(OutT) > sizeof(TabT);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t dead = p.dead;
    const uint32_t d32 = sizeof(TabT) == 2 ? (dead | (dead << 16)) : dead;
    const uint4 dead16 = make_uint4(d32, d32, d32, d32);
    // slices are multiples of 32 bytes of output, so an aligned row has aligned slices
    const bool vec_ok = HAS_OUT && (reinterpret_cast<uintptr_t>(nrow) & (kWiden ? 31 : 15)) == 0;
    const int eos_slice = (p.eos_id >= 0 && q != p.dead && p.accept[q]) ? (p.eos_id >> kShift) : -1;
    const int last_full = p.N >> kShift;  // slices below this index are complete
    const typename E::type* lst = sink.lists + static_cast<size_t>(warp) * kTok;
    OutT* dst = HAS_OUT ? nrow + warp * kTok : nullptr;
    uint32_t* mdst = mrow + warp * (kTok / 32);
    uint4* stage4 = reinterpret_cast<uint4*>(stage);
    // The first 32 survivors of a slice are fetched one slice ahead, so that the trip to
    // the L2-resident scratch overlaps the assembly of the previous slice.
    int cnt = warp < nslices ? sink.counts[warp] : 0;
    typename E::type e0 = 0;
    if (lane < cnt) e0 = lst[lane];
    for (int sl = warp; sl < nslices; sl += kWalkWarps) {
        const int next = sl + kWalkWarps;
        const int cnt_next = next < nslices ? sink.counts[next] : 0;
        typename E::type e_next = 0;
        if (lane < cnt_next) e_next = lst[static_cast<size_t>(kWalkWarps) * kTok + lane];
        stage4[lane] = dead16;
        stage4[lane + 32] = dead16;
        if (lane < kTok / 32) mwords[lane] = 0;
        __syncwarp();
        if (lane < cnt) {
            const uint32_t lid = E::lid(e0);
            stage[lid] = static_cast<TabT>(E::state(e0));
            atomicOr(&mwords[lid >> 5], 1u << (lid & 31));
        }
        for (int i = 32 + lane; i < cnt; i += 32) {
            const typename E::type e = lst[i];
            const uint32_t lid = E::lid(e);
            stage[lid] = static_cast<TabT>(E::state(e));
            atomicOr(&mwords[lid >> 5], 1u << (lid & 31));
        }
        if (sl == eos_slice && lane == 0) {
            const uint32_t lid = p.eos_id & (kTok - 1);
            stage[lid] = static_cast<TabT>(q);
            atomicOr(&mwords[lid >> 5], 1u << (lid & 31));
        }
        __syncwarp();
        if (sl < last_full && (vec_ok || !HAS_OUT)) {
            if (lane < kTok / 32) mdst[lane] = mwords[lane];
            if (HAS_OUT) {
#pragma unroll
                for (int k = 0; k < 2; ++k) {
                    const uint4 v = stage4[lane + 32 * k];
                    if (kWiden) {  // 8 uint16 states -> 8 int32 states, one 32-byte store
                        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                        Vec32B o;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            o.w[2 * i] = w[i] & 0xFFFFu;
                            o.w[2 * i + 1] = w[i] >> 16;
                        }
                        stg_32B(reinterpret_cast<uint8_t*>(dst) + (lane + 32 * k) * 32, o);
                    } else {
                        reinterpret_cast<uint4*>(dst)[lane + 32 * k] = v;
                    }
                }
            }
        } else {  // ragged last slice or unaligned row: element-wise, still coalesced
            const int n = min(kTok, p.N - (sl << kShift));
            for (int i0 = 0; i0 < n; i0 += 32) {
                const int i = i0 + lane;
                const uint32_t sv = i < n ? static_cast<uint32_t>(stage[i]) : dead;
                const uint32_t word = __ballot_sync(kFullWarp, sv != dead);
                if (lane == 0) mdst[i0 >> 5] = word;
                if (HAS_OUT && i < n) dst[i] = static_cast<OutT>(sv);
            }
        }
        __syncwarp();  // staging is refilled by the next slice
        if (lane == 0) sink.counts[sl] = 0;  // ready for the next row's survivors
        cnt = cnt_next;
        e0 = e_next;
        lst += static_cast<size_t>(kWalkWarps) * kTok;
        if (HAS_OUT) dst += kWalkWarps * kTok;
        mdst += kWalkWarps * (kTok / 32);
    }
}

// Exact fallback when the compressed table cannot be used: every token is walked
// through the uncompressed table, one row per CTA pass, with plain stores.
template <typename OutT, bool HAS_OUT>
__device__ void raw_rows(const WalkParams& p) {
    const uint32_t dead = p.dead;
    const int nrows = p.q_end - p.q_begin;
    for (int r = blockIdx.x; r < nrows; r += gridDim.x) {
        const int q = p.q_begin + r;
        OutT* nrow = HAS_OUT ? static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N : nullptr;
        uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G;
        if (HAS_OUT)
            for (int i = threadIdx.x; i < p.N; i += blockDim.x) nrow[i] = static_cast<OutT>(dead);
        for (int i = threadIdx.x; i < p.G; i += blockDim.x) mrow[i] = 0;
        __syncthreads();  // orders the fill before the scattered stores
        if (q != p.dead) {
            for (int v = threadIdx.x; v < p.N; v += blockDim.x) {
                if (v == p.eos_id) continue;
                const int64_t o0 = p.vocab_offsets[v], o1 = p.vocab_offsets[v + 1];
                if (o0 < 0 || o1 <= o0 || o1 > p.vocab_nbytes) continue;
                const uint32_t s = raw_walk(p, q, o0, o1, 0);
                if (s != dead) {
                    if (HAS_OUT) nrow[v] = static_cast<OutT>(s);
                    atomicOr(&mrow[v >> 5], 1u << (v & 31));
                }
            }
            if (threadIdx.x == 0 && p.eos_id >= 0 && p.accept[q]) {
                if (HAS_OUT) nrow[p.eos_id] = static_cast<OutT>(q);
                atomicOr(&mrow[p.eos_id >> 5], 1u << (p.eos_id & 31));
            }
        }
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1)
walk_sparse(const WalkParams p, typename Entry<TabT>::type* scratch, uint32_t table_cap) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ int32_t s_gstart[260];
    __shared__ int s_ctrs[8];      // two sets of row counters (see SurvivorSink::ctrs)
    __shared__ int s_next_row[2];
    if (p.meta->any_bad != 0) {
        raw_rows<OutT, HAS_OUT>(p);
        return;
    }
    constexpr int kTok = Slice<TabT>::kTokens;
    const int nslices = (p.N + kTok - 1) >> Slice<TabT>::kShift;
    // dynamic shared memory: per-warp staging, slice counters, chunk descriptors, table
    const int warp = threadIdx.x >> 5;
    TabT* stage = reinterpret_cast<TabT*>(smem_raw + warp * kStageBytes);
    uint32_t* mwords = reinterpret_cast<uint32_t*>(smem_raw + kWalkWarps * kStageBytes) + warp * kMaskWords;
    int* counts = reinterpret_cast<int*>(smem_raw + kWalkWarps * (kStageBytes + kMaskWords * 4));
    const size_t desc_off = (kWalkWarps * (kStageBytes + kMaskWords * 4) +
                             static_cast<size_t>(nslices) * 4 + 15) / 16 * 16;
    typename Desc<TabT>::type* descs = reinterpret_cast<typename Desc<TabT>::type*>(smem_raw + desc_off);
    const size_t table_off = (desc_off + kDescCap * sizeof(typename Desc<TabT>::type) + 127) / 128 * 128;
    TabT* stab = reinterpret_cast<TabT*>(smem_raw + table_off);

    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int C = p.meta->C;
    const uint32_t Cs = p.meta->Cs;
    const bool two_level = p.meta->two_level != 0;
    // (a bulk copy moves multiples of 16 bytes; the table's workspace has the slack)
    const uint64_t table_bytes = (static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT) + 15) / 16 * 16;
    const bool full = table_bytes <= table_cap;
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
    SurvivorSink<TabT> sink;
    sink.lists = scratch + static_cast<size_t>(blockIdx.x) * nslices * kTok;
    sink.counts = counts;
    sink.descs = descs;
    sink.desc_cap = kDescCap;
    sink.ctrs = s_ctrs;

    // Rows differ in cost (a state that reads the class of the space byte has three times
    // the survivors), so after its first row a CTA takes rows from a global counter, and the
    // rows come in the order of p.row_order: most candidate tokens first.
    //
    // Per row: walk the chunk list | barrier | assemble the row, then enumerate the next
    // row's chunks (no barrier in between: enumeration touches only the descriptor list
    // and its counters, which nobody reads during assembly) | barrier.  The counters are
    // double buffered by row parity; the slice counters are cleared by the warp that
    // assembled the slice.
    const int nrows = p.q_end - p.q_begin;
    auto enumerate = [&](int row, int par) {
        SurvivorSink<TabT> s2 = sink;
        s2.ctrs = s_ctrs + 4 * par;
        if (full)
            walk_row<TabT, true, true>(p, stab, C, Cs, two_level, s_gstart, s2, p.q_begin + row);
        else
            walk_row<TabT, false, true>(p, gtab, C, Cs, two_level, s_gstart, s2, p.q_begin + row);
    };
    for (int i = threadIdx.x; i < nslices; i += kWalkThreads) counts[i] = 0;
    if (threadIdx.x < 8) s_ctrs[threadIdx.x] = 0;
    __syncthreads();
    auto row_at = [&](int i) { return p.row_order != nullptr ? __ldg(p.row_order + i) : i; };
    int at = blockIdx.x, par = 0;  // position in the order
    int r = at < nrows ? row_at(at) : nrows;
    if (at < nrows) enumerate(r, par);
    __syncthreads();  // the chunk list of the first row is complete
    while (at < nrows) {
        const int q = p.q_begin + r;
        OutT* nrow = HAS_OUT ? static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N : nullptr;
        uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G;
        sink.ctrs = s_ctrs + 4 * par;
        if (threadIdx.x == 0) {  // next row and its counters, published by the barrier below
            s_next_row[par ^ 1] = gridDim.x + atomicAdd(p.row_ctr, 1);
            for (int i = 0; i < 4; ++i) s_ctrs[4 * (par ^ 1) + i] = 0;
        }
        if (sink.ctrs[3] == 0) {
            if (full)
                walk_chunks<TabT, true>(p, stab, Cs, two_level, sink);
            else
                walk_chunks<TabT, false>(p, gtab, Cs, two_level, sink);
        } else {
            // more chunks than the list holds (a state that reads almost everything):
            // walk the buckets unit by unit instead
            __syncthreads();
            if (threadIdx.x == 0) sink.ctrs[0] = 0;
            __syncthreads();
            if (full)
                walk_row<TabT, true, false>(p, stab, C, Cs, two_level, s_gstart, sink, q);
            else
                walk_row<TabT, false, false>(p, gtab, C, Cs, two_level, s_gstart, sink, q);
        }
        __syncthreads();  // every survivor of the row is in its list (stores visible CTA-wide)
        at = s_next_row[par ^ 1];
        assemble_row<TabT, OutT, HAS_OUT>(p, sink, stage, mwords, nslices, q, nrow, mrow);
        r = at < nrows ? row_at(at) : nrows;
        if (at < nrows) enumerate(r, par ^ 1);
        __syncthreads();  // slice counters cleared, next chunk list complete
        par ^= 1;
    }
}

// Shared-memory bytes of walk_sparse in front of the table.
template <typename TabT>
size_t sparse_table_offset(int32_t N) {
    const size_t nslices = (static_cast<size_t>(N) + Slice<TabT>::kTokens - 1) >> Slice<TabT>::kShift;
    const size_t desc_off = (kWalkWarps * (kStageBytes + kMaskWords * 4) + nslices * 4 + 15) / 16 * 16;
    return (desc_off + kDescCap * sizeof(typename Desc<TabT>::type) + 127) / 128 * 128;
}

template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_sparse(const WalkParams& p, void* scratch, int grid, cudaStream_t stream) {
    auto kernel = walk_sparse<TabT, OutT, HAS_OUT>;
    const size_t table_off = sparse_table_offset<TabT>(p.N);
    if (table_off + 1024 > p.smem_cap) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    // what is left after staging, counters and the descriptor list may hold the table
    return launch_on(kernel, dim3(grid), dim3(kWalkThreads), p.smem_cap, stream, p,
                             static_cast<typename Entry<TabT>::type*>(scratch),
                             static_cast<uint32_t>(p.smem_cap - table_off));
}

template <typename TabT>
cudaError_t launch_sparse_for(const WalkParams& p, void* scratch, int grid, int32_t state_dtype,
                              bool has_out, cudaStream_t stream) {
    if (!has_out) return launch_sparse<TabT, int32_t, false>(p, scratch, grid, stream);
    if (state_dtype == FSM_STATE_U16) return launch_sparse<TabT, uint16_t, true>(p, scratch, grid, stream);
    return launch_sparse<TabT, int32_t, true>(p, scratch, grid, stream);
}

}  // namespace
}  // namespace fsm
