// Row-wise walk of the index build (paper Section 3, Algorithms 3 and 4): one persistent
// CTA per SM produces one index row (one start state q) at a time.
//
// A row is mostly `dead`, and four out of five of its survivors are tokens of a single
// byte, whose end state is delta(q, byte) - the textbook case "index = transition table".
// So the row is written in two layers:
//
//   fill      every entry of the row comes from one look-up in a small table of the row:
//             lut[c] = delta(q, class c), indexed by the token's one-byte class (the null
//             class, which leads to dead, for every token that is not exactly one byte
//             long).  Threads own whole 32-byte output vectors: 8 (or 16) class ids are
//             read with one load, looked up in shared memory and stored with one 256-bit
//             store.  With up to 127 byte classes the table is replicated per lane
//             (lut[c][lane], bank = lane), so a look-up is conflict-free and its address is
//             a single byte permute of the packed class ids.  The bitmask words of the row
//             are the OR of the bit planes of the one-byte tokens over the classes q reads.
//   patch     tokens of two or more bytes are kept sorted by (class of byte 0, class of
//             byte 1).  The buckets q can read are cut into 32-token chunks (enumerate),
//             the chunks are walked from byte 2 on (lane = token) and each survivor stores
//             its end state straight into the row just written and ORs its bit into the
//             row's bitmask words - about a thousand scattered stores per row, which land
//             in lines that are still in L2.
//
// The compressed table is staged in shared memory once (bulk async copy) when it fits, else
// look-ups use the read-only cache.  Rows are handed out from a global counter in the
// order the preparation ranked them (most candidate tokens first).  Two CTA barriers per
// row: fill | barrier | patch, then table and chunk list of the next row | barrier.  Every
// output word has one writer in the fill; the patches of a row are issued by the same CTA
// after a barrier, to addresses no other CTA touches.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

constexpr int kLutClasses = 128;              // classes (null class included) of the replicated table
constexpr int kLutBytes = kLutClasses * 256;  // per class: two copies (row parity) of 32 lane words
constexpr int kRowDescCap = 2048;             // chunk descriptors kept per row

// Chunk descriptor: up to 32 tokens at sorted position `start`, all in `state` after the
// bytes their bucket key covers.
template <typename TabT> struct Desc;
template <> struct Desc<uint16_t> {
    using type = uint2;
    __device__ static type pack(int start, uint32_t state, int count) {
        return make_uint2(start, state | ((count - 1) << 16));
    }
    __device__ static int start(type d) { return d.x; }
    __device__ static uint32_t state(type d) { return d.y & 0xFFFFu; }
    __device__ static int count(type d) { return ((d.y >> 16) & 31) + 1; }
};
template <> struct Desc<int32_t> {
    using type = uint4;
    __device__ static type pack(int start, uint32_t state, int count) {
        return make_uint4(start, state, count, 0);
    }
    __device__ static int start(type d) { return d.x; }
    __device__ static uint32_t state(type d) { return d.y; }
    __device__ static int count(type d) { return d.z; }
};

// What the phases of one row share (shared memory, one set per row parity).
template <typename TabT>
struct RowCtx {
    typename Desc<TabT>::type* descs;  // [kRowDescCap]
    int* ctrs;                         // [0] unit counter, [1] descriptors written,
                                       // [2] chunk counter, [3] descriptor overflow
    uint8_t* cls;                      // [256] the classes q reads that begin some token ...
    int* ncls;                         // ... and their number
};

// Output side of one row.
template <typename OutT>
struct RowOut {
    OutT* nrow;      // next-state row or null
    uint32_t* mrow;  // bitmask row
};

// ---------------------------------------------------------------------------------------
// One chunk: up to 32 tokens of a bucket (lane = token), all in state `s` after DEPTH bytes.
// Survivors store their end state into the row and OR their bit into the bitmask.
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL, int DEPTH>
__device__ __forceinline__ void chunk_patch(const WalkParams& p, const TabT* __restrict__ tab,
                                            uint32_t Cs, const RowOut<OutT>& out, const uint4& rec,
                                            uint32_t s) {
    const uint32_t dead = p.dead;
    const int len = rec.x & 0xFFu;
    const int32_t id = static_cast<int32_t>(rec.w);
    bool go = len > DEPTH;
    uint32_t st = walk_rest<TabT, FULL, DEPTH, kSortedInline>(tab, Cs, dead, rec, len, s, go,
                                                              static_cast<uint32_t>(p.Q) * Cs, p.status);
    if (go && idx_ok(id, p.N, p.status))  // longer than the record covers and still alive:
        st = raw_walk(p, st, p.vocab_offsets[id], p.vocab_offsets[id + 1], kSortedInline);  // the raw bytes
    // (a one-byte token of a one-level bucket already has its entry from the fill)
    if (id >= 0 && len > 1 && st != dead && idx_ok(id, p.N, p.status)) {
        if (HAS_OUT) out.nrow[id] = static_cast<OutT>(st);
        atomicOr(out.mrow + (id >> 5), 1u << (id & 31));
    }
}

template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void chunk_patch_level(const WalkParams& p, const TabT* __restrict__ tab,
                                                  uint32_t Cs, bool two_level, const RowOut<OutT>& out,
                                                  const uint4& rec, uint32_t s) {
    if (two_level)
        chunk_patch<TabT, OutT, HAS_OUT, FULL, 2>(p, tab, Cs, out, rec, s);
    else
        chunk_patch<TabT, OutT, HAS_OUT, FULL, 1>(p, tab, Cs, out, rec, s);
}

// The lane's record of a chunk (length 1 and id -1 beyond the chunk's end: nothing to walk).
__device__ __forceinline__ uint4 chunk_fetch(const WalkParams& p, int pos, int count, int lane) {
    uint4 rec = make_uint4(1, 0, 0, 0xFFFFFFFFu);
    if (lane < count && idx_ok(pos + lane, p.N, p.status)) rec = __ldg(p.srec + pos + lane);
    return rec;
}

// Visits every readable bucket of tokens longer than one byte of state q; warps take units
// (readable first class, block of 32 second keys) from a shared counter.  With ENUMERATE
// the buckets are cut into chunk descriptors; otherwise they are walked on the spot (a row
// with more chunks than the list holds).
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL, bool ENUMERATE>
__device__ __forceinline__ void visit_buckets(const WalkParams& p, const TabT* __restrict__ tab,
                                              int C, uint32_t Cs, bool two_level,
                                              const int32_t* s_gstart, const RowCtx<TabT>& ctx,
                                              const RowOut<OutT>& out, int q) {
    const uint32_t dead = p.dead;
    const int lane = threadIdx.x & 31;
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (!idx_ok(static_cast<size_t>(s) * Cs + c, static_cast<size_t>(p.Q) * Cs, p.status)) return dead;
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
    if (ENUMERATE && threadIdx.x < 32) {  // warp 0 lists them for the bitmask pass
        int at = 0;
#pragma unroll
        for (int cb = 0; cb < 8; ++cb) {
            const int slot = at + __popc(lm[cb] & ((1u << lane) - 1u));
            if (((lm[cb] >> lane) & 1u) && idx_ok(slot, 256, p.status))
                ctx.cls[slot] = static_cast<uint8_t>(cb * 32 + lane);
            at += __popc(lm[cb]);
        }
        if (lane == 0) *ctx.ncls = n_live;
    }
    const int KB = two_level ? (C + 1 + 31) / 32 : 1;  // blocks of 32 second-level keys
    const int U = n_live * KB;
    while (true) {
        int j = 0;
        if (lane == 0) j = atomicAdd(&ctx.ctrs[0], 1);
        j = __shfl_sync(kFullWarp, j, 0);
        if (j >= U) break;
        const int li = j / KB, kb = j - li * KB;
        int c0 = 0, rem = li;  // the li-th readable class
#pragma unroll
        for (int cb = 0; cb < 8; ++cb) {
            const int pc = __popc(lm[cb]);
            if (rem >= 0 && rem < pc) {
                uint32_t m = lm[cb];
                for (int k = 0; k < rem; ++k) m &= m - 1;
                c0 = cb * 32 + __ffs(m) - 1;
                rem = -1;
            } else if (rem >= 0) {
                rem -= pc;
            }
        }
        const uint32_t s1 = lookup(q, c0);
        // lane = second-level key: bucket size, position and state after its bytes.  Key 0
        // holds the one-byte tokens, which the fill has covered.
        int cnt = 0, start = 0;
        uint32_t s2 = dead;
        if (two_level) {
            const int key2 = kb * 32 + lane;
            if (key2 >= 1 && key2 <= C && idx_ok(c0 * kKeyStride + key2, kKeys, p.status)) {
                cnt = __ldg(p.count2 + c0 * kKeyStride + key2);
                start = __ldg(p.start2 + c0 * kKeyStride + key2);
                s2 = lookup(s1, key2 - 1);
            }
        } else if (lane == 0 && idx_ok(c0, 256, p.status)) {
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
            if (lane == 0) base = atomicAdd(&ctx.ctrs[1], total);
            base = __shfl_sync(kFullWarp, base, 0);
            if (base + total > kRowDescCap) {
                if (lane == 0) ctx.ctrs[3] = 1;  // the row is walked without the list
                continue;
            }
            const int at = base + incl - nch;
            // long buckets are cut up by the whole warp, short ones by their lane
            uint32_t big = __ballot_sync(kFullWarp, nch > 4);
            while (big) {
                const int l = __ffs(big) - 1;
                big &= big - 1;
                const int b_at = __shfl_sync(kFullWarp, at, l);
                const int b_start = __shfl_sync(kFullWarp, start, l);
                const int b_cnt = __shfl_sync(kFullWarp, cnt, l);
                const uint32_t b_s = __shfl_sync(kFullWarp, s2, l);
                for (int k = lane; k * 32 < b_cnt; k += 32)
                    if (idx_ok(b_at + k, kRowDescCap, p.status))
                        ctx.descs[b_at + k] = Desc<TabT>::pack(b_start + 32 * k, b_s, min(32, b_cnt - 32 * k));
            }
            if (nch <= 4)
                for (int k = 0; k < nch; ++k)
                    if (idx_ok(at + k, kRowDescCap, p.status))
                        ctx.descs[at + k] = Desc<TabT>::pack(start + 32 * k, s2, min(32, cnt - 32 * k));
        } else {
            uint32_t m = __ballot_sync(kFullWarp, alive);
            while (m) {
                const int l = __ffs(m) - 1;
                m &= m - 1;
                const int bstart = __shfl_sync(kFullWarp, start, l);
                const int bn = __shfl_sync(kFullWarp, cnt, l);
                const uint32_t bs = __shfl_sync(kFullWarp, s2, l);
                for (int i0 = 0; i0 < bn; i0 += 32) {
                    const uint4 rec = chunk_fetch(p, bstart + i0, bn - i0, lane);
                    chunk_patch_level<TabT, OutT, HAS_OUT, FULL>(p, tab, Cs, two_level, out, rec, bs);
                }
            }
        }
    }
}

// Walks the chunks of the descriptor list; a warp takes two at a time and issues the loads
// of both before walking either.
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void walk_chunk_list(const WalkParams& p, const TabT* __restrict__ tab,
                                                uint32_t Cs, bool two_level, const RowCtx<TabT>& ctx,
                                                const RowOut<OutT>& out) {
    using D = Desc<TabT>;
    constexpr int kPull = 2;
    const int lane = threadIdx.x & 31;
    int total = ctx.ctrs[1];
    if (!idx_ok(total, kRowDescCap + 1, p.status)) total = 0;
    while (true) {
        int i = 0;
        if (lane == 0) i = atomicAdd(&ctx.ctrs[2], kPull);
        i = __shfl_sync(kFullWarp, i, 0);
        if (i >= total) break;
        typename D::type d[kPull];
        uint4 rec[kPull];
#pragma unroll
        for (int k = 0; k < kPull; ++k) {
            const bool have = i + k < total;
            d[k] = ctx.descs[have ? i + k : i];
            rec[k] = chunk_fetch(p, D::start(d[k]), have ? D::count(d[k]) : 0, lane);
        }
#pragma unroll
        for (int k = 0; k < kPull; ++k)
            if (i + k < total)
                chunk_patch_level<TabT, OutT, HAS_OUT, FULL>(p, tab, Cs, two_level, out, rec[k], D::state(d[k]));
    }
}

// ---------------------------------------------------------------------------------------
// The row's look-up table lut[c] = delta(q, class c) for c = 0 .. C (the null class C leads
// to dead).  Replicated form (C < kLutClasses): word (c, parity, lane) at byte
// c * 256 + parity * 128 + lane * 4.  Plain form: word c of the parity's 1,040-byte half.
template <typename TabT, bool FULL>
__device__ __forceinline__ void build_row_table(const TabT* __restrict__ tab, uint32_t Cs, int C,
                                                bool repl, uint32_t* lut, int par, int q) {
    auto lookup = [&](uint32_t c) -> uint32_t {
        return FULL ? tab[static_cast<uint32_t>(q) * Cs + c] : __ldg(tab + static_cast<size_t>(q) * Cs + c);
    };
    if (repl) {
        for (int i = threadIdx.x; i < (C + 1) * 32; i += kWalkThreads)
            lut[(i >> 5) * 64 + par * 32 + (i & 31)] = lookup(i >> 5);
    } else {
        for (int i = threadIdx.x; i <= C; i += kWalkThreads) lut[par * 260 + i] = lookup(i);
    }
}

// Look-up of byte k (0..3) of a word of four packed class ids.
template <bool REPL>
__device__ __forceinline__ uint32_t lut_get(const uint8_t* lut_base, uint32_t lane_off,
                                            uint32_t packed, int k, int32_t* status) {
    if (REPL) {
        // byte 0 = lane_off (parity * 128 + lane * 4), byte 1 = class id: c * 256 + lane_off
        const uint32_t off = __byte_perm(packed, lane_off, 0x5504u | (static_cast<uint32_t>(k) << 4));
        if (!idx_ok(off, kLutBytes - 3, status)) return 0;
        return *reinterpret_cast<const uint32_t*>(lut_base + off);
    }
    const uint32_t c = (packed >> (8 * k)) & 0xFFu;
    if (!idx_ok(lane_off + c * 4, kLutBytes - 3, status)) return 0;
    return *reinterpret_cast<const uint32_t*>(lut_base + lane_off + c * 4);
}

// Fills the next-state row from the table: thread = 32-byte output vector.
template <typename OutT, bool REPL>
__device__ __forceinline__ void fill_row(const WalkParams& p, const uint8_t* lut_base,
                                         uint32_t lane_off, OutT* nrow) {
    constexpr int EPV = 32 / sizeof(OutT);  // entries per vector: 8 or 16
    const uint8_t* c1 = p.tok_c1;
    int done = 0;
    if ((reinterpret_cast<uintptr_t>(nrow) & 31) == 0) {
        const int nvec = p.N / EPV;
        constexpr int kUnroll = 32 / EPV;  // class ids of this many vectors are fetched at once
        for (int j0 = threadIdx.x; j0 < nvec; j0 += kWalkThreads * kUnroll) {
            uint32_t cc[kUnroll][EPV / 4];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int j = j0 + u * kWalkThreads;
                if (j < nvec) {
                    if constexpr (EPV == 8) {
                        const uint2 v = __ldg(reinterpret_cast<const uint2*>(c1) + j);
                        cc[u][0] = v.x;
                        cc[u][1] = v.y;
                    } else {
                        const uint4 v = __ldg(reinterpret_cast<const uint4*>(c1) + j);
                        cc[u][0] = v.x;
                        cc[u][1] = v.y;
                        cc[u][2] = v.z;
                        cc[u][3] = v.w;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int j = j0 + u * kWalkThreads;
                if (j >= nvec) break;
                Vec32B o;
                if constexpr (EPV == 8) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) o.w[k] = lut_get<REPL>(lut_base, lane_off, cc[u][k >> 2], k & 3, p.status);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        const uint32_t lo = lut_get<REPL>(lut_base, lane_off, cc[u][(2 * k) >> 2], (2 * k) & 3, p.status);
                        const uint32_t hi = lut_get<REPL>(lut_base, lane_off, cc[u][(2 * k + 1) >> 2], (2 * k + 1) & 3, p.status);
                        o.w[k] = __byte_perm(lo, hi, 0x5410u);
                    }
                }
                stg_32B(reinterpret_cast<uint8_t*>(nrow) + static_cast<size_t>(j) * 32, o);
            }
        }
        done = nvec * EPV;
    }
    // ragged tail, or a row that is not 32-byte aligned: entry by entry, still coalesced
    for (int v = done + threadIdx.x; v < p.N; v += kWalkThreads) {
        const uint32_t off = lane_off + c1[v] * (REPL ? 256 : 4);
        if (idx_ok(off, kLutBytes - 3, p.status))
            nrow[v] = static_cast<OutT>(*reinterpret_cast<const uint32_t*>(lut_base + off));
    }
}

// Bitmask words of the one-byte tokens: OR of the bit planes of the classes q reads.
// Thread = four consecutive words.  (Bits of longer tokens are ORed in by the patches.)
// `cls` lists the classes q reads (`ncls` of them); four planes are fetched per round trip.
__device__ __forceinline__ void mask_row_from_planes(const WalkParams& p, const uint8_t* cls,
                                                     int ncls, uint32_t* mrow) {
    const int Gp = plane_stride(p.G);
    const bool vec_ok = (p.G & 3) == 0 && (reinterpret_cast<uintptr_t>(mrow) & 15) == 0;
    constexpr int kBatch = 4;
    for (int it = threadIdx.x; it * 4 < p.G; it += kWalkThreads) {
        uint4 acc = make_uint4(0, 0, 0, 0);
        const uint4* col = reinterpret_cast<const uint4*>(p.planes) + it;
        for (int j0 = 0; j0 < ncls; j0 += kBatch) {
            uint4 v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                v[u] = make_uint4(0, 0, 0, 0);
                if (j0 + u < ncls && idx_ok(j0 + u, 256, p.status))
                    v[u] = __ldg(col + static_cast<size_t>(cls[j0 + u]) * (Gp / 4));
            }
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                acc.x |= v[u].x;
                acc.y |= v[u].y;
                acc.z |= v[u].z;
                acc.w |= v[u].w;
            }
        }
        if (vec_ok) {
            reinterpret_cast<uint4*>(mrow)[it] = acc;
        } else {
            const int w = it * 4;
            mrow[w] = acc.x;
            if (w + 1 < p.G) mrow[w + 1] = acc.y;
            if (w + 2 < p.G) mrow[w + 2] = acc.z;
            if (w + 3 < p.G) mrow[w + 3] = acc.w;
        }
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
        __syncthreads();
    }
}

// Shared-memory bytes of walk_rows in front of the table.
template <typename TabT>
__host__ __device__ constexpr size_t rows_table_offset() {
    return (kLutBytes + 2 * kRowDescCap * sizeof(typename Desc<TabT>::type) + 127) / 128 * 128;
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk_rows(const WalkParams p, uint32_t table_cap) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ int32_t s_gstart[260];
    __shared__ int s_ctrs[8];  // two sets of row counters (see RowCtx::ctrs)
    __shared__ int s_next_row[2];
    __shared__ uint8_t s_cls[2][256];
    __shared__ int s_ncls[2];
    if (p.meta->any_bad != 0) {
        raw_rows<OutT, HAS_OUT>(p);
        return;
    }
    using D = Desc<TabT>;
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem_raw);
    typename D::type* descs = reinterpret_cast<typename D::type*>(smem_raw + kLutBytes);
    TabT* stab = reinterpret_cast<TabT*>(smem_raw + rows_table_offset<TabT>());

    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int C = p.meta->C;
    const uint32_t Cs = p.meta->Cs;
    const bool two_level = p.meta->two_level != 0;  // also: the replicated row table fits
    // (a bulk copy moves multiples of 16 bytes; the table's workspace has the slack)
    const uint64_t table_bytes = (static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT) + 15) / 16 * 16;
    const bool full = table_bytes <= table_cap;
    for (int i = threadIdx.x; i < 257; i += kWalkThreads) s_gstart[i] = p.gstart[i];
    if (threadIdx.x < 8) s_ctrs[threadIdx.x] = 0;
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
        if (ok && p.wait_probe > 0) ok = mbar_wait_bounded(&bar, 1, p.wait_probe);  // never completes
        if (!__syncthreads_and(ok)) {
            if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
            return;
        }
    } else {
        __syncthreads();
    }

    const int nrows = p.q_end - p.q_begin;
    const int lane = threadIdx.x & 31;
    auto ctx_of = [&](int par) {
        RowCtx<TabT> c;
        c.descs = descs + par * kRowDescCap;
        c.ctrs = s_ctrs + 4 * par;
        c.cls = s_cls[par];
        c.ncls = &s_ncls[par];
        return c;
    };
    // table and chunk list of a row (parity `par`); touches nothing the patch phase of the
    // row before reads
    auto prepare_row = [&](int row, int par) {
        const int q = p.q_begin + row;
        const RowCtx<TabT> ctx = ctx_of(par);
        const RowOut<OutT> none = {nullptr, nullptr};
        if (full) {
            if (HAS_OUT) build_row_table<TabT, true>(stab, Cs, C, two_level, lut, par, q);
            visit_buckets<TabT, OutT, HAS_OUT, true, true>(p, stab, C, Cs, two_level, s_gstart, ctx, none, q);
        } else {
            if (HAS_OUT) build_row_table<TabT, false>(gtab, Cs, C, two_level, lut, par, q);
            visit_buckets<TabT, OutT, HAS_OUT, false, true>(p, gtab, C, Cs, two_level, s_gstart, ctx, none, q);
        }
    };
    // Rows are taken in the order the preparation ranked them; position i of that order.
    // The CTA's first row has a fixed place; one thread draws the later ones, always one row
    // ahead (position and row number are on their way while a row is filled).
    auto row_at = [&](int i) {
        if (i >= nrows) return -1;
        const int r = p.row_order != nullptr ? __ldg(p.row_order + i) : i;
        return idx_ok(r, nrows, p.status) ? r : -1;
    };
    int par = 0;
    int row = row_at(blockIdx.x);
    int at_next = 0;  // thread 0: position of the next row
    if (threadIdx.x == 0) at_next = gridDim.x + atomicAdd(p.row_ctr, 1);
    if (row >= 0) prepare_row(row, par);
    __syncthreads();
    while (row >= 0) {
        const int q = p.q_begin + row;
        RowOut<OutT> out;
        out.nrow = HAS_OUT ? static_cast<OutT*>(p.next) + static_cast<size_t>(row) * p.N : nullptr;
        out.mrow = p.mask + static_cast<size_t>(row) * p.G;
        const RowCtx<TabT> ctx = ctx_of(par);
        int row_next = -1, at_after = 0;
        if (threadIdx.x == 0) {
            row_next = row_at(at_next);
            at_after = gridDim.x + atomicAdd(p.row_ctr, 1);
        }
        // ---- fill: every entry and every bitmask word of the row is written once
        mask_row_from_planes(p, ctx.cls, *ctx.ncls, out.mrow);
        if (HAS_OUT) {
            const uint8_t* lut_bytes = reinterpret_cast<const uint8_t*>(lut);
            if (two_level)
                fill_row<OutT, true>(p, lut_bytes, par * 128 + lane * 4, out.nrow);
            else
                fill_row<OutT, false>(p, lut_bytes, par * 1040, out.nrow);
        }
        if (threadIdx.x == 0) {  // next row and its counters, published by the barrier below
            s_next_row[par ^ 1] = row_next;
            for (int i = 0; i < 4; ++i) s_ctrs[4 * (par ^ 1) + i] = 0;
        }
        __syncthreads();  // the row is written: patches may land
        // ---- patch: survivors among the longer tokens, EOS
        if (ctx.ctrs[3] == 0) {
            if (full)
                walk_chunk_list<TabT, OutT, HAS_OUT, true>(p, stab, Cs, two_level, ctx, out);
            else
                walk_chunk_list<TabT, OutT, HAS_OUT, false>(p, gtab, Cs, two_level, ctx, out);
        } else {
            // more chunks than the list holds (a state that reads almost everything): walk
            // the buckets unit by unit instead
            if (threadIdx.x == 0) ctx.ctrs[0] = 0;
            __syncthreads();
            if (full)
                visit_buckets<TabT, OutT, HAS_OUT, true, false>(p, stab, C, Cs, two_level, s_gstart, ctx, out, q);
            else
                visit_buckets<TabT, OutT, HAS_OUT, false, false>(p, gtab, C, Cs, two_level, s_gstart, ctx, out, q);
        }
        if (threadIdx.x == 0 && p.eos_id >= 0 && q != p.dead && p.accept[q]) {
            if (HAS_OUT) out.nrow[p.eos_id] = static_cast<OutT>(q);
            atomicOr(out.mrow + (p.eos_id >> 5), 1u << (p.eos_id & 31));
        }
        // ---- the next row's table and chunk list (other parity)
        row = s_next_row[par ^ 1];
        if (row >= 0) prepare_row(row, par ^ 1);
        __syncthreads();
        par ^= 1;
        at_next = at_after;
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_rows(const WalkParams& p, int grid, cudaStream_t stream) {
    auto kernel = walk_rows<TabT, OutT, HAS_OUT>;
    const size_t table_off = rows_table_offset<TabT>();
    if (table_off + 1024 > p.smem_cap) return cudaErrorInvalidValue;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    // what is left after the row table and the chunk lists may hold the compressed table
    return launch_on(kernel, dim3(grid), dim3(kWalkThreads), p.smem_cap, stream, p,
                     static_cast<uint32_t>(p.smem_cap - table_off));
}

template <typename TabT>
cudaError_t launch_rows_for(const WalkParams& p, int grid, int32_t state_dtype, bool has_out,
                            cudaStream_t stream) {
    if (!has_out) return launch_rows<TabT, int32_t, false>(p, grid, stream);
    if (state_dtype == FSM_STATE_U16) return launch_rows<TabT, uint16_t, true>(p, grid, stream);
    return launch_rows<TabT, int32_t, true>(p, grid, stream);
}

// Smallest dynamic shared memory walk_rows can work with.
template <typename TabT>
constexpr size_t rows_min_smem() {
    return rows_table_offset<TabT>() + 4096;
}

}  // namespace
}  // namespace fsm
