// Preparation of the index build: byte classes, compressed table, token layouts.
//
// One cooperative launch (one block per SM, all resident) in three phases separated by grid
// barriers: hash_phase (a hash of each byte column of delta), prepare_phase (every block
// derives the byte classes from the hashes, then the blocks share the table rows and the
// tokens) and, for the work-avoiding walks, sort_phase (every block scans the key counts,
// then the blocks share the tokens).  The small serial steps are repeated by every block
// instead of being phases of their own.
#pragma once

#include <cooperative_groups.h>

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

// ---------------------------------------------------------------------------- 1
// Thread (b, lane) owns byte column b of delta for rows lane, lane+4, ... of the block's
// share (coalesced 1 KB row reads).  The per-column hash is a wrap-around sum of mixed
// (row, value) pairs, so equal columns hash alike and partial sums simply add.  The
// blocks also clear the counters of the token sort and the flag of the class check.
constexpr int kHashRowLanes = 4;

// (`nparts` blocks hash; every block helps clear the counters.)
__device__ __forceinline__ void hash_phase(const int32_t* __restrict__ trans, int32_t Q, int32_t dead,
                                           uint64_t* __restrict__ partial, int nparts, int weak,
                                           IndexMeta* meta, int32_t* __restrict__ count2,
                                           int32_t* __restrict__ cursor2, int32_t* __restrict__ row_ctr,
                                           int32_t* status) {
    __shared__ uint64_t part[kHashRowLanes][256];
    const int b = threadIdx.x & 255, rl = threadIdx.x >> 8;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *row_ctr = 0;
        meta->any_bad = 0;
    }
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < kKeys; i += gridDim.x * blockDim.x) {
        count2[i] = 0;
        cursor2[i] = 0;
    }
    if (static_cast<int>(blockIdx.x) >= nparts) return;
    uint64_t h = 0;
    bool bad = false;
#pragma unroll 4
    for (int q = blockIdx.x * kHashRowLanes + rl; q < Q; q += nparts * kHashRowLanes) {
        const int32_t v = trans[static_cast<size_t>(q) * 256 + b];
        if (q == dead) continue;
        bad |= static_cast<uint32_t>(v) >= static_cast<uint32_t>(Q);
        h += mix64((static_cast<uint64_t>(q) << 32) | static_cast<uint32_t>(v));
    }
    part[rl][b] = h;
    const int any_bad = __syncthreads_or(bad);
    if (rl == 0) {
        uint64_t sum = 0;
#pragma unroll
        for (int k = 0; k < kHashRowLanes; ++k) sum += part[k][b];
        partial[blockIdx.x * 256 + b] = weak ? 0 : sum;
    }
    if (any_bad && threadIdx.x == 0) raise_flag(status, FSM_FLAG_TRANS_RANGE);
}

// ---------------------------------------------------------------------------- 2
constexpr int kPrepThreads = 1024;
constexpr int kPrepRows = kPrepThreads / 256;  // table rows handled per pass
constexpr int kPrepTokens = kPrepThreads;      // tokens handled per pass

// Byte classes from the column hashes, computed by the first 256 threads of a block
// (thread = byte) into shared memory.  Bytes whose hashes are equal form a class,
// represented by the smallest such byte; class ids are the ranks of the representatives.
// Equal hashes are found through a small open-addressing table.  Returns the number of
// classes; ends with a barrier.
struct ClassScratch {
    unsigned long long keys[1024];
    int min_byte[1024];
    uint32_t rep_bits[8];
};

__device__ __forceinline__ int derive_classes(const uint64_t* partial, int nparts,
                                              ClassScratch& cs, uint8_t* s_cls, uint8_t* s_rep) {
    constexpr int kSlots = 1024;
    constexpr unsigned long long kEmpty = ~0ull;
    const int b = threadIdx.x;
    for (int i = b; i < kSlots; i += blockDim.x) {
        cs.keys[i] = kEmpty;
        cs.min_byte[i] = 256;
    }
    __syncthreads();
    int slot = 0;
    if (b < 256) {
        uint64_t sum = 0;
#pragma unroll 8
        for (int k = 0; k < nparts; ++k) sum += partial[k * 256 + b];
        // kEmpty marks a free slot; folding that one value onto its neighbour can only
        // merge two classes, which the exact verification of the table rows would catch.
        const unsigned long long key = (sum == kEmpty) ? sum - 1 : sum;
        // at most 256 distinct keys in 1024 slots: linear probing ends within kSlots steps
        slot = static_cast<int>((key ^ (key >> 29)) & (kSlots - 1));
        for (int probe = 0; probe < kSlots; ++probe) {
            const unsigned long long was = atomicCAS(&cs.keys[slot], kEmpty, key);
            if (was == kEmpty || was == key) break;
            slot = (slot + 1) & (kSlots - 1);
        }
        atomicMin(&cs.min_byte[slot], b);
    }
    __syncthreads();
    int r = 0;
    if (b < 256) {  // warps 0..7, whole warps
        r = cs.min_byte[slot];
        const uint32_t m = __ballot_sync(kFullWarp, r == b);
        if ((b & 31) == 0) cs.rep_bits[b >> 5] = m;
    }
    __syncthreads();
    int C = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) C += __popc(cs.rep_bits[w]);
    if (b < 256) {
        int id = __popc(cs.rep_bits[r >> 5] & ((1u << (r & 31)) - 1u));
        for (int w = 0; w < (r >> 5); ++w) id += __popc(cs.rep_bits[w]);
        s_cls[b] = static_cast<uint8_t>(id);
        if (r == b) s_rep[id] = static_cast<uint8_t>(b);
    }
    __syncthreads();
    return C;
}

// Every block derives the classes; block 0 publishes them.  Then the blocks share
//   - the table rows: compressed row [Cs] with exact verification that every byte's column
//     equals its class representative's column, and (bucket walk) the classes the state
//     reads.  Column C (the null class) and the padding columns lead to the dead state, as
//     does the whole row of the dead state;
//   - the tokens: class records in token order (dense walk), or the counts of the bucket
//     keys (work-avoiding walks: class of the first byte and, with at most kTwoLevelMaxC
//     classes, class of the second byte; key 0 = one-byte token) and (bucket walk) the bit
//     planes of the one-byte tokens.  Keys are counted in shared memory over all tokens
//     of the block, so that global memory sees one atomic per block and key: tokens that
//     start with a space are a third of a BPE vocabulary and would otherwise all hit the
//     same few counters.
template <typename TabT>
__device__ __forceinline__ void prepare_phase(
    const int32_t* __restrict__ trans, const uint8_t* __restrict__ vocab_bytes,
    const int32_t* __restrict__ vocab_offsets, int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead,
    int32_t eos_id, const uint64_t* partial, int nparts, IndexMeta* meta, uint8_t* __restrict__ cls_out,
    TabT* __restrict__ table, uint4* __restrict__ tok_cls, uint8_t* __restrict__ tok_len,
    uint32_t* __restrict__ live, int32_t* __restrict__ count2, uint32_t* __restrict__ planes,
    uint16_t* __restrict__ tok_head, uint8_t* __restrict__ tok_c1, int32_t* status,
    int* s_cnt /* [kKeys] when keys are counted */, int32_t row_first, const TokenRaw& raw_first,
    bool bad_tok) {
    __shared__ ClassScratch cs;
    __shared__ uint8_t s_cls[256], s_rep[256];
    __shared__ int32_t rows[kPrepRows][256];
    const int tid = threadIdx.x;
    const int C = derive_classes(partial, nparts, cs, s_cls, s_rep);
    const int Cs = table_row_stride<TabT>(C);
    const bool two = C <= kTwoLevelMaxC;
    if (blockIdx.x == 0) {
        if (tid < 256) cls_out[tid] = s_cls[tid];
        if (tid == 0) {
            meta->C = C;
            meta->Cs = Cs;
            meta->two_level = two ? 1 : 0;
            // 256 distinct columns leave no byte value for the null class: such a table
            // is walked uncompressed.
            if (C > 255) atomicExch(&meta->any_bad, 1);
        }
    }
    // ---- table rows, kPrepRows at a time (thread = (row lane, byte))
    {
        const int rl = tid >> 8, b = tid & 255;
        bool bad = false;
        for (int q0 = blockIdx.x * kPrepRows; q0 < Q; q0 += gridDim.x * kPrepRows) {
            const int q = q0 + rl;
            __syncthreads();
            if (q < Q) {
                const int32_t v = q0 == static_cast<int>(blockIdx.x) * kPrepRows
                                      ? row_first
                                      : trans[static_cast<size_t>(q) * 256 + b];
                rows[rl][b] = clamp_state(v, Q, dead);
            }
            __syncthreads();
            if (q < Q) {
                if (q != dead) bad |= rows[rl][b] != rows[rl][s_rep[s_cls[b]]];
                for (int c = b; c < Cs; c += 256) {
                    const int32_t v = (q == dead || c >= C) ? dead : rows[rl][s_rep[c]];
                    table[static_cast<size_t>(q) * Cs + c] = static_cast<TabT>(v);
                }
            }
            if (live != nullptr) {  // thread (rl, c): does q read class c?
                const bool reads = q < Q && q != dead && b < C && rows[rl][s_rep[b < C ? b : 0]] != dead;
                const uint32_t m = __ballot_sync(kFullWarp, reads);
                if ((b & 31) == 0 && q < Q) live[static_cast<size_t>(q) * 8 + (b >> 5)] = m;
            }
        }
        if (__syncthreads_or(bad) && tid == 0) {
            atomicExch(&meta->any_bad, 1);
            raise_flag(status, FSM_FLAG_CLASS_SPLIT);
        }
    }
    // ---- tokens in token order: class records of the dense walk
    if (tok_cls != nullptr) {
        const int64_t slots = (static_cast<int64_t>(N) + 31) / 32 * 32;
        for (int64_t v = static_cast<int64_t>(blockIdx.x) * kPrepTokens + tid; v < slots;
             v += static_cast<int64_t>(gridDim.x) * kPrepTokens) {
            uint32_t w[4] = {static_cast<uint32_t>(C), 0, 0, 0};  // an empty token reads the null class
            int len = 0;
            uint32_t first_byte = 0;
            if (v < N && v != eos_id) {
                const int64_t o0 = vocab_offsets[v], o1 = vocab_offsets[v + 1];
                if (o0 < 0 || o1 < o0 || o1 > vocab_nbytes) {
                    raise_flag(status, FSM_FLAG_OFFSETS);
                } else {
                    len = static_cast<int>(min(o1 - o0, static_cast<int64_t>(kInlineBytes + 1)));
                    const int n = min(len, kInlineBytes);
                    if (n > 0) w[0] = 0;
                    uint8_t raw[kInlineBytes];
#pragma unroll
                    for (int i = 0; i < kInlineBytes; ++i)  // independent loads, issued together
                        raw[i] = i < n ? vocab_bytes[o0 + i] : 0;
                    first_byte = raw[0];
#pragma unroll
                    for (int i = 0; i < kInlineBytes; ++i)
                        if (i < n) w[i >> 2] |= static_cast<uint32_t>(s_cls[raw[i]]) << ((i & 3) * 8);
                }
            }
            tok_cls[v] = make_uint4(w[0], w[1], w[2], w[3]);
            tok_len[v] = static_cast<uint8_t>(len);
            if (tok_head != nullptr && v < N)  // first byte and length, for the compressed rows
                tok_head[v] = static_cast<uint16_t>(first_byte | (static_cast<uint32_t>(len) << 8));
        }
    }
    // ---- bucket keys of the tokens, kPrepTokens at a time
    const int nchunks = (N + kPrepTokens - 1) / kPrepTokens;
    if (count2 != nullptr && static_cast<int>(blockIdx.x) < nchunks) {
        const int nkeys = two ? kKeys : 256;
        const int W = (N + 31) / 32, Wp = plane_stride(W);
        for (int i = tid; i < nkeys; i += kPrepThreads) s_cnt[i] = 0;
        bool bad = bad_tok;
        for (int chunk = blockIdx.x; chunk < nchunks; chunk += gridDim.x) {
            // bucket walk: plane c holds the bits of the one-byte tokens of class c; the
            // 32 words of this pass are cleared first
            if (planes != nullptr)
                for (int i = tid; i < C * 32; i += kPrepThreads) {
                    const int word = chunk * 32 + (i & 31);
                    if (word < Wp) planes[static_cast<size_t>(i >> 5) * Wp + word] = 0;
                }
            __syncthreads();
            const int64_t v = static_cast<int64_t>(chunk) * kPrepTokens + tid;
            const TokenRaw raw = chunk == static_cast<int>(blockIdx.x)
                                     ? raw_first
                                     : token_raw(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, v, &bad);
            const TokenInfo t = token_classify(raw, s_cls);
            if (tok_head != nullptr && v < N)  // first byte and length, for the compressed rows
                tok_head[v] = static_cast<uint16_t>(raw.b0 | (static_cast<uint32_t>(raw.len) << 8));
            if (tok_c1 != nullptr)  // (the array is padded to whole passes)
                tok_c1[v] = static_cast<uint8_t>(t.len == 1 ? t.first : C);
            const int key = bucket_key(two, t.first, t.second_key);
            if (t.len > 0 && idx_ok(key, nkeys, status)) atomicAdd(&s_cnt[key], 1);
            if (planes != nullptr) {
                const bool one = t.len == 1;
                const uint32_t peers = __match_any_sync(kFullWarp, one ? t.first : 0xFFFF);
                if (one && (tid & 31) == __ffs(peers) - 1 && idx_ok(t.first, C, status) && idx_ok(v >> 5, Wp, status))
                    planes[static_cast<size_t>(t.first) * Wp + (v >> 5)] = peers;
            }
        }
        if (__syncthreads_or(bad) && tid == 0) raise_flag(status, FSM_FLAG_OFFSETS);
        for (int i = tid; i < nkeys; i += kPrepThreads)
            if (s_cnt[i] > 0) atomicAdd(&count2[i], s_cnt[i]);
    }
}

// ---------------------------------------------------------------------------- 3
// Token order of the work-avoiding walks: a counting sort by bucket key.  Keys are
// numbered first class major, so the exclusive prefix sum of the key counts is the first
// sorted position of every key; every block computes it in shared memory (block 0
// publishes it, and the first position of every first class, for the walk).  Then the
// blocks share the tokens, kPrepTokens at a time: rank within the pass by shared-memory
// counters, one global atomic per key present in the pass to reserve its positions.  A
// record keeps the length (capped at kSortedInline + 1), the classes of bytes
// 1 .. kSortedInline - 1 and, in its last word, the token id.
constexpr int kScanPer = (kKeys + kPrepThreads - 1) / kPrepThreads;  // keys per thread
constexpr int kKeysPad = kScanPer * kPrepThreads;
constexpr int kOrderBuckets = 2048;  // candidate-count buckets of the row order

__device__ __forceinline__ void sort_phase(
    const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
    int64_t vocab_nbytes, int32_t N, int32_t eos_id, const IndexMeta* meta, const uint8_t* cls,
    const int32_t* count2, int32_t* cursor2, int32_t* __restrict__ start2, int32_t* __restrict__ gstart,
    uint4* __restrict__ srec, const uint32_t* live, int32_t q_begin, int32_t q_end, int32_t* row_order,
    int32_t* win_order, int* s_sort /* s_start[kKeysPad], s_cnt[kKeys] */, const TokenRaw& raw_first,
    const uint8_t (&bytes_first)[kSortedInline], int32_t* status) {
    int* s_start = s_sort;
    int* s_cnt = s_sort + kKeysPad;
    __shared__ int wsum[kPrepThreads / 32];
    __shared__ uint8_t s_cls[256];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 256) s_cls[tid] = cls[tid];
    const bool two = meta->two_level != 0;
    const int nkeys = two ? kKeys : 256;
#pragma unroll
    for (int j = 0; j < kScanPer; ++j) {
        const int i = tid + j * kPrepThreads;
        s_start[i] = i < nkeys ? count2[i] : 0;
    }
    __syncthreads();
    // exclusive prefix sum: kScanPer consecutive keys per thread
    int local[kScanPer], sum = 0;
#pragma unroll
    for (int j = 0; j < kScanPer; ++j) {
        local[j] = sum;
        sum += s_start[tid * kScanPer + j];
    }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(kFullWarp, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) wsum[warp] = incl;
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < kPrepThreads / 32; ++w) {
        if (w < warp) before += wsum[w];
        total += wsum[w];
    }
#pragma unroll
    for (int j = 0; j < kScanPer; ++j) s_start[tid * kScanPer + j] = before + incl - sum + local[j];
    __syncthreads();
    // With a row order asked for, the last block of the grid sorts no tokens: it ranks the
    // states by the number of tokens that start with a byte they read (the candidates the
    // row-wise walk has to look at, between none and most of the vocabulary), largest first.
    // Rows handed out in that order leave the CTAs of the walk finishing together; in
    // index order a CTA that draws a long row last keeps the kernel waiting.
    const bool ordering = row_order != nullptr || win_order != nullptr;
    const int sort_grid = static_cast<int>(gridDim.x) - (ordering ? 1 : 0);
    if (win_order != nullptr && static_cast<int>(blockIdx.x) == sort_grid) {
        // The same for the bucket walk: a window of 32 sorted tokens costs one scan of the
        // states per (first class, second class) key in it, so the windows are ranked by the
        // number of buckets of longer tokens that begin in them (0 to 32), most first; the
        // bucket that reaches in from the window before is one more in nearly every window
        // and is left out.  (Host: win_order only when the windows fit s_cnt.)
        const int nwin = (total + 31) >> 5;
        for (int i = tid; i < nwin; i += kPrepThreads) s_cnt[i] = 0;
        __shared__ int s_hist[40];
        if (tid < 40) s_hist[tid] = 0;
        __syncthreads();
        if (two) {
            for (int key = tid; key < kKeys; key += kPrepThreads) {
                const int st = s_start[key], en = s_start[key + 1];
                if (en > st && key % kKeyStride != 0 && idx_ok(st >> 5, nwin, status)) atomicAdd(&s_cnt[st >> 5], 1);
            }
        }
        __syncthreads();
        // counting sort by that number, descending: the lanes of a warp that hold the same
        // number find each other and reserve their places with one atomic
        const int rounds = (nwin + kPrepThreads - 1) / kPrepThreads;
        for (int pass = 0; pass < 2; ++pass) {
            for (int it = 0; it < rounds; ++it) {
                const int w = it * kPrepThreads + tid;
                const int b = w < nwin ? 32 - min(s_cnt[w], 32) : 33;
                const uint32_t m = __match_any_sync(kFullWarp, b);
                const int leader = __ffs(m) - 1;
                int base = 0;
                if (lane == leader) base = atomicAdd(&s_hist[b], __popc(m));
                base = __shfl_sync(kFullWarp, base, leader);
                const int at = base + __popc(m & ((1u << lane) - 1));
                if (pass == 1 && w < nwin && idx_ok(at, nwin, status)) win_order[at] = w;
            }
            __syncthreads();
            if (pass == 0 && tid == 0) {  // counts -> first positions
                int run = 0;
                for (int v = 0; v <= 33; ++v) {
                    const int c = s_hist[v];
                    s_hist[v] = run;
                    run += c;
                }
            }
            __syncthreads();
        }
        return;
    }
    if (row_order != nullptr && static_cast<int>(blockIdx.x) == sort_grid) {
        __shared__ int s_group[256];  // tokens per first-byte class
        if (tid < 256) {
            const int stride = two ? kKeyStride : 1, groups = two ? kKeyStride : 256;
            const int g0 = tid < groups ? s_start[tid * stride] : total;
            const int g1 = tid + 1 < groups ? s_start[(tid + 1) * stride] : total;
            s_group[tid] = g1 - g0;
        }
        for (int i = tid; i < kOrderBuckets; i += kPrepThreads) s_cnt[i] = 0;
        __syncthreads();
        const int nrows = q_end - q_begin;
        auto bucket_of = [&](int r) {  // bucket 0 holds the heaviest rows
            const uint32_t* lv = live + static_cast<size_t>(q_begin + r) * 8;
            int64_t candidates = 0;
            for (int w = 0; w < 8; ++w) {
                uint32_t m = lv[w];
                while (m) {
                    candidates += s_group[w * 32 + __ffs(m) - 1];
                    m &= m - 1;
                }
            }
            const int64_t b = candidates * kOrderBuckets / (static_cast<int64_t>(N) + 1);
            return kOrderBuckets - 1 - static_cast<int>(b < kOrderBuckets - 1 ? b : kOrderBuckets - 1);
        };
        for (int r = tid; r < nrows; r += kPrepThreads) atomicAdd(&s_cnt[bucket_of(r)], 1);
        __syncthreads();
        static_assert(kOrderBuckets == 2 * kPrepThreads, "two buckets per thread");
        const int a0 = s_cnt[2 * tid], a1 = s_cnt[2 * tid + 1];
        int inc2 = a0 + a1;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullWarp, inc2, off);
            if (lane >= off) inc2 += o;
        }
        __syncthreads();  // wsum is read by every thread above
        if (lane == 31) wsum[warp] = inc2;
        __syncthreads();
        int front = 0;
        for (int w = 0; w < warp; ++w) front += wsum[w];
        s_cnt[2 * tid] = front + inc2 - a0 - a1;
        s_cnt[2 * tid + 1] = front + inc2 - a1;
        __syncthreads();
        for (int r = tid; r < nrows; r += kPrepThreads) {
            const int at = atomicAdd(&s_cnt[bucket_of(r)], 1);
            if (idx_ok(at, nrows, status)) row_order[at] = r;
        }
        return;
    }
    if (blockIdx.x == 0) {
        for (int i = tid; i < nkeys; i += kPrepThreads) start2[i] = s_start[i];
        if (tid <= 256) {
            int g = total;
            if (two) {
                if (tid < kKeyStride) g = s_start[tid * kKeyStride];
            } else if (tid < 256) {
                g = s_start[tid];
            }
            gstart[tid] = g;
        }
    }
    const int nchunks = (N + kPrepTokens - 1) / kPrepTokens;
    for (int chunk = blockIdx.x; chunk < nchunks; chunk += sort_grid) {
        __syncthreads();  // the previous pass is done with s_cnt
        for (int i = tid; i < nkeys; i += kPrepThreads) s_cnt[i] = 0;
        __syncthreads();
        bool bad = false;
        const int64_t v = static_cast<int64_t>(chunk) * kPrepTokens + tid;
        const bool first = chunk == static_cast<int>(blockIdx.x);
        const TokenRaw raw = first ? raw_first
                                   : token_raw(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, v, &bad);
        const TokenInfo t = token_classify(raw, s_cls);
        const int key = t.len > 0 ? bucket_key(two, t.first, t.second_key) : 0;
        int rank = 0;
        const bool placed = t.len > 0 && idx_ok(key, nkeys, status);
        if (placed) rank = atomicAdd(&s_cnt[key], 1);
        uint8_t bytes[kSortedInline];
#pragma unroll
        for (int i = 1; i < kSortedInline; ++i) {  // independent loads, issued together
            if (first)
                bytes[i] = bytes_first[i];
            else
                bytes[i] = i < t.len ? vocab_bytes[t.start + i] : 0;
        }
        __syncthreads();
        // one global atomic per key present in the pass reserves its positions; a thread
        // issues all of its atomics before it uses the first result
        {
            int cnt[kScanPer], base[kScanPer];
#pragma unroll
            for (int j = 0; j < kScanPer; ++j) {
                const int i = tid + j * kPrepThreads;
                cnt[j] = i < nkeys ? s_cnt[i] : 0;
            }
#pragma unroll
            for (int j = 0; j < kScanPer; ++j) {
                base[j] = 0;
                if (cnt[j] > 0) base[j] = atomicAdd(&cursor2[tid + j * kPrepThreads], cnt[j]);
            }
#pragma unroll
            for (int j = 0; j < kScanPer; ++j) {
                const int i = tid + j * kPrepThreads;
                if (cnt[j] > 0) s_cnt[i] = s_start[i] + base[j];
            }
        }
        __syncthreads();
        if (placed && idx_ok(s_cnt[key] + rank, N, status)) {
            const int pos = s_cnt[key] + rank;
            uint32_t w[3] = {static_cast<uint32_t>(min(t.len, kSortedInline + 1)), 0, 0};
            const int nb = min(t.len, kSortedInline);
#pragma unroll
            for (int i = 1; i < kSortedInline; ++i)
                if (i < nb) w[i >> 2] |= static_cast<uint32_t>(s_cls[bytes[i]]) << ((i & 3) * 8);
            srec[pos] = make_uint4(w[0], w[1], w[2], static_cast<uint32_t>(v));
        }
    }
}

// ---------------------------------------------------------------------------- fused
// The whole preparation as one cooperative kernel (one block per SM).  The blocks fetch
// what depends on the build's inputs only (their first table rows, their first tokens)
// before the first grid barrier.
struct PrepParams {
    const int32_t* trans;
    const uint8_t* vocab_bytes;
    const int32_t* vocab_offsets;
    int64_t vocab_nbytes;
    int32_t Q, N, dead, eos_id, q_begin, q_end;
    int nparts;  // blocks that hash table rows
    int weak;
    int sorted;  // tokens are sorted by bucket key (work-avoiding walks)
    uint64_t* partial;
    IndexMeta* meta;
    uint8_t* cls;
    void* table;
    uint4* tok_cls;
    uint8_t* tok_len;
    uint32_t* live;
    int32_t* count2;
    int32_t* cursor2;
    int32_t* start2;
    int32_t* gstart;
    int32_t* row_ctr;
    uint32_t* planes;
    uint16_t* tok_head;
    uint8_t* tok_c1;
    uint4* srec;
    int32_t* row_order;
    int32_t* win_order;
    int32_t* status;
};

template <typename TabT>
__global__ void __launch_bounds__(kPrepThreads, 1) prepare_fused(const PrepParams a) {
    extern __shared__ int s_dyn[];  // key counters (prepare), scan + counters (sort)
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    const int tid = threadIdx.x;
    // ---- inputs of the build, fetched before anything else is known
    int32_t row_first = a.dead;
    if (static_cast<int>(blockIdx.x) * kPrepRows + (tid >> 8) < a.Q)
        row_first = a.trans[(static_cast<size_t>(blockIdx.x) * kPrepRows + (tid >> 8)) * 256 + (tid & 255)];
    bool bad_tok = false;
    TokenRaw raw_first = {0, 0, 0, 0};
    uint8_t bytes_first[kSortedInline];
#pragma unroll
    for (int i = 0; i < kSortedInline; ++i) bytes_first[i] = 0;
    if (a.sorted) {
        raw_first = token_raw(a.vocab_bytes, a.vocab_offsets, a.vocab_nbytes, a.N, a.eos_id,
                              static_cast<int64_t>(blockIdx.x) * kPrepTokens + tid, &bad_tok);
#pragma unroll
        for (int i = 2; i < kSortedInline; ++i)
            bytes_first[i] = i < raw_first.len ? a.vocab_bytes[raw_first.start + i] : 0;
        bytes_first[0] = static_cast<uint8_t>(raw_first.b0);
        bytes_first[1] = static_cast<uint8_t>(raw_first.b1);
    }
    hash_phase(a.trans, a.Q, a.dead, a.partial, a.nparts, a.weak, a.meta, a.count2, a.cursor2, a.row_ctr,
               a.status);
    grid.sync();
    prepare_phase<TabT>(a.trans, a.vocab_bytes, a.vocab_offsets, a.vocab_nbytes, a.Q, a.N, a.dead, a.eos_id,
                        a.partial, a.nparts, a.meta, a.cls, static_cast<TabT*>(a.table),
                        a.sorted ? nullptr : a.tok_cls, a.tok_len, a.live, a.sorted ? a.count2 : nullptr,
                        a.planes, a.tok_head, a.tok_c1, a.status, s_dyn, row_first, raw_first, bad_tok);
    if (!a.sorted) return;
    grid.sync();
    sort_phase(a.vocab_bytes, a.vocab_offsets, a.vocab_nbytes, a.N, a.eos_id, a.meta, a.cls, a.count2,
               a.cursor2, a.start2, a.gstart, a.srec, a.live, a.q_begin, a.q_end, a.row_order, a.win_order,
               s_dyn, raw_first, bytes_first, a.status);
}

}  // namespace
}  // namespace fsm
