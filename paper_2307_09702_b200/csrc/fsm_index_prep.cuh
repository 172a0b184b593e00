// Preparation kernels of the index build: byte classes, compressed table, token layouts.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

// ---------------------------------------------------------------------------- 1
// Thread (b, lane) owns byte column b of delta for rows lane, lane+4, ... of the block's
// share (coalesced 1 KB row reads).  The per-column hash is a wrap-around sum of mixed
// (row, value) pairs, so equal columns hash alike and partial sums simply add.  The
// blocks also clear the counters of the token sort.
constexpr int kHashRowLanes = 4;

__global__ void __launch_bounds__(256 * kHashRowLanes)
hash_columns(const int32_t* __restrict__ trans, int32_t Q, int32_t dead,
             uint64_t* __restrict__ partial, int weak, int32_t* __restrict__ gcount,
             int32_t* __restrict__ count2, int32_t* __restrict__ cursor2,
             int32_t* __restrict__ row_ctr, int32_t* status) {
    if (blockIdx.x == 0 && threadIdx.x == 0) *row_ctr = 0;
    __shared__ uint64_t part[kHashRowLanes][256];
    const int b = threadIdx.x & 255, rl = threadIdx.x >> 8;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < kKeys; i += gridDim.x * blockDim.x) {
        count2[i] = 0;
        cursor2[i] = 0;
        if (i < 256) gcount[i] = 0;
    }
    uint64_t h = 0;
    bool bad = false;
    for (int q = blockIdx.x * kHashRowLanes + rl; q < Q; q += gridDim.x * kHashRowLanes) {
        if (q == dead) continue;
        int32_t v = trans[static_cast<size_t>(q) * 256 + b];
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
// One block.  Bytes whose column hashes are equal form a class, represented by the
// smallest such byte; class ids are the ranks of the representatives.  Equal hashes
// are found through a small open-addressing table in shared memory.
__global__ void __launch_bounds__(256) derive_classes(const uint64_t* __restrict__ partial,
                                                     int nblocks, IndexMeta* meta, uint8_t* cls,
                                                     uint8_t* class_rep) {
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
        meta->two_level = (C <= kTwoLevelMaxC) ? 1 : 0;
    }
}

// ---------------------------------------------------------------------------- 3
// Blocks [0, row_blocks) compress and verify table rows and, for the bucket walk, note
// which classes each state reads (`live`); the remaining blocks write the class records of
// the tokens in token order (dense walk; the launch for the other walks has no such
// blocks).  Column C of the compressed table (the null class) and the padding columns lead
// to the dead state, as does the whole row of the dead state.
template <typename TabT>
__global__ void __launch_bounds__(256)
prepare_inputs(const int32_t* __restrict__ trans, const uint8_t* __restrict__ vocab_bytes,
               const int32_t* __restrict__ vocab_offsets, int64_t vocab_nbytes, int32_t Q,
               int32_t N, int32_t dead, int32_t eos_id, int row_blocks, IndexMeta* meta,
               const uint8_t* __restrict__ cls, const uint8_t* __restrict__ class_rep,
               TabT* __restrict__ table, uint4* __restrict__ tok_cls,
               uint8_t* __restrict__ tok_len, uint32_t* __restrict__ live, int32_t* status) {
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
            if (live != nullptr) {  // thread c: does q read class c?
                const int c = threadIdx.x;
                const bool reads = q != dead && c < C && row[s_rep[c < C ? c : 0]] != dead;
                const uint32_t m = __ballot_sync(kFullWarp, reads);
                if ((c & 31) == 0) live[static_cast<size_t>(q) * 8 + (c >> 5)] = m;
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
                uint8_t raw[kInlineBytes];
#pragma unroll
                for (int i = 0; i < kInlineBytes; ++i)  // independent loads, issued together
                    raw[i] = i < n ? vocab_bytes[o0 + i] : 0;
#pragma unroll
                for (int i = 0; i < kInlineBytes; ++i)
                    if (i < n) w[i >> 2] |= static_cast<uint32_t>(cls[raw[i]]) << ((i & 3) * 8);
            }
        }
        tok_cls[v] = make_uint4(w[0], w[1], w[2], w[3]);
        tok_len[v] = static_cast<uint8_t>(len);
    }
}

// ---------------------------------------------------------------------------- 3b
// Token order of the sparse walk: a counting sort by bucket key - the class of the
// first byte and, when there are at most kTwoLevelMaxC classes, the class of the second
// byte (key 0 = one-byte token).  scan_keys turns the counts into first positions
// (block c0 handles the keys of first class c0); count_keys / sort_tokens handle 1,024
// tokens per block.  A record keeps the length and the classes of bytes 1..15; `sid` holds the
// token id.
__global__ void __launch_bounds__(256)
scan_keys(const IndexMeta* __restrict__ meta, const int32_t* __restrict__ gcount,
          const int32_t* __restrict__ count2, int32_t* __restrict__ gstart,
          int32_t* __restrict__ start2) {
    __shared__ int gst[257];
    __shared__ int wsum[8];
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
    const int c0 = blockIdx.x;
    if (c0 == 0) {
        gstart[threadIdx.x] = gst[threadIdx.x];
        if (threadIdx.x == 0) gstart[256] = gst[256];
    }
    const int C = meta->C;
    if (meta->two_level == 0) {
        if (c0 == 0) start2[threadIdx.x] = gst[threadIdx.x];
        return;
    }
    if (c0 >= C) return;
    // exclusive prefix over the C + 1 <= 128 keys of first class c0
    const int t = threadIdx.x;
    const int mine = t <= C ? count2[c0 * kKeyStride + t] : 0;
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(kFullWarp, incl, off);
        if ((t & 31) >= off) incl += o;
    }
    if ((t & 31) == 31) wsum[t >> 5] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < (t >> 5); ++w) before += wsum[w];
    if (t <= C) start2[c0 * kKeyStride + t] = gst[c0] + before + incl - mine;
}

// Bucket keys are counted and ranked per block of kSortTokens tokens in shared memory
// (one counter per key), so that global memory sees one atomic per block and key instead
// of one per token: tokens that start with a space are a third of a BPE vocabulary and
// would otherwise all hit the same few counters.
constexpr int kSortThreads = 1024;
constexpr int kSortTokens = kSortThreads;

__global__ void __launch_bounds__(kSortThreads)
count_keys(const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
           int64_t vocab_nbytes, int32_t N, int32_t eos_id, const IndexMeta* __restrict__ meta,
           const uint8_t* __restrict__ cls, int32_t* __restrict__ gcount,
           int32_t* __restrict__ count2, uint32_t* __restrict__ planes, int32_t* status) {
    extern __shared__ int s_cnt[];  // [kKeys]
    __shared__ int hist[256];
    __shared__ uint8_t s_cls[256];
    if (threadIdx.x < 256) {
        hist[threadIdx.x] = 0;
        s_cls[threadIdx.x] = cls[threadIdx.x];
    }
    const bool two = meta->two_level != 0;
    const int nkeys = two ? kKeys : 256;
    for (int i = threadIdx.x; i < nkeys; i += kSortThreads) s_cnt[i] = 0;
    // bucket walk: plane c holds the bits of the one-byte tokens of class c; the block owns
    // 32 words of every plane and clears them first
    const int W = (N + 31) / 32;
    if (planes != nullptr) {
        const int C = meta->C;
        for (int i = threadIdx.x; i < C * 32; i += kSortThreads) {
            const int word = blockIdx.x * 32 + (i & 31);
            if (word < W) planes[static_cast<size_t>(i >> 5) * W + word] = 0;
        }
    }
    __syncthreads();
    bool bad = false;
    const int64_t v = static_cast<int64_t>(blockIdx.x) * kSortTokens + threadIdx.x;
    const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
    if (t.len > 0) {
        atomicAdd(&hist[t.first], 1);
        atomicAdd(&s_cnt[bucket_key(two, t.first, t.second_key)], 1);
    }
    if (planes != nullptr) {
        const bool one = t.len == 1;
        const uint32_t peers = __match_any_sync(kFullWarp, one ? t.first : 0xFFFF);
        if (one && (threadIdx.x & 31) == __ffs(peers) - 1)
            planes[static_cast<size_t>(t.first) * W + (v >> 5)] = peers;
    }
    if (__syncthreads_or(bad) && threadIdx.x == 0) raise_flag(status, FSM_FLAG_OFFSETS);
    for (int i = threadIdx.x; i < nkeys; i += kSortThreads)
        if (s_cnt[i] > 0) atomicAdd(&count2[i], s_cnt[i]);
    if (threadIdx.x < 256 && hist[threadIdx.x] > 0) atomicAdd(&gcount[threadIdx.x], hist[threadIdx.x]);
}

__global__ void __launch_bounds__(kSortThreads)
sort_tokens(const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
            int64_t vocab_nbytes, int32_t N, int32_t eos_id, const IndexMeta* __restrict__ meta,
            const uint8_t* __restrict__ cls, const int32_t* __restrict__ start2,
            int32_t* __restrict__ cursor2, uint4* __restrict__ srec, int32_t* __restrict__ sid) {
    extern __shared__ int s_cnt[];  // [kKeys] count, then the block's base position per key
    __shared__ uint8_t s_cls[256];
    if (threadIdx.x < 256) s_cls[threadIdx.x] = cls[threadIdx.x];
    const bool two = meta->two_level != 0;
    const int nkeys = two ? kKeys : 256;
    for (int i = threadIdx.x; i < nkeys; i += kSortThreads) s_cnt[i] = 0;
    __syncthreads();
    bool bad = false;
    const int64_t v = static_cast<int64_t>(blockIdx.x) * kSortTokens + threadIdx.x;
    const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
    const int key = t.len > 0 ? bucket_key(two, t.first, t.second_key) : 0;
    int rank = 0;
    if (t.len > 0) rank = atomicAdd(&s_cnt[key], 1);
    __syncthreads();
    // one global atomic per key present in the block reserves its positions
    for (int i = threadIdx.x; i < nkeys; i += kSortThreads) {
        const int c = s_cnt[i];
        if (c > 0) s_cnt[i] = start2[i] + atomicAdd(&cursor2[i], c);
    }
    __syncthreads();
    if (t.len > 0) {
        const int pos = s_cnt[key] + rank;
        uint32_t w[4] = {static_cast<uint32_t>(t.len), 0, 0, 0};
        const int nb = min(t.len, kInlineBytes);
        uint8_t raw[kInlineBytes];
#pragma unroll
        for (int i = 1; i < kInlineBytes; ++i)  // independent loads, issued together
            raw[i] = i < nb ? vocab_bytes[t.start + i] : 0;
#pragma unroll
        for (int i = 1; i < kInlineBytes; ++i)
            if (i < nb) w[i >> 2] |= static_cast<uint32_t>(s_cls[raw[i]]) << ((i & 3) * 8);
        srec[pos] = make_uint4(w[0], w[1], w[2], w[3]);
        sid[pos] = static_cast<int32_t>(v);
    }
}

}  // namespace
}  // namespace fsm
