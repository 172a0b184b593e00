// Preparation kernels of the index build: byte classes, compressed table, token layouts.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

// ---------------------------------------------------------------------------- 1
// Thread b owns byte column b of delta; a block strides over rows (coalesced 1 KB row
// reads).  The per-column hash is a wrap-around sum of mixed (row, value) pairs, so
// equal columns hash alike and partial sums from different blocks simply add.
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
// are found through a small open-addressing table in shared memory.  Also clears the
// counters of the token sort.
__global__ void __launch_bounds__(256) derive_classes(const uint64_t* __restrict__ partial,
                                                     int nblocks, IndexMeta* meta, uint8_t* cls,
                                                     uint8_t* class_rep, int32_t* gcount,
                                                     int32_t* count2, int32_t* cursor2) {
    constexpr int kSlots = 1024;
    __shared__ unsigned long long keys[kSlots];
    __shared__ int min_byte[kSlots];
    __shared__ uint32_t rep_bits[8];
    constexpr unsigned long long kEmpty = ~0ull;
    const int b = threadIdx.x;
    gcount[b] = 0;
    for (int i = b; i < kKeys; i += 256) {
        count2[i] = 0;
        cursor2[i] = 0;
    }
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
// Blocks [0, row_blocks) compress and verify table rows; the remaining blocks work on
// tokens: class records in token order for the dense walk (count2 == nullptr), or
// bucket counts for the sparse walk.  Column C of the compressed table (the null class)
// and the padding columns lead to the dead state, as does the whole row of the dead state.
template <typename TabT>
__global__ void __launch_bounds__(256)
prepare_inputs(const int32_t* __restrict__ trans, const uint8_t* __restrict__ vocab_bytes,
               const int32_t* __restrict__ vocab_offsets, int64_t vocab_nbytes, int32_t Q,
               int32_t N, int32_t dead, int32_t eos_id, int row_blocks, IndexMeta* meta,
               const uint8_t* __restrict__ cls, const uint8_t* __restrict__ class_rep,
               TabT* __restrict__ table, uint4* __restrict__ tok_cls,
               uint8_t* __restrict__ tok_len, int32_t* __restrict__ gcount,
               int32_t* __restrict__ count2, int32_t* status) {
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
    } else if (count2 != nullptr) {
        __shared__ int hist[256];
        __shared__ uint8_t s_cls[256];
        hist[threadIdx.x] = 0;
        s_cls[threadIdx.x] = cls[threadIdx.x];
        __syncthreads();
        bool bad = false;
        const bool two = meta->two_level != 0;
        const int64_t v = static_cast<int64_t>(blockIdx.x - row_blocks) * 256 + threadIdx.x;
        const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
        if (t.len > 0) {
            atomicAdd(&hist[t.first], 1);
            atomicAdd(&count2[bucket_key(two, t.first, t.second_key)], 1);
        }
        if (__syncthreads_or(bad) && threadIdx.x == 0) raise_flag(status, FSM_FLAG_OFFSETS);
        if (hist[threadIdx.x] > 0) atomicAdd(&gcount[threadIdx.x], hist[threadIdx.x]);
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

// ---------------------------------------------------------------------------- 3b
// Token order of the sparse walk: a counting sort by bucket key - the class of the
// first byte and, when there are at most kTwoLevelMaxC classes, the class of the second
// byte (key 0 = one-byte token).  Blocks [0, token_blocks) place 256 tokens each; the
// remaining blocks publish the first sorted position of every key (start2).  A record
// keeps the length and the classes of bytes 1..15; `sid` holds the token id.
__global__ void __launch_bounds__(256)
sort_tokens(const uint8_t* __restrict__ vocab_bytes, const int32_t* __restrict__ vocab_offsets,
            int64_t vocab_nbytes, int32_t N, int32_t eos_id, int token_blocks,
            const IndexMeta* __restrict__ meta, const uint8_t* __restrict__ cls,
            const int32_t* __restrict__ gcount, const int32_t* __restrict__ count2,
            int32_t* __restrict__ cursor2, int32_t* __restrict__ gstart,
            int32_t* __restrict__ start2, uint4* __restrict__ srec, int32_t* __restrict__ sid) {
    __shared__ int gst[257];
    __shared__ uint8_t s_cls[256];
    s_cls[threadIdx.x] = cls[threadIdx.x];
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
    const bool two = meta->two_level != 0;
    const int C = meta->C;
    if (static_cast<int>(blockIdx.x) >= token_blocks) {
        const int c0 = blockIdx.x - token_blocks;
        if (c0 == 0) {
            gstart[threadIdx.x] = gst[threadIdx.x];
            if (threadIdx.x == 0) gstart[256] = gst[256];
        }
        if (two) {
            if (c0 < C && static_cast<int>(threadIdx.x) <= C) {
                int before = 0;
                for (int k = 0; k < static_cast<int>(threadIdx.x); ++k)
                    before += count2[c0 * kKeyStride + k];
                start2[c0 * kKeyStride + threadIdx.x] = gst[c0] + before;
            }
        } else if (c0 == 0) {
            start2[threadIdx.x] = gst[threadIdx.x];
        }
        return;
    }
    bool bad = false;
    const int64_t v = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
    const TokenInfo t = token_info(vocab_bytes, vocab_offsets, vocab_nbytes, N, eos_id, s_cls, v, &bad);
    if (t.len > 0) {
        int before = 0;
        if (two)
            for (int k = 0; k < t.second_key; ++k) before += count2[t.first * kKeyStride + k];
        const int pos = gst[t.first] + before +
                        atomicAdd(&cursor2[bucket_key(two, t.first, t.second_key)], 1);
        uint32_t w[4] = {static_cast<uint32_t>(t.len), 0, 0, 0};
        const int nb = min(t.len, kInlineBytes);
        for (int i = 1; i < nb; ++i)
            w[i >> 2] |= static_cast<uint32_t>(s_cls[vocab_bytes[t.start + i]]) << ((i & 3) * 8);
        srec[pos] = make_uint4(w[0], w[1], w[2], w[3]);
        sid[pos] = static_cast<int32_t>(v);
    }
}

}  // namespace
}  // namespace fsm
