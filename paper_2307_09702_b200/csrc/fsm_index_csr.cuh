// Compressed-row form of the index: sigma(q) as the list of q's allowed tokens (the
// paper's own data structure, Algorithm 4) with the end state of each beside it.  Most
// (state, token) pairs are not allowed, so this form is a tenth of the dense table.
//
// The rows are cut out of the bitmask of a bitmask-only build:
//   csr_count  allowed tokens per row (population count of the row's bitmask words)
//   csr_scan   exclusive prefix sum -> row_offsets (one block)
//   csr_fill   one block per row, a warp per run of bitmask words: 32 words at a time are
//              expanded into the list of their token ids (increasing), then lane = token:
//              the end state of a one-byte token is delta(q, byte), the other tokens are
//              collected and walked once more through the uncompressed table.
// An automaton of fewer than kCsrDenseRows states (a typical regular expression) gives the
// walks too few rows to spread over the SMs, and its rows are long: for it the dense table
// is built into the workspace (16-bit states) and csr_fill copies the end states from it.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

constexpr int kCsrThreads = 256;
constexpr int kCsrRankBuckets = 1024;  // row-length buckets of csr_fill's row order

__global__ void __launch_bounds__(kCsrThreads)
csr_count(const uint32_t* __restrict__ mask, int32_t G, int32_t nrows, int32_t* __restrict__ row_count) {
    __shared__ int wsum[kCsrThreads / 32];
    for (int r = blockIdx.x; r < nrows; r += gridDim.x) {
        const uint32_t* mrow = mask + static_cast<size_t>(r) * G;
        int n = 0;
        for (int i = threadIdx.x; i < G; i += kCsrThreads) n += __popc(mrow[i]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) n += __shfl_xor_sync(kFullWarp, n, off);
        if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = n;
        __syncthreads();
        if (threadIdx.x == 0) {
            int t = 0;
            for (int w = 0; w < kCsrThreads / 32; ++w) t += wsum[w];
            row_count[r] = t;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(1024)
csr_scan(const int32_t* __restrict__ row_count, int32_t nrows, int64_t* __restrict__ row_offsets,
         int64_t capacity, int32_t N, int32_t* __restrict__ row_order, int32_t* status) {
    __shared__ long long wsum[32];
    __shared__ long long carry;
    __shared__ int s_rank[kCsrRankBuckets];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < nrows; base += 1024) {
        const int r = base + threadIdx.x;
        const long long mine = r < nrows ? row_count[r] : 0;
        long long incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const long long o = __shfl_up_sync(kFullWarp, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        long long before = carry;
        for (int w = 0; w < warp; ++w) before += wsum[w];
        if (r < nrows) row_offsets[r] = before + incl - mine;
        __syncthreads();
        if (threadIdx.x == 1023) carry = before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        row_offsets[nrows] = carry;
        if (carry > capacity) raise_flag(status, FSM_FLAG_CSR_OVERFLOW);
    }
    // The rows in the order csr_fill takes them: longest first (counting sort by length), so
    // that the blocks of the long rows do not start last.
    auto bucket_of = [&](int r) {
        const long long b = static_cast<long long>(row_count[r]) * kCsrRankBuckets / (static_cast<long long>(N) + 1);
        return kCsrRankBuckets - 1 - static_cast<int>(b < kCsrRankBuckets - 1 ? b : kCsrRankBuckets - 1);
    };
    static_assert(kCsrRankBuckets == 1024, "one bucket per thread");
    s_rank[threadIdx.x] = 0;
    __syncthreads();
    for (int r = threadIdx.x; r < nrows; r += 1024) atomicAdd(&s_rank[bucket_of(r)], 1);
    __syncthreads();
    {
        const int mine = s_rank[threadIdx.x];
        int incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(kFullWarp, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int before = 0;
        for (int w = 0; w < warp; ++w) before += static_cast<int>(wsum[w]);
        s_rank[threadIdx.x] = before + incl - mine;
    }
    __syncthreads();
    for (int r = threadIdx.x; r < nrows; r += 1024) {
        const int at = atomicAdd(&s_rank[bucket_of(r)], 1);
        if (idx_ok(at, nrows, status)) row_order[at] = r;
    }
}

constexpr int kFillThreads = 128;
constexpr int kFillWarps = kFillThreads / 32;
constexpr int kLongCap = 256;  // tokens set aside for a walk before the warp walks them

__global__ void __launch_bounds__(kFillThreads)
csr_fill(const WalkParams p, const uint16_t* __restrict__ tok_head,
         const uint16_t* __restrict__ dense_next, const int32_t* __restrict__ row_order,
         const int64_t* __restrict__ row_offsets,
         int32_t* __restrict__ csr_tokens, int32_t* __restrict__ csr_next, int64_t capacity) {
    __shared__ int wsum[kFillWarps], wfront[kFillWarps];
    __shared__ uint16_t s_ids[kFillWarps][1024];   // tokens of 32 bitmask words, in order (id - 32 * first word)
    __shared__ int2 s_long[kFillWarps][kLongCap];  // (entry position - row start, token) to walk
    const int nrows = p.q_end - p.q_begin;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // block (x, y) owns part y of the words of rows x, x + gridDim.x, ...; a warp owns a run
    // (a multiple of 32) of those words.  Short runs keep the chains of dependent loads short.
    const int bper = ((p.G + static_cast<int>(gridDim.y) - 1) / static_cast<int>(gridDim.y) + 31) / 32 * 32;
    const int b0 = min(p.G, static_cast<int>(blockIdx.y) * bper), b1 = min(p.G, b0 + bper);
    const int wper = ((b1 - b0 + kFillWarps - 1) / kFillWarps + 31) / 32 * 32;
    const int w0 = min(b1, b0 + warp * wper), w1 = min(b1, w0 + wper);
    uint16_t* ids = s_ids[warp];
    int2* longs = s_long[warp];
    for (int ri = blockIdx.x; ri < nrows; ri += gridDim.x) {
        const int r = row_order[ri];
        if (!idx_ok(r, nrows, p.status)) continue;  // (block-uniform)
        const int q = p.q_begin + r;
        const uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G;
        const int32_t* trow = p.trans + static_cast<size_t>(q) * 256;
        // entries of the row in front of this warp's run: words [0, b0) are shared out over
        // the block, words [b0, w0) belong to the warps before this one
        int front = 0, mine = 0;
        for (int i = threadIdx.x; i < b0; i += kFillThreads) front += __popc(mrow[i]);
        for (int i = w0 + lane; i < w1; i += 32) mine += __popc(mrow[i]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            front += __shfl_xor_sync(kFullWarp, front, off);
            mine += __shfl_xor_sync(kFullWarp, mine, off);
        }
        if (lane == 0) {
            wfront[warp] = front;
            wsum[warp] = mine;
        }
        __syncthreads();
        const int64_t row_at = row_offsets[r];
        int at = 0;  // entries of the row in front of the current 32 words
        for (int w = 0; w < kFillWarps; ++w) at += wfront[w] + (w < warp ? wsum[w] : 0);
        int nlong = 0;
        // walks the tokens set aside so far, 32 at a time (all lanes busy)
        auto walk_longs = [&]() {
            for (int t = lane; t < nlong; t += 32) {
                const int2 e = longs[t];
                if (!idx_ok(e.y, p.N, p.status) || !idx_ok(row_at + e.x, capacity, p.status)) continue;
                const uint32_t s = raw_walk(p, q, p.vocab_offsets[e.y], p.vocab_offsets[e.y + 1], 0);
                csr_next[row_at + e.x] = static_cast<int32_t>(s);
            }
            nlong = 0;
            __syncwarp();
        };
        for (int base = w0; base < w1; base += 32) {  // lane = bitmask word
            const int wi = base + lane;
            uint32_t bits = wi < w1 ? mrow[wi] : 0u;
            const int cnt = __popc(bits);
            int incl = cnt;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(kFullWarp, incl, off);
                if (lane >= off) incl += o;
            }
            const int total = __shfl_sync(kFullWarp, incl, 31);
            int k = incl - cnt;
            while (bits) {
                if (idx_ok(k, 1024, p.status)) ids[k] = static_cast<uint16_t>(lane * 32 + __ffs(bits) - 1);
                ++k;
                bits &= bits - 1;
            }
            __syncwarp();
            // lane = allowed token: one-byte tokens (and EOS) need one lookup, the others are
            // set aside and walked together once enough of them have come up
            for (int j0 = 0; j0 < total; j0 += 32) {
                const int j = j0 + lane;
                bool walk = false;
                int v = 0;
                if (j < total && idx_ok(j, 1024, p.status) && idx_ok(base * 32 + ids[j], p.N, p.status)) {
                    v = base * 32 + ids[j];
                    uint32_t s = q;  // EOS keeps the state
                    if (dense_next != nullptr) {  // small automaton: the dense table was built
                        s = __ldg(dense_next + static_cast<size_t>(r) * p.N + v);
                    } else {
                        const uint32_t head = __ldg(tok_head + v);
                        walk = v != p.eos_id && (head >> 8) != 1;
                        if (v != p.eos_id && !walk)
                            s = clamp_state(__ldg(trow + (head & 0xFFu)), p.Q, p.dead);
                    }
                    if (row_at + at + j < capacity) {
                        csr_tokens[row_at + at + j] = v;
                        if (!walk) csr_next[row_at + at + j] = static_cast<int32_t>(s);
                    } else {
                        walk = false;
                    }
                }
                const uint32_t m = __ballot_sync(kFullWarp, walk);
                if (nlong + __popc(m) > kLongCap) {
                    __syncwarp();  // the entries other lanes set aside are visible to the walk
                    walk_longs();
                }
                const int slot = nlong + __popc(m & ((1u << lane) - 1u));
                if (walk && idx_ok(slot, kLongCap, p.status)) longs[slot] = make_int2(at + j, v);
                nlong += __popc(m);
            }
            at += total;
            __syncwarp();  // the id list is rewritten by the next 32 words
        }
        __syncwarp();
        walk_longs();
        __syncthreads();  // wsum is reused by the next row
    }
}

}  // namespace
}  // namespace fsm
