// Work-avoiding walk of the index build.
//
// Most (state, token) walks die on their first or second byte.  Tokens are therefore
// kept sorted by bucket key - the class of byte 0 and (with few enough classes) the class
// of byte 1 - so that one table lookup settles a whole bucket:
//
//   fill    every row of the next-state table is first set to `dead` and its bitmask
//           row to 0.  The fill is done by the bulk-copy engine (cp.async.bulk, shared
//           -> global) from a constant buffer in shared memory, issued one row ahead of
//           the walk by a single thread, so it costs no issue slots and overlaps the
//           walk of the previous row.
//   walk    for a state q, only buckets whose key q can read are visited: a unit of
//           work is (readable first class, block of 32 second keys); the units of all
//           rows of a CTA are dealt round-robin to its 32 warps, which work without any
//           CTA-wide barrier.  Inside a bucket, lane = token, 32 tokens at a time, from
//           the first byte the bucket key does not cover.
//   scatter survivors store their end state into the row and OR their bit into the
//           bitmask row.  The row was written moments earlier from the same SM, so these
//           partial writes merge in L2.
//
// One persistent CTA per SM; the compressed table is staged in shared memory once
// (bulk async copy) when it fits, else lookups go through the read-only cache.
// Results are identical to the dense walk.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

constexpr uint32_t kFillBytes = 16384;  // shared-memory source of the row fill
constexpr uint32_t kZeroBytes = 4096;   // shared-memory source of the bitmask fill
constexpr uint32_t kSparseFixedSmem = kFillBytes + kZeroBytes;

__device__ __forceinline__ void bulk_store_s2g(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
                 "r"(smem_addr(src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int kPending>
__device__ __forceinline__ void bulk_wait() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(kPending) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async;" ::: "memory");
}

// Fills `count` elements at `dst` with the pattern held in `src` (a shared-memory
// buffer of `src_bytes` bytes): the 16-byte aligned middle by bulk stores, the ragged
// head and tail with plain stores.  Called by one thread.
template <typename T>
__device__ __forceinline__ void fill_async(T* dst, int64_t count, T value, const void* src,
                                           uint32_t src_bytes) {
    const uintptr_t addr = reinterpret_cast<uintptr_t>(dst);
    int64_t head = static_cast<int64_t>(((16 - (addr & 15)) & 15) / sizeof(T));
    if (head > count) head = count;
    for (int64_t i = 0; i < head; ++i) dst[i] = value;
    const int64_t mid_bytes = (count - head) * static_cast<int64_t>(sizeof(T)) / 16 * 16;
    uint8_t* mid = reinterpret_cast<uint8_t*>(dst + head);
    for (int64_t o = 0; o < mid_bytes; o += src_bytes) {
        const int64_t left = mid_bytes - o;
        bulk_store_s2g(mid + o, src, left < src_bytes ? static_cast<uint32_t>(left) : src_bytes);
    }
    for (int64_t i = head + mid_bytes / static_cast<int64_t>(sizeof(T)); i < count; ++i) dst[i] = value;
}

// Bounded wait for the fill of this CTA's k-th row.
__device__ __forceinline__ bool wait_row_filled(const int* flag, int k) {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        int v;
        asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_addr(flag)) : "memory");
        if (v >= k) return true;
        __nanosleep(64);
    }
    return false;
}

// One chunk: up to 32 tokens of a bucket (lane = token), starting at sorted position
// `pos`, all in state `s` after the DEPTH bytes the bucket key covers.
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL, int DEPTH>
__device__ __forceinline__ void walk_chunk(const WalkParams& p, const TabT* __restrict__ tab,
                                           uint32_t Cs, OutT* nrow, uint32_t* mrow, int pos,
                                           int count, uint32_t s, int lane) {
    const uint32_t dead = p.dead;
    uint4 rec = make_uint4(0, 0, 0, 0);
    int32_t id = -1;
    if (lane < count) {
        rec = __ldg(p.srec + pos + lane);
        id = __ldg(p.sid + pos + lane);
    }
    const int len = rec.x & 0xFFu;
    bool go = len > DEPTH;
    uint32_t st = walk_rest<TabT, FULL, DEPTH>(tab, Cs, dead, rec, len, s, go);
    if (go)  // longer than the inline record and still alive: finish on the raw bytes
        st = raw_walk(p, st, p.vocab_offsets[id], p.vocab_offsets[id + 1], kInlineBytes);
    if (id >= 0 && st != dead) {
        if (HAS_OUT) nrow[id] = static_cast<OutT>(st);
        atomicOr(&mrow[id >> 5], 1u << (id & 31));
    }
}

template <typename TabT, typename OutT, bool HAS_OUT, bool FULL>
__device__ __forceinline__ void sparse_rows(const WalkParams& p, const TabT* __restrict__ tab,
                                            int C, uint32_t Cs, bool two_level,
                                            const int32_t* s_gstart, int* filled,
                                            const void* fillbuf, const void* zerobuf, int nmine) {
    const uint32_t dead = p.dead;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (FULL) return tab[s * Cs + c];
        return __ldg(tab + static_cast<size_t>(s) * Cs + c);
    };
    auto issue_fill = [&](int k) {  // thread 0 only
        const int r = blockIdx.x + k * gridDim.x;
        if (HAS_OUT)
            fill_async<OutT>(static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N, p.N,
                             static_cast<OutT>(dead), fillbuf, kFillBytes);
        fill_async<uint32_t>(p.mask + static_cast<size_t>(r) * p.G, p.G, 0u, zerobuf, kZeroBytes);
        bulk_commit();
    };

    if (threadIdx.x == 0 && nmine > 0) issue_fill(0);
    const int KB = two_level ? (C + 1 + 31) / 32 : 1;  // blocks of 32 second-level keys
    int u_base = 0;                                    // units dealt so far, modulo 32
    for (int k = 0; k < nmine; ++k) {
        const int r = blockIdx.x + k * gridDim.x;
        const int q = p.q_begin + r;
        if (threadIdx.x == 0) {
            // keep the fill one row ahead, then publish that row k is ready
            if (k + 1 < nmine) {
                issue_fill(k + 1);
                bulk_wait<1>();
            } else {
                bulk_wait<0>();
            }
            fence_proxy_async();
            asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_addr(filled)), "r"(k) : "memory");
        }
        __syncwarp();
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
        const int U = n_live * KB;
        const int first = (warp - u_base) & 31;
        u_base = (u_base + U) & 31;
        const bool eos_mine = (p.eos_id >= 0) && ((k & 31) == warp);
        if (first >= U && !eos_mine) continue;
        if (!wait_row_filled(filled, k)) {
            if (lane == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
            return;
        }
        OutT* nrow = HAS_OUT ? static_cast<OutT*>(p.next) + static_cast<size_t>(r) * p.N : nullptr;
        uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G;
        if (eos_mine && lane == 0 && q != p.dead && p.accept[q]) {
            if (HAS_OUT) nrow[p.eos_id] = static_cast<OutT>(q);
            atomicOr(&mrow[p.eos_id >> 5], 1u << (p.eos_id & 31));
        }
        for (int j = first; j < U; j += 32) {
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
            uint32_t m = __ballot_sync(kFullWarp, cnt > 0 && s2 != dead);
            while (m) {
                const int l = __ffs(m) - 1;
                m &= m - 1;
                const int bstart = __shfl_sync(kFullWarp, start, l);
                const int bn = __shfl_sync(kFullWarp, cnt, l);
                const uint32_t bs = __shfl_sync(kFullWarp, s2, l);
                if (two_level && !(kb == 0 && l == 0)) {
                    for (int i0 = 0; i0 < bn; i0 += 32)
                        walk_chunk<TabT, OutT, HAS_OUT, FULL, 2>(p, tab, Cs, nrow, mrow, bstart + i0,
                                                                 bn - i0, bs, lane);
                } else {
                    for (int i0 = 0; i0 < bn; i0 += 32)
                        walk_chunk<TabT, OutT, HAS_OUT, FULL, 1>(p, tab, Cs, nrow, mrow, bstart + i0,
                                                                 bn - i0, bs, lane);
                }
            }
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
            for (int i = threadIdx.x; i < p.N; i += kWalkThreads) nrow[i] = static_cast<OutT>(dead);
        for (int i = threadIdx.x; i < p.G; i += kWalkThreads) mrow[i] = 0;
        __syncthreads();  // orders the fill before the scattered stores
        if (q != p.dead) {
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
            if (threadIdx.x == 0 && p.eos_id >= 0 && p.accept[q]) {
                if (HAS_OUT) nrow[p.eos_id] = static_cast<OutT>(q);
                atomicOr(&mrow[p.eos_id >> 5], 1u << (p.eos_id & 31));
            }
        }
    }
}

template <typename TabT, typename OutT, bool HAS_OUT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk_sparse(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ int filled;
    __shared__ int32_t s_gstart[260];
    uint8_t* fillbuf = smem_raw;
    uint8_t* zerobuf = smem_raw + kFillBytes;
    TabT* stab = reinterpret_cast<TabT*>(smem_raw + kSparseFixedSmem);

    if (p.meta->any_bad != 0) {
        raw_rows<OutT, HAS_OUT>(p);
        return;
    }
    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int C = p.meta->C, Cs = p.meta->Cs;
    const bool two_level = p.meta->two_level != 0;
    const uint64_t table_bytes = static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT);
    const bool full = p.smem_cap > kSparseFixedSmem && table_bytes <= p.smem_cap - kSparseFixedSmem;

    // constant sources of the fills, bucket starts, table
    {
        const uint32_t d = sizeof(OutT) == 2 ? (p.dead | (p.dead << 16)) : p.dead;
        for (uint32_t i = threadIdx.x; i < kFillBytes / 16; i += kWalkThreads)
            reinterpret_cast<uint4*>(fillbuf)[i] = make_uint4(d, d, d, d);
        for (uint32_t i = threadIdx.x; i < kZeroBytes / 16; i += kWalkThreads)
            reinterpret_cast<uint4*>(zerobuf)[i] = make_uint4(0, 0, 0, 0);
        for (int i = threadIdx.x; i < 257; i += kWalkThreads) s_gstart[i] = p.gstart[i];
        if (threadIdx.x == 0) {
            filled = -1;
            mbar_init(&bar, 1);
            fence_mbar_init();
        }
        fence_proxy_async();  // the bulk engine reads fillbuf / zerobuf written above
    }
    __syncthreads();
    if (full) {
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
    const int nrows = p.q_end - p.q_begin;
    const int nmine = nrows > static_cast<int>(blockIdx.x)
                          ? (nrows - blockIdx.x + gridDim.x - 1) / gridDim.x
                          : 0;
    if (full)
        sparse_rows<TabT, OutT, HAS_OUT, true>(p, stab, C, Cs, two_level, s_gstart, &filled, fillbuf,
                                               zerobuf, nmine);
    else
        sparse_rows<TabT, OutT, HAS_OUT, false>(p, gtab, C, Cs, two_level, s_gstart, &filled, fillbuf,
                                                zerobuf, nmine);
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

}  // namespace
}  // namespace fsm
