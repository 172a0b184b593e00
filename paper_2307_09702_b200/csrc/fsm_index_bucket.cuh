// Bucket walk of the index build for bitmask-only builds (no next-state table): two kernels
// that never visit a (state, token) pair whose first two bytes the state cannot read.
//
//   mask_onebyte  A token of one byte is allowed in state q iff q reads the class of that
//                 byte, so the bitmask words of all one-byte tokens are the OR, over the
//                 classes q reads, of per-class bit planes prepared once per vocabulary.
//                 The kernel writes every bitmask word (tokens of two or more bytes get
//                 their bits from walk_buckets).
//   walk_buckets  Tokens are kept sorted by (class of byte 0, class of byte 1).  A warp
//                 takes 32 consecutive sorted tokens (lane = token, record in registers)
//                 and a block of 128 states; for every key present in the window it scans
//                 the states (lane = state, two table lookups) and walks the window from
//                 each state that reads the key, starting at byte 2.  A surviving token
//                 sets its bitmask bit with an atomic OR.
//
// The compressed table is staged in shared memory (bulk async copy) when it fits, else
// lookups use the read-only cache.  Results are identical to the dense walk.
#pragma once

#include "fsm_index_common.cuh"
#include "fsm_index_rows.cuh"

namespace fsm {
namespace {

constexpr int kStatesPerTask = 128;   // states scanned by one walk_buckets task

// Stages the whole compressed table in shared memory when it fits.  Returns false (after
// raising the flag) when the bounded wait gave up; `full` tells whether the table is in
// shared memory.
template <typename TabT>
__device__ __forceinline__ bool stage_table(const WalkParams& p, TabT* stab, uint64_t* bar,
                                            uint32_t table_cap, uint32_t Cs, bool& full) {
    // (a bulk copy moves multiples of 16 bytes; the table's workspace has the slack)
    const uint64_t table_bytes = (static_cast<uint64_t>(p.Q) * Cs * sizeof(TabT) + 15) / 16 * 16;
    full = table_bytes <= table_cap;
    if (!full) return true;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t bytes = static_cast<uint32_t>(table_bytes);
        mbar_expect_tx(bar, bytes);
        for (uint32_t o = 0; o < bytes; o += kBulkChunk)
            bulk_copy_g2s(reinterpret_cast<uint8_t*>(stab) + o,
                          reinterpret_cast<const uint8_t*>(p.table) + o, min(kBulkChunk, bytes - o),
                          bar);
    }
    bool ok = mbar_wait_bounded(bar, 0);
    if (!ok) ok = mbar_wait_bounded(bar, 0);  // drain before giving up
    if (ok && p.wait_probe > 0) ok = mbar_wait_bounded(bar, 1, p.wait_probe);  // never completes
    if (!__syncthreads_and(ok)) {
        if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
        return false;
    }
    return true;
}

// ---------------------------------------------------------------------------------------
// Bitmask words of the one-byte tokens (and zeros elsewhere).  Block (x, y): the 128
// bitmask words 128x .. 128x+127 of the rows 8y + warp, 8y + warp + 8 gridDim.y, ...; those
// words of the first 64 planes sit in shared memory; lane l handles words 4l .. 4l+3.
constexpr int kObThreads = 256;
constexpr int kObWords = 128;
constexpr int kObSmemClasses = 64;  // planes of further classes are read through the cache

__global__ void __launch_bounds__(kObThreads) mask_onebyte(const WalkParams p) {
    __shared__ __align__(16) uint32_t s_pl[kObSmemClasses * kObWords];  // planes of the first classes
    __shared__ uint8_t s_live[kObThreads / 32][256];      // classes read by the warp's row
    if (p.meta->any_bad != 0) {
        // exact fallback: every token walked through the uncompressed table
        if (blockIdx.y == 0) raw_rows<int32_t, false>(p);
        return;
    }
    const int C = p.meta->C;
    const int nrows = p.q_end - p.q_begin;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int w0 = blockIdx.x * kObWords;
    const int c_smem = min(C, kObSmemClasses);
    for (int i = threadIdx.x; i < c_smem * kObWords; i += kObThreads) {
        const int wd = w0 + (i & (kObWords - 1));
        s_pl[i] = wd < p.G ? p.planes[static_cast<size_t>(i / kObWords) * plane_stride(p.G) + wd] : 0;
    }
    __syncthreads();
    const int eos_word = p.eos_id >= 0 ? (p.eos_id >> 5) - w0 : -1;
    uint8_t* mine = s_live[warp];
    for (int r = blockIdx.y * (kObThreads / 32) + warp; r < nrows; r += gridDim.y * (kObThreads / 32)) {
        const int q = p.q_begin + r;
        // the classes q reads, as a list
        int nlive = 0;
        for (int k = 0; k * 32 < C; ++k) {
            const uint32_t m = __ldg(p.live + static_cast<size_t>(q) * 8 + k);
            const int slot = nlive + __popc(m & ((1u << lane) - 1u));
            if (((m >> lane) & 1u) && idx_ok(slot, 256, p.status)) mine[slot] = static_cast<uint8_t>(k * 32 + lane);
            nlive += __popc(m);
        }
        __syncwarp();
        // lane l holds words 4l .. 4l+3 of the block's 128
        uint4 acc = make_uint4(0, 0, 0, 0);
        const int wl = w0 + 4 * lane;
        if (!idx_ok(nlive, 257, p.status)) nlive = 0;
        for (int j = 0; j < nlive; ++j) {
            const int c = mine[j];
            uint4 v;
            if (c < kObSmemClasses) {
                v = *reinterpret_cast<const uint4*>(s_pl + c * kObWords + 4 * lane);
            } else {
                const uint32_t* pl = p.planes + static_cast<size_t>(c) * plane_stride(p.G) + wl;
                v.x = wl < p.G ? __ldg(pl) : 0u;
                v.y = wl + 1 < p.G ? __ldg(pl + 1) : 0u;
                v.z = wl + 2 < p.G ? __ldg(pl + 2) : 0u;
                v.w = wl + 3 < p.G ? __ldg(pl + 3) : 0u;
            }
            acc.x |= v.x;
            acc.y |= v.y;
            acc.z |= v.z;
            acc.w |= v.w;
        }
        if (eos_word >= 0 && eos_word < kObWords && (eos_word >> 2) == lane && q != p.dead && p.accept[q]) {
            const uint32_t bit = 1u << (p.eos_id & 31);
            const int k = eos_word & 3;
            acc.x |= k == 0 ? bit : 0u;
            acc.y |= k == 1 ? bit : 0u;
            acc.z |= k == 2 ? bit : 0u;
            acc.w |= k == 3 ? bit : 0u;
        }
        uint32_t* mrow = p.mask + static_cast<size_t>(r) * p.G + wl;
        if (wl + 3 < p.G && (reinterpret_cast<uintptr_t>(mrow) & 15) == 0) {
            *reinterpret_cast<uint4*>(mrow) = acc;
        } else {
            if (wl < p.G) mrow[0] = acc.x;
            if (wl + 1 < p.G) mrow[1] = acc.y;
            if (wl + 2 < p.G) mrow[2] = acc.z;
            if (wl + 3 < p.G) mrow[3] = acc.w;
        }
        __syncwarp();  // the list is rewritten for the next row
    }
}

// ---------------------------------------------------------------------------------------
// Survivors among the tokens of two or more bytes.
template <typename TabT, bool FULL>
__device__ __forceinline__ void bucket_tasks(const WalkParams& p, const TabT* __restrict__ tab,
                                             uint32_t Cs, const int32_t* s_gstart, int* s_next) {
    const uint32_t dead = p.dead;
    auto lookup = [&](uint32_t s, uint32_t c) -> uint32_t {
        if (!idx_ok(static_cast<size_t>(s) * Cs + c, static_cast<size_t>(p.Q) * Cs, p.status)) return dead;
        if (FULL) return tab[s * Cs + c];
        return __ldg(tab + static_cast<size_t>(s) * Cs + c);
    };
    const int lane = threadIdx.x & 31;
    const int n_sorted = s_gstart[256];
    const int nwin = (n_sorted + 31) >> 5;
    const int nrows = p.q_end - p.q_begin;
    const int parts = (nrows + kStatesPerTask - 1) / kStatesPerTask;
    const int64_t ntasks = static_cast<int64_t>(nwin) * parts;
    // Tasks cost very differently (a window of rare keys holds many keys, each with its own
    // scan of the states).  The windows come in the order of p.win_order, most keys first;
    // task i of this CTA is task i * gridDim.x + blockIdx.x of that order, so that every CTA
    // gets the same mix, and inside the CTA warps draw from a counter, heaviest tasks first.
    while (true) {
        int i = 0;
        if (lane == 0) i = atomicAdd(s_next, 1);
        i = __shfl_sync(kFullWarp, i, 0);
        const int64_t t = static_cast<int64_t>(i) * gridDim.x + blockIdx.x;
        if (t >= ntasks) break;
        const int wat = static_cast<int>(t / parts);
        const int part = static_cast<int>(t - static_cast<int64_t>(wat) * parts);
        int win = p.win_order != nullptr ? __ldg(p.win_order + wat) : wat;
        if (!idx_ok(win, nwin, p.status)) win = nwin;  // (nothing to walk there)
        const int pos = win * 32 + lane;
        uint4 rec = make_uint4(0, 0, 0, 0);
        int32_t id = -1;
        if (pos < n_sorted && idx_ok(pos, p.N, p.status)) {
            rec = __ldg(p.srec + pos);
            id = static_cast<int32_t>(rec.w);
            if (!idx_ok(id, p.N, p.status)) id = -1;
        }
        const int len = rec.x & 0xFFu;
        const bool active = id >= 0 && len >= 2;
        uint32_t todo = __ballot_sync(kFullWarp, active);
        if (todo == 0) continue;
        // first-byte class: the last c with gstart[c] <= pos
        int c0 = 0;
#pragma unroll
        for (int step = 128; step > 0; step >>= 1)
            if (s_gstart[c0 + step] <= pos) c0 += step;
        const uint32_t key = (static_cast<uint32_t>(c0) << 8) | ((rec.x >> 8) & 0xFFu);
        const uint32_t bit = 1u << (id & 31);
        const int word = id >> 5;
        while (todo) {
            const uint32_t kl = __shfl_sync(kFullWarp, key, __ffs(todo) - 1);
            const bool same = active && key == kl;
            todo &= ~__ballot_sync(kFullWarp, same);
            const uint32_t c0l = kl >> 8, c1l = kl & 0xFFu;
            for (int g = 0; g < kStatesPerTask / 32; ++g) {
                const int rbase = part * kStatesPerTask + g * 32;
                if (rbase >= nrows) break;
                uint32_t s2 = dead;
                if (rbase + lane < nrows) s2 = lookup(lookup(p.q_begin + rbase + lane, c0l), c1l);
                uint32_t m = __ballot_sync(kFullWarp, s2 != dead);
                while (m) {
                    const int l = __ffs(m) - 1;
                    m &= m - 1;
                    const uint32_t s = __shfl_sync(kFullWarp, s2, l);
                    bool go = same && len > 2;
                    uint32_t st = walk_rest<TabT, FULL, 2, kSortedInline>(tab, Cs, dead, rec, len, s, go,
                                                                          static_cast<uint32_t>(p.Q) * Cs, p.status);
                    if (go)  // longer than the record covers and still alive
                        st = raw_walk(p, st, p.vocab_offsets[id], p.vocab_offsets[id + 1], kSortedInline);
                    if (same && st != dead)
                        atomicOr(p.mask + static_cast<size_t>(rbase + l) * p.G + word, bit);
                }
            }
        }
    }
}

template <typename TabT>
__global__ void __launch_bounds__(kWalkThreads, 1) walk_buckets(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    __shared__ int32_t s_gstart[260];
    __shared__ int s_next;
    if (p.meta->any_bad != 0) return;  // mask_onebyte did the whole build
    TabT* stab = reinterpret_cast<TabT*>(smem_raw);
    const uint32_t Cs = p.meta->Cs;
    for (int i = threadIdx.x; i < 257; i += kWalkThreads) s_gstart[i] = p.gstart[i];
    if (threadIdx.x == 0) s_next = 0;
    bool full;
    if (!stage_table<TabT>(p, stab, &bar, p.smem_cap, Cs, full)) return;
    __syncthreads();
    if (full)
        bucket_tasks<TabT, true>(p, stab, Cs, s_gstart, &s_next);
    else
        bucket_tasks<TabT, false>(p, static_cast<const TabT*>(p.table), Cs, s_gstart, &s_next);
}

// ---------------------------------------------------------------------------------------
template <typename TabT>
cudaError_t launch_bucket(const WalkParams& p, int sms, cudaStream_t stream) {
    const int nrows = p.q_end - p.q_begin;
    // mask_onebyte: 128 bitmask words per block column, rows spread over the block rows
    const int ycap = (nrows + 7) / 8;
    const int cols = (p.G + kObWords - 1) / kObWords;
    int ymax = 5 * sms / cols;  // five blocks per SM (six fit): one even wave
    if (ymax < 1) ymax = 1;
    dim3 grid_a(cols, ycap < ymax ? ycap : ymax);
    cudaError_t e = launch_on(mask_onebyte, grid_a, dim3(kObThreads), 0, stream, p);
    if (e != cudaSuccess) return e;
    auto k1 = walk_buckets<TabT>;
    e = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    return launch_on(k1, dim3(sms), dim3(kWalkThreads), p.smem_cap, stream, p);
}

}  // namespace
}  // namespace fsm
