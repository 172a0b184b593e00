// Dense warp-tile walk of the index build: every (state, token) pair is walked.
// One warp owns 32 consecutive tokens (lane = token) and a run of 32 states; the
// compressed table - or, when it does not fit, a tile of start-state rows - is staged in
// shared memory by bulk async copy; a warp ballot gives each bitmask word and the end
// states go out as one coalesced store per state.
#pragma once

#include "fsm_index_common.cuh"

namespace fsm {
namespace {

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
template <typename TabT, typename OutT, bool HAS_OUT, bool FULL, bool HAS_EOS>
__device__ __forceinline__ void walk_task(const WalkParams& p, const TabT* __restrict__ first,
                                          const TabT* __restrict__ tab, int Cs, int q0, int nq,
                                          int g, int lane) {
    const int v = g * 32 + lane;
    const uint4 tk = p.tok_cls[v];
    const int len = p.tok_len[v];
    const uint32_t dead = p.dead;
    const bool multi = len > 1;
    const bool eos_lane = HAS_EOS && (v == p.eos_id);
    const bool store_ok = HAS_OUT && (v < p.N);
    const bool class_ok = idx_ok(tk.x & 0xFFu, Cs, p.status);  // (first byte's class: a column)
    const TabT* f = first + (class_ok ? (tk.x & 0xFFu) : 0u);
    const size_t r0 = static_cast<size_t>(q0 - p.q_begin);
    OutT* outp = HAS_OUT ? static_cast<OutT*>(p.next) + r0 * p.N + v : nullptr;
    uint32_t* mp = p.mask + r0 * p.G + g;
    for (int j = 0; j < nq; ++j) {
        uint32_t s = class_ok ? static_cast<uint32_t>(*f) : dead;
        bool go = multi && (s != dead);
        s = walk_rest<TabT, FULL, 1>(tab, Cs, dead, tk, len, s, go, static_cast<uint32_t>(p.Q) * Cs, p.status);
        if (go)  // longer than the inline record and still alive: finish on the raw bytes
            s = raw_walk(p, s, p.vocab_offsets[v], p.vocab_offsets[v + 1], kInlineBytes);
        if (HAS_EOS) {
            const int q = q0 + j;
            if (eos_lane) s = (q != p.dead && p.accept[q]) ? q : dead;
        }
        if (store_ok) *outp = static_cast<OutT>(s);
        const uint32_t word = __ballot_sync(kFullWarp, s != dead);
        if (lane == 0) *mp = word;
        f += Cs;
        if (HAS_OUT) outp += p.N;
        mp += p.G;
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

// CHUNK: states per warp task.  kChunk as a rule; kSmallChunk for a build so small that the
// device's warps would not get two tasks each (a task walks its states one after the other,
// so its length is latency).  kSmallChunk divides kChunk: tiles still start on a chunk.
template <typename TabT, typename OutT, bool HAS_OUT, int CHUNK>
__global__ void __launch_bounds__(kWalkThreads, 1) walk(const WalkParams p) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    __shared__ uint64_t bar;
    TabT* tile = reinterpret_cast<TabT*>(smem_raw);
    const TabT* gtab = static_cast<const TabT*>(p.table);
    const int Cs = p.meta->Cs;
    const bool raw = p.meta->any_bad != 0;
    const uint32_t row_bytes = Cs * sizeof(TabT);
    const int nrows = p.q_end - p.q_begin;
    // Four rows are a multiple of 16 bytes (the row stride is an odd number of words): a
    // tile starts at a row that is a multiple of four, and its size is rounded up to 16 bytes.
    const uint32_t tile_cap = p.smem_cap - 16;
    const bool full = static_cast<uint64_t>(p.Q) * row_bytes <= tile_cap;
    const int cap_rows = max(kChunk, (static_cast<int>(tile_cap / row_bytes) - 3) / kChunk * kChunk);
    const int ntiles = full ? 1 : (nrows + cap_rows - 1) / cap_rows;
    const int lane = threadIdx.x & 31;
    // warp w of CTA b starts at task w * gridDim.x + b: a build with fewer tasks than warps
    // on the device still spreads over all the SMs
    const int64_t wg = static_cast<int64_t>(threadIdx.x >> 5) * gridDim.x + blockIdx.x;
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
        const int t_s0 = t_q0 & ~3;                                     // first row in the tile
        const int w_q0 = full ? p.q_begin : t_q0;                       // first start state
        const int w_rows = full ? nrows : t_rows;
        if (!raw) {
            if (ti > 0) __syncthreads();  // every warp is done with the previous tile
            if (threadIdx.x == 0) {
                const uint32_t bytes =
                    (static_cast<uint32_t>(t_q0 - t_s0 + t_rows) * row_bytes + 15u) / 16u * 16u;
                const uint8_t* src =
                    reinterpret_cast<const uint8_t*>(gtab) + static_cast<size_t>(t_s0) * row_bytes;
                mbar_expect_tx(&bar, bytes);
                for (uint32_t o = 0; o < bytes; o += kBulkChunk)
                    bulk_copy_g2s(smem_raw + o, src + o, min(kBulkChunk, bytes - o), &bar);
            }
            bool ok = mbar_wait_bounded(&bar, parity);
            if (!ok) ok = mbar_wait_bounded(&bar, parity);  // drain before giving up
            if (ok && p.wait_probe > 0)  // the phase after this one: nothing completes it
                ok = mbar_wait_bounded(&bar, parity ^ 1, p.wait_probe);
            parity ^= 1;
            if (!__syncthreads_and(ok)) {
                if (threadIdx.x == 0) raise_flag(p.status, FSM_FLAG_WAIT_TIMEOUT);
                return;
            }
        }
        const int nchunks = (w_rows + CHUNK - 1) / CHUNK;
        const int64_t ntasks = static_cast<int64_t>(nchunks) * p.G;
        for (int64_t t = wg; t < ntasks; t += TW) {
            const int chunk = static_cast<int>(t / p.G);
            const int g = static_cast<int>(t - static_cast<int64_t>(chunk) * p.G);
            const int q0 = w_q0 + chunk * CHUNK;
            const int nq = min(CHUNK, w_q0 + w_rows - q0);
            if (raw) {
                walk_task_raw<OutT, HAS_OUT>(p, q0, nq, g, lane);
            } else {
                const TabT* first = tile + static_cast<size_t>(q0 - t_s0) * Cs;
                const bool has_eos = (p.eos_id >= 0) && ((p.eos_id >> 5) == g);
                if (has_eos) {  // rare: one group in the whole vocabulary
                    if (full)
                        walk_task<TabT, OutT, HAS_OUT, true, true>(p, first, tile, Cs, q0, nq, g, lane);
                    else
                        walk_task<TabT, OutT, HAS_OUT, false, true>(p, first, gtab, Cs, q0, nq, g, lane);
                } else if (full) {
                    walk_task<TabT, OutT, HAS_OUT, true, false>(p, first, tile, Cs, q0, nq, g, lane);
                } else {
                    walk_task<TabT, OutT, HAS_OUT, false, false>(p, first, gtab, Cs, q0, nq, g, lane);
                }
            }
        }
    }
}


template <typename TabT, typename OutT, bool HAS_OUT>
cudaError_t launch_walk(const WalkParams& p, int grid, cudaStream_t stream) {
    auto kernel = p.chunk == kSmallChunk ? walk<TabT, OutT, HAS_OUT, kSmallChunk>
                                         : walk<TabT, OutT, HAS_OUT, kChunk>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(p.smem_cap));
    if (e != cudaSuccess) return e;
    return launch_on(kernel, dim3(grid), dim3(kWalkThreads), p.smem_cap, stream, p);
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
