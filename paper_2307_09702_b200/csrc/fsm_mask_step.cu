// Masked decode step (paper Algorithm 2) for sm_100a: greedy selection (Section 2.1) or
// the categorical draw of Algorithm 2 itself, as a Gumbel-max over the allowed tokens.
//
// One thread-block cluster of `k` CTAs owns one logits row.  Each thread streams
// 32-byte vectors of the row: it first reads the vector's bits of the allowed-token
// bitmask row sigma(state) (L2 resident), loads the logits only when at least one
// bit is set (a vector with no allowed token becomes -inf whatever it held), writes
// the masked vector and keeps a running (value, lowest id) maximum over the allowed
// entries.  The maxima are reduced by warp shuffles, through shared memory, and
// across the cluster through distributed shared memory; the cluster's first CTA
// then looks up the next state and updates states / finished / tokens_out.
#include <cooperative_groups.h>

#include "fsm_common.cuh"

namespace cg = cooperative_groups;

namespace fsm {
namespace {

constexpr int kStepThreads = 256;
constexpr int kStepWarps = kStepThreads / 32;
constexpr int kNone = 0x7FFFFFFF;

struct StepParams {
    const void* in;
    void* out;
    int64_t row_stride;
    int32_t* states;
    uint8_t* finished;
    int32_t* tokens;
    const uint32_t* mask;
    const void* next;
    int32_t state_u16;
    int32_t Q, N, W, B, dead, eos_id, k;
    int32_t* status;
    // compressed-row index (csr_offsets != nullptr): next states by search in the row
    const int64_t* csr_offsets;
    const int32_t* csr_tokens;
    const int32_t* csr_next;
    int64_t csr_capacity;  // entries the two arrays hold
    // sampling
    float inv_temperature;
    uint32_t seed_lo, seed_hi, draw_lo, draw_hi;
};

struct Best {
    float val;
    int idx;
};

// `b` replaces `a` when it is the better candidate: larger value, or equal value
// and lower id; kNone marks "no allowed token seen".
__device__ __forceinline__ Best better(Best a, Best b) {
    const bool take = (b.idx != kNone) &&
                      (a.idx == kNone || b.val > a.val || (b.val == a.val && b.idx < a.idx));
    return take ? b : a;
}

template <typename T> struct Elem;
template <> struct Elem<uint32_t> {  // fp32 bit patterns
    static constexpr int kPerWord = 1;
    static constexpr uint32_t kNegInfWord = 0xFF800000u;
    __device__ static float get(uint32_t w, int) { return __uint_as_float(w); }
    // keeps the allowed element, -inf otherwise
    __device__ static uint32_t select(uint32_t w, uint32_t bits) { return (bits & 1u) ? w : kNegInfWord; }
    // largest value of a masked vector of NW words
    template <int NW>
    __device__ static float vmax(const uint32_t (&w)[NW]) {
        float m = __uint_as_float(w[0]);
#pragma unroll
        for (int i = 1; i < NW; ++i) m = fmaxf(m, __uint_as_float(w[i]));
        return m;
    }
};
template <> struct Elem<uint16_t> {  // bf16 bit patterns, two per word
    static constexpr int kPerWord = 2;
    static constexpr uint32_t kNegInfWord = 0xFF80FF80u;
    __device__ static float get(uint32_t w, int j) { return __uint_as_float(j ? (w & 0xFFFF0000u) : (w << 16)); }
    // one byte permute per word: allowed halves come from w, the others from -inf
    __device__ static uint32_t select(uint32_t w, uint32_t bits) {
        const uint32_t sel = 0x7654u ^ ((bits & 1u) * 0x0044u) ^ ((bits & 2u) * 0x2200u);
        return __byte_perm(w, kNegInfWord, sel);
    }
    template <int NW>
    __device__ static float vmax(const uint32_t (&w)[NW]) {
        uint32_t m = w[0];
#pragma unroll
        for (int i = 1; i < NW; ++i) asm("max.bf16x2 %0, %0, %1;" : "+r"(m) : "r"(w[i]));
        return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
    }
};

// Running maximum of one thread.  The position inside the winning vector is not
// tracked while streaming: the vector's index and bitmask bits are kept and the
// position is found once, at the end (see locate()).
struct ThreadBest {
    float val;      // NaN until the first vector with an allowed entry
    int vec;        // index of the vector that holds it, -1 = none
    uint32_t bits;  // allowed bits of that vector
};

// Masks one vector of NW words in place and folds its maximum into `tb`.
template <typename T, int NW>
__device__ __forceinline__ void process(uint32_t (&w)[NW], uint32_t bits, int vec, ThreadBest& tb) {
    constexpr int PW = Elem<T>::kPerWord;
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = Elem<T>::select(w[i], (bits >> (i * PW)) & ((1u << PW) - 1u));
    const float m = Elem<T>::template vmax<NW>(w);
    if (!(m <= tb.val)) {  // strictly larger, or the first allowed entries (val is NaN)
        tb.val = m;
        tb.vec = vec;
        tb.bits = bits;
    }
}

// Lowest allowed position of a vector whose value equals `val` (IEEE equality).
template <typename T, int NW>
__device__ __forceinline__ int locate(const uint32_t (&w)[NW], uint32_t bits, float val) {
    constexpr int PW = Elem<T>::kPerWord;
    int pos = NW * PW;
#pragma unroll
    for (int j = NW * PW - 1; j >= 0; --j)
        if (((bits >> j) & 1u) && Elem<T>::get(w[j / PW], j % PW) == val) pos = j;
    return pos;
}

// ---------------------------------------------------------------------------------------
// Categorical draw (Algorithm 2): argmax over the allowed tokens of
// logit / temperature + G with G a standard Gumbel variate.  The random bits come from
// Philox4x32-10 (Salmon et al., SC'11) with key = seed and counter = (token id / 4, batch
// row, draw number); token v uses output word v % 4.  Every floating-point step is an
// explicitly rounded fp32 operation and the library is built without flush-to-zero, so
// subnormal logits take part in the score as they are.
__device__ __forceinline__ uint32_t philox_word(uint32_t v, uint32_t row, const StepParams& p) {
    uint32_t c0 = v >> 2, c1 = row, c2 = p.draw_lo, c3 = p.draw_hi;
    uint32_t k0 = p.seed_lo, k1 = p.seed_hi;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const unsigned long long a = static_cast<unsigned long long>(c0) * 0xD2511F53ull;
        const unsigned long long b = static_cast<unsigned long long>(c2) * 0xCD9E8D57ull;
        c0 = static_cast<uint32_t>(b >> 32) ^ c1 ^ k0;
        c2 = static_cast<uint32_t>(a >> 32) ^ c3 ^ k1;
        c1 = static_cast<uint32_t>(b);
        c3 = static_cast<uint32_t>(a);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    const uint32_t sel = v & 3u;
    return sel == 0 ? c0 : sel == 1 ? c1 : sel == 2 ? c2 : c3;
}

// ln x of a positive normal x: x = m 2^e with m in (sqrt(1/2), sqrt(2)], s = (m-1)/(m+1),
// ln m = 2 s (1 + s^2/3 + s^4/5 + s^6/7 + s^8/9) by Horner's rule.
__device__ __forceinline__ float ln_rn(float x) {
    const uint32_t b = __float_as_uint(x);
    int e = static_cast<int>(b >> 23) - 127;
    float m = __uint_as_float((b & 0x007FFFFFu) | 0x3F800000u);
    if (m > 1.41421354f) {
        m = __fmul_rn(m, 0.5f);
        e += 1;
    }
    const float s = __fdiv_rn(__fadd_rn(m, -1.0f), __fadd_rn(m, 1.0f));
    const float z = __fmul_rn(s, s);
    float t = __fmaf_rn(z, 1.0f / 9.0f, 1.0f / 7.0f);
    t = __fmaf_rn(z, t, 1.0f / 5.0f);
    t = __fmaf_rn(z, t, 1.0f / 3.0f);
    t = __fmaf_rn(z, t, 1.0f);
    return __fmaf_rn(static_cast<float>(e), 0.693147182f, __fmul_rn(__fadd_rn(s, s), t));
}

__device__ __forceinline__ float gumbel_score(float x, uint32_t v, uint32_t row, const StepParams& p) {
    const uint32_t bits = philox_word(v, row, p);
    // u: an odd multiple of 2^-24 strictly inside (0, 1)
    const float u = __fmul_rn(static_cast<float>(2u * (bits >> 9) + 1u), 5.9604644775390625e-08f);
    const float y = -ln_rn(u);
    return __fmaf_rn(x, p.inv_temperature, -ln_rn(y));
}

// The better candidate has the larger score, or an equal score and the lower id (whatever
// the visiting order).
__device__ __forceinline__ void take_better(Best& a, float score, int id) {
    if (a.idx == kNone || score > a.val || (score == a.val && id < a.idx)) {
        a.val = score;
        a.idx = id;
    }
}

// Scores the allowed entries of one vector on the spot (rows that are not 32-byte aligned).
template <typename T, int NW>
__device__ __forceinline__ void score_vector(const uint32_t (&w)[NW], uint32_t bits, int first_id,
                                             uint32_t row, const StepParams& p, Best& best) {
    constexpr int PW = Elem<T>::kPerWord;
    uint32_t todo = bits;
    while (todo) {
        const int j = __ffs(todo) - 1;
        todo &= todo - 1;
        uint32_t word = w[0];
#pragma unroll
        for (int i = 1; i < NW; ++i) word = (j / PW == i) ? w[i] : word;
        take_better(best, gumbel_score(Elem<T>::get(word, j % PW), first_id + j, row, p), first_id + j);
    }
}

template <typename T, int NW>
__device__ __forceinline__ void mask_vector(uint32_t (&w)[NW], uint32_t bits) {
    constexpr int PW = Elem<T>::kPerWord;
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = Elem<T>::select(w[i], (bits >> (i * PW)) & ((1u << PW) - 1u));
}

// Pool of allowed entries of one warp.  Few entries of a vector are allowed (one in
// eighteen in the benchmark's index), so scoring them lane by lane would run the draw with
// most lanes idle; instead every lane appends the ids of its allowed entries to the warp's
// queue and the warp scores 32 queued entries at a time, each lane fetching its entry's
// logit again by id (the row was read a moment ago: an L2 hit, and one instruction instead
// of picking the value out of the vector's registers).  kQueue holds the leftovers of one round
// (< 32) plus every entry of one 32-byte vector per lane (at most 16 bf16 values).
constexpr int kQueue = 32 + 16 * 32;
struct WarpQueue {
    int id[kQueue];
};

// The logit of token `id` as fp32 (allowed entries are the same in the input and in the
// masked output, so reading the input is right even while the row is being rewritten).
template <typename T>
__device__ __forceinline__ float logit_of(const T* in, int id) {
    const T raw = in[id];
    return sizeof(T) == 4 ? __uint_as_float(static_cast<uint32_t>(raw))
                          : __uint_as_float(static_cast<uint32_t>(raw) << 16);
}

// The queues of a CTA; the greedy variant has none.
template <bool SAMPLE> struct QueueStore {
    __device__ static WarpQueue* get() {
        __shared__ WarpQueue queues[kStepWarps];
        return queues;
    }
};
template <> struct QueueStore<false> {
    __device__ static WarpQueue* get() { return nullptr; }
};

// All 32 lanes call this with the allowed bits of their vector (0: nothing to add).
template <typename T>
__device__ __forceinline__ void pool_vector(uint32_t bits, int first_id, const T* in, uint32_t row,
                                            const StepParams& p, WarpQueue& q, int& qn, Best& best) {
    const int lane = threadIdx.x & 31;
    const int mine = __popc(bits);
    int incl = mine;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(kFullWarp, incl, off);
        if (lane >= off) incl += o;
    }
    const int total = __shfl_sync(kFullWarp, incl, 31);
    if (total == 0) return;
    int at = qn + incl - mine;
    for (uint32_t todo = bits; todo != 0; todo &= todo - 1, ++at)
        if (idx_ok(at, kQueue, p.status)) q.id[at] = first_id + __ffs(todo) - 1;
    qn += total;
    __syncwarp();
    int head = 0;
    for (; qn - head >= 32; head += 32) {
        const int id = q.id[head + lane];
        if (idx_ok(id, p.N, p.status)) take_better(best, gumbel_score(logit_of(in, id), id, row, p), id);
    }
    if (head > 0) {  // leftovers to the front
        const int rem = qn - head;
        int id = 0;
        if (lane < rem) id = q.id[head + lane];
        __syncwarp();
        if (lane < rem) q.id[lane] = id;
        qn = rem;
    }
    __syncwarp();
}

template <typename T, bool WRITE, bool SAMPLE>
__global__ void __launch_bounds__(kStepThreads) mask_step(const StepParams p) {
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ Best warp_best[kStepWarps];
    __shared__ Best cta_best[8];  // slot r of the cluster's first CTA receives CTA r's result

    const int k = p.k;
    const int row = blockIdx.x / k;
    const int rank = blockIdx.x - row * k;  // == cluster.block_rank() for 1-D clusters
    // Uniform over the cluster: nobody reaches the cluster barrier for a finished row.
    if (p.finished[row] != 0) {
        if (rank == 0 && threadIdx.x == 0) p.tokens[row] = -1;
        return;
    }
    int q = p.states[row];
    const bool bad_state = static_cast<uint32_t>(q) >= static_cast<uint32_t>(p.Q);
    const uint32_t* mrow = p.mask + static_cast<size_t>(bad_state ? 0 : q) * p.W;
    const uint32_t live = bad_state ? 0u : 0xFFFFFFFFu;

    constexpr int EPV = 32 / sizeof(T);   // elements per 32-byte vector
    constexpr int EPH = 16 / sizeof(T);   // elements per 16-byte vector
    const T* in = static_cast<const T*>(p.in) + static_cast<size_t>(row) * p.row_stride;
    T* out = WRITE ? static_cast<T*>(p.out) + static_cast<size_t>(row) * p.row_stride : nullptr;
    const bool wide = ((reinterpret_cast<uintptr_t>(in) | (WRITE ? reinterpret_cast<uintptr_t>(out) : 0)) & 31) == 0;

    ThreadBest tb{__int_as_float(0x7FC00000), -1, 0u};
    Best best{0.0f, kNone};
    const int tid = rank * kStepThreads + threadIdx.x;
    const int nthreads = k * kStepThreads;

    int done = 0;  // elements covered by whole vectors
    if (wide) {
        // Per thread and pass: the bitmask bits of kGroup vectors are fetched first (one
        // round trip to L2), then the vectors are streamed kUnroll at a time - every needed
        // logits load of a batch is issued before any arithmetic.  Two loads in flight per
        // thread keep the greedy kernel at 48 registers (five CTAs per SM), which measured
        // faster than four or eight loads at 80 to 160 registers.
        constexpr int kUnroll = 2, kGroup = 4;
        const int nvec = p.N / EPV;
        constexpr uint32_t kBitsMask = (EPV == 32) ? 0xFFFFFFFFu : ((1u << EPV) - 1u);
        WarpQueue& queue = QueueStore<SAMPLE>::get()[SAMPLE ? (threadIdx.x >> 5) : 0];
        int qn = 0;
        // (the bound is the same for the 32 lanes of a warp: the pooled draw is a warp-wide step)
        for (int g0 = tid; g0 - (SAMPLE ? static_cast<int>(threadIdx.x & 31) : 0) < nvec;
             g0 += nthreads * kGroup) {
            uint32_t bits[kGroup];
#pragma unroll
            for (int u = 0; u < kGroup; ++u) {
                const int vi = g0 + u * nthreads;
                const int e0 = vi * EPV;
                bits[u] = vi < nvec ? (live & (__ldg(mrow + (e0 >> 5)) >> (e0 & 31)) & kBitsMask) : 0u;
            }
#pragma unroll
            for (int h = 0; h < kGroup; h += kUnroll) {
                Vec32B v[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u)
                    if (bits[h + u] != 0)
                        v[u] = ldg_stream_32B(in + static_cast<size_t>(g0 + (h + u) * nthreads) * EPV);
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    const int vi = g0 + (h + u) * nthreads;
                    if (SAMPLE) pool_vector<T>(bits[h + u], vi * EPV, in, row, p, queue, qn, best);
                    if (vi < nvec) {
                        if (bits[h + u] != 0) {
                            if (SAMPLE)
                                mask_vector<T, 8>(v[u].w, bits[h + u]);
                            else
                                process<T, 8>(v[u].w, bits[h + u], vi, tb);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) v[u].w[i] = Elem<T>::kNegInfWord;
                        }
                        if (WRITE) stg_32B(out + static_cast<size_t>(vi) * EPV, v[u]);
                    }
                }
            }
        }
        if (SAMPLE && static_cast<int>(threadIdx.x & 31) < qn) {  // what is left in the pool
            const int id = queue.id[threadIdx.x & 31];
            take_better(best, gumbel_score(logit_of(in, id), id, row, p), id);
        }
        done = nvec * EPV;
    } else {
        const int nvec = p.N / EPH;
        for (int vi = tid; vi < nvec; vi += nthreads) {
            const int e0 = vi * EPH;
            const uint32_t bits = live & (mrow[e0 >> 5] >> (e0 & 31)) & ((1u << EPH) - 1u);
            uint32_t w[4];
            if (bits != 0) {
                const uint4 v = *reinterpret_cast<const uint4*>(in + e0);
                w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
                if (SAMPLE) {
                    score_vector<T, 4>(w, bits, e0, row, p, best);
                    mask_vector<T, 4>(w, bits);
                } else {
                    process<T, 4>(w, bits, vi, tb);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = Elem<T>::kNegInfWord;
            }
            if (WRITE) *reinterpret_cast<uint4*>(out + e0) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        done = nvec * EPH;
    }
    // Position of the thread's maximum: re-read the winning vector (the allowed entries
    // are unchanged by the masking, wherever it was written) and take the lowest
    // allowed position that holds the value.
    if (!SAMPLE && tb.vec >= 0) {
        const T* src = (WRITE ? static_cast<const T*>(out) : in);
        best.val = tb.val;
        if (wide) {
            Vec32B v = ldg_stream_32B(src + static_cast<size_t>(tb.vec) * EPV);
            best.idx = tb.vec * EPV + locate<T, 8>(v.w, tb.bits, tb.val);
        } else {
            const uint4 v = *reinterpret_cast<const uint4*>(src + static_cast<size_t>(tb.vec) * EPH);
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
            best.idx = tb.vec * EPH + locate<T, 4>(w, tb.bits, tb.val);
        }
    }
    // Ragged tail (fewer elements than one vector): one element per thread of the last CTA.
    if (rank == k - 1) {
        const int e = done + threadIdx.x;
        if (e < p.N) {
            const bool allowed = (live & (mrow[e >> 5] >> (e & 31)) & 1u) != 0;
            const T raw = in[e];
            if (allowed) {
                float x = sizeof(T) == 4 ? __uint_as_float(static_cast<uint32_t>(raw))
                                         : __uint_as_float(static_cast<uint32_t>(raw) << 16);
                if (SAMPLE) {
                    take_better(best, gumbel_score(x, e, row, p), e);
                } else if (best.idx == kNone || x > best.val) {  // tail ids exceed every vector id
                    best.val = x;
                    best.idx = e;
                }
            } else if (WRITE) {
                out[e] = static_cast<T>(sizeof(T) == 4 ? 0xFF800000u : 0xFF80u);
            }
            if (allowed && WRITE) out[e] = raw;
        }
    }

    // A thread's own ids only grow, so its (val, idx) already holds the lowest id
    // among equal values; combining needs the full ordering.
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Best o;
        o.val = __shfl_xor_sync(kFullWarp, best.val, off);
        o.idx = __shfl_xor_sync(kFullWarp, best.idx, off);
        best = better(best, o);
    }
    if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        Best b = warp_best[0];
#pragma unroll
        for (int i = 1; i < kStepWarps; ++i) b = better(b, warp_best[i]);
        Best* dst = (k > 1) ? cluster.map_shared_rank(&cta_best[rank], 0) : &cta_best[0];
        *dst = b;
    }
    if (k > 1) cluster.sync();
    if (rank == 0 && threadIdx.x == 0) {
        Best b = cta_best[0];
        for (int i = 1; i < k; ++i) b = better(b, cta_best[i]);
        if (bad_state) raise_flag(p.status, FSM_FLAG_STATE_RANGE);
        if (b.idx == kNone) {
            p.finished[row] = 2;
            p.tokens[row] = -1;
        } else if (b.idx == p.eos_id) {
            p.finished[row] = 1;
            p.tokens[row] = b.idx;
        } else if (!idx_ok(b.idx, p.N, p.status)) {
            p.finished[row] = 2;  // (range-checked build only: a winner outside the vocabulary)
            p.tokens[row] = -1;
        } else {
            p.tokens[row] = b.idx;
            if (p.csr_offsets != nullptr) {
                // the row's tokens are in increasing order: binary search for the chosen one.
                // row_offsets is complete even when the index has more entries than the arrays
                // hold, so the search stays inside the part that exists.
                const int64_t cap = p.csr_capacity;
                int64_t lo = min(max(p.csr_offsets[q], static_cast<int64_t>(0)), cap);
                const int64_t end = min(max(p.csr_offsets[q + 1], lo), cap);
                int64_t hi = end;
                while (lo < hi) {
                    const int64_t mid = (lo + hi) >> 1;
                    if (p.csr_tokens[mid] < b.idx)
                        lo = mid + 1;
                    else
                        hi = mid;
                }
                const bool found = lo < end && p.csr_tokens[lo] == b.idx;
                p.states[row] = found ? p.csr_next[lo] : p.dead;  // (an entry lost to a too small
                                                                  // capacity leads to dead)
            } else {
                const size_t at = static_cast<size_t>(q) * p.N + b.idx;
                p.states[row] = p.state_u16 ? static_cast<int32_t>(static_cast<const uint16_t*>(p.next)[at])
                                            : static_cast<const int32_t*>(p.next)[at];
            }
        }
    }
}

template <typename T, bool WRITE, bool SAMPLE>
cudaError_t launch(const StepParams& p, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.B) * p.k, 1, 1);
    cfg.blockDim = dim3(kStepThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = p.k;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, mask_step<T, WRITE, SAMPLE>, p);
}

}  // namespace
}  // namespace fsm

namespace {
int step_impl(const void* logits_in, void* logits_out, int32_t logits_dtype, int64_t row_stride,
              int32_t* states, uint8_t* finished, int32_t* tokens_out,
              const uint32_t* allowed_mask, const void* next_state, int32_t state_dtype, int32_t Q,
              int32_t N, int32_t B, int32_t dead_state, int32_t eos_id, bool sample,
              float inv_temperature, uint64_t seed, uint64_t draw, int32_t* status_word,
              void* cuda_stream, const int64_t* csr_offsets = nullptr,
              const int32_t* csr_tokens = nullptr, const int32_t* csr_next = nullptr,
              int64_t csr_capacity = 0) {
    using namespace fsm;
    if (Q <= 0 || N <= 0 || B < 0 || row_stride < N) return FSM_ERR_SHAPE;
    if (!logits_in || !states || !finished || !tokens_out || !allowed_mask) return FSM_ERR_NULL;
    if (csr_offsets ? (csr_capacity > 0 && (!csr_tokens || !csr_next)) : !next_state) return FSM_ERR_NULL;
    if (csr_capacity < 0) return FSM_ERR_SHAPE;
    if (logits_dtype != FSM_LOGITS_F32 && logits_dtype != FSM_LOGITS_BF16) return FSM_ERR_DTYPE;
    if (state_dtype != FSM_STATE_I32 && state_dtype != FSM_STATE_U16) return FSM_ERR_DTYPE;
    if (state_dtype == FSM_STATE_U16 && Q > 65535) return FSM_ERR_DTYPE;
    if (dead_state < 0 || dead_state >= Q || eos_id < -1 || eos_id >= N) return FSM_ERR_RANGE;
    const size_t esize = logits_dtype == FSM_LOGITS_F32 ? 4 : 2;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(logits_in, 16) || misaligned(logits_out, 16) ||
        (static_cast<uint64_t>(row_stride) * esize) % 16 != 0)
        return FSM_ERR_ALIGN;
    if (misaligned(states, 4) || misaligned(tokens_out, 4) || misaligned(allowed_mask, 4) ||
        misaligned(next_state, state_dtype == FSM_STATE_U16 ? 2 : 4) || misaligned(status_word, 4))
        return FSM_ERR_ALIGN;
    if (static_cast<int64_t>(B) * 8 > 0x7FFFFFFF) return FSM_ERR_SHAPE;
    if (B == 0) return FSM_OK;

    const DeviceInfo& dev = device_info();
    if (!dev.ok) return FSM_ERR_CUDA;
    if (dev.cc_major != 10) return FSM_ERR_DEVICE;

    // CTAs per row: the smallest cluster that gives at least three CTAs per SM (four fit, by
    // registers, so the whole grid is resident at once), but at least a few vectors per
    // thread.  Measured at B = 256, N = 128,256, bf16: 32.9 / 26.9 / 29.3 us with 1 / 2 / 4.
    // The categorical draw is bound by instruction issue and its CTAs differ in length (the
    // work follows the allowed tokens), so it takes CTAs half as long, which fill the SMs
    // more evenly as they come and go: 72.1 / 52.0 / 46.7 / 47.0 us with 1 / 2 / 4 / 8.
    int k = tunables().mask_cluster;
    if (k != 1 && k != 2 && k != 4 && k != 8) {
        k = 1;
        const int64_t vectors = static_cast<int64_t>(N) * esize / 32;
        const int64_t ctas_wanted = (sample ? 6LL : 3LL) * dev.sm_count;
        while (k < 8 && static_cast<int64_t>(B) * k < ctas_wanted &&
               vectors / (2 * k * kStepThreads) >= 2)
            k *= 2;
        // A grid of between one and two and a half waves ends with a thin last wave, which
        // costs the more the longer a CTA runs: CTAs of twelve or more vectors per thread
        // are halved until there are more waves (B = 1,024: 96 -> 90 us greedy, 155 -> 137 us
        // drawn).
        const int64_t places = static_cast<int64_t>(dev.sm_count) * (sample ? 4 : 5);  // resident CTAs
        while (k < 8 && static_cast<int64_t>(B) * k > places &&
               2 * static_cast<int64_t>(B) * k < 5 * places && vectors / (k * kStepThreads) >= 12)
            k *= 2;
    }

    StepParams p;
    p.in = logits_in;
    p.out = logits_out;
    p.row_stride = row_stride;
    p.states = states;
    p.finished = finished;
    p.tokens = tokens_out;
    p.mask = allowed_mask;
    p.next = next_state;
    p.state_u16 = state_dtype == FSM_STATE_U16;
    p.Q = Q;
    p.N = N;
    p.W = (N + 31) / 32;
    p.B = B;
    p.dead = dead_state;
    p.eos_id = eos_id;
    p.k = k;
    p.status = status_word;
    p.csr_offsets = csr_offsets;
    p.csr_tokens = csr_tokens;
    p.csr_next = csr_next;
    p.csr_capacity = csr_capacity;
    p.inv_temperature = inv_temperature;
    p.seed_lo = static_cast<uint32_t>(seed);
    p.seed_hi = static_cast<uint32_t>(seed >> 32);
    p.draw_lo = static_cast<uint32_t>(draw);
    p.draw_hi = static_cast<uint32_t>(draw >> 32);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    const bool write = logits_out != nullptr;
    if (sample) {
        if (logits_dtype == FSM_LOGITS_F32)
            e = write ? launch<uint32_t, true, true>(p, stream) : launch<uint32_t, false, true>(p, stream);
        else
            e = write ? launch<uint16_t, true, true>(p, stream) : launch<uint16_t, false, true>(p, stream);
    } else if (logits_dtype == FSM_LOGITS_F32) {
        e = write ? launch<uint32_t, true, false>(p, stream) : launch<uint32_t, false, false>(p, stream);
    } else {
        e = write ? launch<uint16_t, true, false>(p, stream) : launch<uint16_t, false, false>(p, stream);
    }
    return e == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
}
}  // namespace

extern "C" int guided_mask_step(const void* logits_in, void* logits_out, int32_t logits_dtype,
                                int64_t row_stride, int32_t* states, uint8_t* finished,
                                int32_t* tokens_out, const uint32_t* allowed_mask,
                                const void* next_state, int32_t state_dtype, int32_t Q, int32_t N,
                                int32_t B, int32_t dead_state, int32_t eos_id,
                                int32_t* status_word, void* cuda_stream) {
    return step_impl(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                     allowed_mask, next_state, state_dtype, Q, N, B, dead_state, eos_id, false, 1.0f,
                     0, 0, status_word, cuda_stream);
}

extern "C" int guided_sample_step(const void* logits_in, void* logits_out, int32_t logits_dtype,
                                  int64_t row_stride, int32_t* states, uint8_t* finished,
                                  int32_t* tokens_out, const uint32_t* allowed_mask,
                                  const void* next_state, int32_t state_dtype, int32_t Q,
                                  int32_t N, int32_t B, int32_t dead_state, int32_t eos_id,
                                  float inv_temperature, uint64_t seed, uint64_t draw,
                                  int32_t* status_word, void* cuda_stream) {
    if (!(inv_temperature > 0.0f) || !(inv_temperature < 3.0e38f)) return FSM_ERR_RANGE;
    return step_impl(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                     allowed_mask, next_state, state_dtype, Q, N, B, dead_state, eos_id, true,
                     inv_temperature, seed, draw, status_word, cuda_stream);
}

extern "C" int guided_step_csr(const void* logits_in, void* logits_out, int32_t logits_dtype,
                               int64_t row_stride, int32_t* states, uint8_t* finished,
                               int32_t* tokens_out, const uint32_t* allowed_mask,
                               const int64_t* row_offsets, const int32_t* csr_tokens,
                               const int32_t* csr_next, int64_t capacity, int32_t Q, int32_t N,
                               int32_t B, int32_t dead_state, int32_t eos_id, int32_t sample,
                               float inv_temperature, uint64_t seed, uint64_t draw,
                               int32_t* status_word, void* cuda_stream) {
    if (!row_offsets) return FSM_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(row_offsets) % 8 != 0 ||
        reinterpret_cast<uintptr_t>(csr_tokens) % 4 != 0 || reinterpret_cast<uintptr_t>(csr_next) % 4 != 0)
        return FSM_ERR_ALIGN;
    if (sample && (!(inv_temperature > 0.0f) || !(inv_temperature < 3.0e38f))) return FSM_ERR_RANGE;
    return step_impl(logits_in, logits_out, logits_dtype, row_stride, states, finished, tokens_out,
                     allowed_mask, nullptr, FSM_STATE_I32, Q, N, B, dead_state, eos_id, sample != 0,
                     sample ? inv_temperature : 1.0f, seed, draw, status_word, cuda_stream,
                     row_offsets, csr_tokens, csr_next, capacity);
}
