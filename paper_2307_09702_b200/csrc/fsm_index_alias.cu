// Merging of identical index rows.  The paper's index maps a state to its set of allowed
// tokens (Section 3, Algorithm 4) and is built from automata that are not reduced (Section
// 5), so different states can carry the same row.  row_alias[q] = the smallest state whose
// row - bitmask words and, when a next-state table is given, every end state - equals q's.
//
//   alias_hash    a 64-bit hash per row (block = row; wrap-around sums of mixed
//                 (position, value) pairs, so the threads' partial sums simply add and the
//                 hash does not depend on how a row happens to be aligned in memory)
//   alias_group   rows with equal hashes meet in an open-addressing table; the smallest row
//                 of each hash value becomes the candidate of the others
//   alias_verify  exact comparison with the candidate (block = row).  A row that differs
//                 from its candidate although the hashes agree compares itself with every
//                 earlier row of the same hash, so the result never depends on the hash.
#include "fsm_common.cuh"

namespace fsm {
namespace {

constexpr int kAliasThreads = 512;
constexpr unsigned long long kEmptyKey = ~0ull;

struct AliasWorkspace {
    unsigned long long* hash;  // [Q]
    unsigned long long* keys;  // [slots]
    int32_t* min_row;          // [slots]
    int32_t* slot_of;          // [Q]
    uint32_t slots;            // power of two >= 2Q
    size_t bytes;
};

AliasWorkspace carve_alias(void* base, int32_t Q) {
    AliasWorkspace w;
    uint32_t slots = 64;
    while (slots < 2u * static_cast<uint32_t>(Q)) slots <<= 1;
    w.slots = slots;
    uint8_t* p = static_cast<uint8_t*>(base);
    size_t off = 0;
    auto take = [&](size_t n) {
        uint8_t* r = p ? p + off : nullptr;
        off += align_up(n, 256);
        return r;
    };
    w.hash = reinterpret_cast<unsigned long long*>(take(sizeof(unsigned long long) * Q));
    w.keys = reinterpret_cast<unsigned long long*>(take(sizeof(unsigned long long) * slots));
    w.min_row = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * slots));
    w.slot_of = reinterpret_cast<int32_t*>(take(sizeof(int32_t) * Q));
    w.bytes = off;
    return w;
}

// Contribution of value v at position i of a row: one multiply-xorshift round keyed by the
// position in the low half, the same value times an odd multiplier of the position in the
// high half.  Cheap on purpose - the pass should run at the speed of its reads - and good
// enough: every merge is verified entry by entry afterwards.
__device__ __forceinline__ unsigned long long mix_at(uint32_t v, uint32_t i) {
    uint32_t x = (v ^ (i * 0x9E3779B1u)) * 0x85EBCA6Bu;
    x ^= x >> 15;
    return (static_cast<unsigned long long>(x * (2u * i + 1u)) << 32) + x;
}

// Sum of mix_at over row[0..n) for this thread's share; positions start at `base`.
// Reads 16 bytes at a time where the row allows it.
template <typename T>
__device__ __forceinline__ unsigned long long hash_part(const T* __restrict__ row, int n, uint32_t base) {
    constexpr int EPV = 16 / sizeof(T);
    unsigned long long h = 0;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(row);
    int head = static_cast<int>(((16 - (addr & 15)) & 15) / sizeof(T));  // elements before a 16-byte boundary
    if (head > n) head = n;
    for (int i = threadIdx.x; i < head; i += blockDim.x) h += mix_at(row[i], base + i);
    const int nvec = (n - head) / EPV;
    const uint4* vec = reinterpret_cast<const uint4*>(row + head);
    for (int j = threadIdx.x; j < nvec; j += blockDim.x) {
        const uint4 v = __ldg(vec + j);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        const uint32_t i0 = base + head + j * EPV;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if constexpr (sizeof(T) == 4) {
                h += mix_at(w[k], i0 + k);
            } else {
                h += mix_at(w[k] & 0xFFFFu, i0 + 2 * k);
                h += mix_at(w[k] >> 16, i0 + 2 * k + 1);
            }
        }
    }
    for (int i = head + nvec * EPV + threadIdx.x; i < n; i += blockDim.x) h += mix_at(row[i], base + i);
    return h;
}

template <typename T>
__global__ void __launch_bounds__(kAliasThreads)
alias_hash(const uint32_t* __restrict__ mask, const T* __restrict__ next, int32_t Q, int32_t N, int32_t W,
           int weak, AliasWorkspace ws, int32_t* n_unique) {
    __shared__ unsigned long long part[kAliasThreads / 32];
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < ws.slots; i += gridDim.x * blockDim.x) {
        ws.keys[i] = kEmptyKey;
        ws.min_row[i] = 0x7FFFFFFF;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) *n_unique = 0;
    for (int q = blockIdx.x; q < Q; q += gridDim.x) {
        unsigned long long h = hash_part<uint32_t>(mask + static_cast<size_t>(q) * W, W, 0);
        if (next != nullptr) h += hash_part<T>(next + static_cast<size_t>(q) * N, N, static_cast<uint32_t>(W));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) h += __shfl_xor_sync(kFullWarp, h, off);
        if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = h;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long sum = 0;
            for (int w = 0; w < kAliasThreads / 32; ++w) sum += part[w];
            if (sum == kEmptyKey) sum -= 1;  // (the table's free-slot mark; exactness is the verifier's job)
            ws.hash[q] = weak ? 0ull : sum;
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256) alias_group(int32_t Q, AliasWorkspace ws, int32_t* status) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= Q) return;
    const unsigned long long key = ws.hash[q];
    uint32_t slot = static_cast<uint32_t>(key ^ (key >> 31)) & (ws.slots - 1);
    // at most Q distinct keys in >= 2Q slots: linear probing ends within `slots` steps
    for (uint32_t probe = 0; probe < ws.slots; ++probe) {
        const unsigned long long was = atomicCAS(&ws.keys[slot], kEmptyKey, key);
        if (was == kEmptyKey || was == key) break;
        slot = (slot + 1) & (ws.slots - 1);
    }
    if (idx_ok(slot, ws.slots, status)) {
        atomicMin(&ws.min_row[slot], q);
        ws.slot_of[q] = static_cast<int32_t>(slot);
    }
}

// Do rows a and b (n entries each) hold the same values?  All threads of the block call it
// and get the same answer; it stops at the first chunk that differs.
template <typename T>
__device__ __forceinline__ bool rows_equal(const T* __restrict__ a, const T* __restrict__ b, int n) {
    constexpr int kPer = 8;
    for (int i0 = 0; i0 < n; i0 += kAliasThreads * kPer) {
        bool diff = false;
#pragma unroll
        for (int k = 0; k < kPer; ++k) {
            const int i = i0 + k * kAliasThreads + threadIdx.x;
            if (i < n) diff |= a[i] != b[i];
        }
        if (__syncthreads_or(diff)) return false;
    }
    return true;
}

template <typename T>
__global__ void __launch_bounds__(kAliasThreads)
alias_verify(const uint32_t* __restrict__ mask, const T* __restrict__ next, int32_t Q, int32_t N, int32_t W,
             AliasWorkspace ws, int32_t* __restrict__ row_alias, int32_t* n_unique, int32_t* status) {
    auto same = [&](int a, int b) {
        if (!rows_equal<uint32_t>(mask + static_cast<size_t>(a) * W, mask + static_cast<size_t>(b) * W, W))
            return false;
        return next == nullptr ||
               rows_equal<T>(next + static_cast<size_t>(a) * N, next + static_cast<size_t>(b) * N, N);
    };
    for (int q = blockIdx.x; q < Q; q += gridDim.x) {
        int rep = ws.min_row[ws.slot_of[q]];
        if (!idx_ok(rep, q + 1, status)) rep = q;
        int alias = q;
        if (rep != q) {
            if (same(rep, q)) {
                alias = rep;
            } else {
                // equal hashes, different rows: the earlier rows of this hash, one by one
                const unsigned long long key = ws.hash[q];
                for (int r = rep + 1; r < q; ++r) {
                    if (ws.hash[r] != key) continue;  // (block-uniform)
                    if (same(r, q)) {
                        alias = r;
                        break;
                    }
                }
            }
        }
        if (threadIdx.x == 0) {
            row_alias[q] = alias;
            if (alias == q) atomicAdd(n_unique, 1);
        }
    }
}

template <typename T>
cudaError_t launch_alias(const uint32_t* mask, const void* next, int32_t Q, int32_t N, const AliasWorkspace& ws,
                         int32_t* row_alias, int32_t* n_unique, int32_t* status, int sms, int weak,
                         cudaStream_t stream) {
    const int W = (N + 31) / 32;
    const int blocks = Q < 8 * sms ? Q : 8 * sms;
    const T* nxt = static_cast<const T*>(next);
    alias_hash<T><<<blocks, kAliasThreads, 0, stream>>>(mask, nxt, Q, N, W, weak, ws, n_unique);
    alias_group<<<(Q + 255) / 256, 256, 0, stream>>>(Q, ws, status);
    alias_verify<T><<<blocks, kAliasThreads, 0, stream>>>(mask, nxt, Q, N, W, ws, row_alias, n_unique, status);
    return cudaGetLastError();
}

}  // namespace
}  // namespace fsm

extern "C" size_t fsm_row_alias_workspace_bytes(int32_t Q) {
    if (Q <= 0) return 0;
    return fsm::carve_alias(nullptr, Q).bytes;
}

extern "C" int fsm_index_row_alias(const uint32_t* allowed_mask, const void* next_state, int32_t state_dtype,
                                   int32_t Q, int32_t N, int32_t* row_alias, int32_t* n_unique,
                                   void* workspace, size_t workspace_bytes, int32_t* status_word,
                                   void* cuda_stream) {
    using namespace fsm;
    if (!allowed_mask || !row_alias || !n_unique) return FSM_ERR_NULL;
    if (Q <= 0 || N <= 0) return FSM_ERR_SHAPE;
    if (state_dtype != FSM_STATE_I32 && state_dtype != FSM_STATE_U16) return FSM_ERR_DTYPE;
    if (next_state && state_dtype == FSM_STATE_U16 && Q > 65535) return FSM_ERR_DTYPE;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(allowed_mask, 4) || misaligned(row_alias, 4) || misaligned(n_unique, 4) ||
        misaligned(next_state, state_dtype == FSM_STATE_U16 ? 2 : 4) || misaligned(status_word, 4))
        return FSM_ERR_ALIGN;
    const AliasWorkspace ws = carve_alias(workspace, Q);
    if (!workspace || misaligned(workspace, 256) || workspace_bytes < ws.bytes) return FSM_ERR_WORKSPACE;
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return FSM_ERR_CUDA;
    if (dev.cc_major != 10) return FSM_ERR_DEVICE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int weak = tunables().weak_hash;
    cudaError_t e;
    if (next_state && state_dtype == FSM_STATE_U16)
        e = launch_alias<uint16_t>(allowed_mask, next_state, Q, N, ws, row_alias, n_unique, status_word,
                                   dev.sm_count, weak, stream);
    else
        e = launch_alias<int32_t>(allowed_mask, next_state, Q, N, ws, row_alias, n_unique, status_word,
                                  dev.sm_count, weak, stream);
    return e == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
}
