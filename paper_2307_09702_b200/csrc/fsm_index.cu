// Vocabulary index construction (paper Section 3, Algorithms 3 and 4) for sm_100a:
// host entry points.  The kernels live in the fsm_index_*.cuh headers.
//
// Launches on the caller's stream, no host synchronisation:
//   1. prepare_fused   (cooperative, three phases with grid barriers in between)
//        hash     one pass over delta: a 64-bit hash of each of the 256 byte columns
//        prepare  bytes with equal column hashes share a byte class; class-compressed
//                 table [Q x Cs] with exact verification that every byte's column
//                 equals its class representative's column; token records (dense
//                 walk) or bucket key counts (work-avoiding walks)
//        sort     work-avoiding walks only: tokens sorted by (first, second) byte class
//   2. walk            dense: every (state, token) pair walked by warp tiles;
//      walk_rows       rows filled from a per-row table, longer tokens of readable buckets
//                      walked and patched in;
//      mask_onebyte + walk_buckets   bitmask-only builds
// If the verification fails (a 64-bit hash collision) the walk reads the uncompressed
// table instead, so the result is exact in every case.
#include "fsm_index_common.cuh"
#include "fsm_index_dense.cuh"
#include "fsm_index_prep.cuh"
#include "fsm_index_rows.cuh"
#include "fsm_index_bucket.cuh"
#include "fsm_index_csr.cuh"

extern "C" size_t fsm_index_workspace_bytes(int32_t Q, int32_t N, int64_t vocab_nbytes) {
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0) return 0;
    return fsm::carve(nullptr, Q, N).bytes;
}

namespace {
// `dense_only`: the workspace holds only what the dense walk needs (no survivor scratch).
int build_rows_impl(const int32_t* dfa_trans, const uint8_t* accept, const uint8_t* vocab_bytes,
                    const int32_t* vocab_offsets, int64_t vocab_nbytes, int32_t Q, int32_t N,
                    int32_t dead_state, int32_t eos_id, int32_t q_begin, int32_t q_end,
                    uint32_t* allowed_mask, void* next_state, int32_t state_dtype, void* workspace,
                    size_t workspace_bytes, int32_t* status_word, void* cuda_stream,
                    bool dense_only, bool want_tok_head = false) {
    using namespace fsm;
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0 || N > 0x7FFFFFE0) return FSM_ERR_SHAPE;
    if (!dfa_trans || !accept || !vocab_offsets || !allowed_mask) return FSM_ERR_NULL;
    if (!vocab_bytes && vocab_nbytes > 0) return FSM_ERR_NULL;
    if (state_dtype != FSM_STATE_I32 && state_dtype != FSM_STATE_U16) return FSM_ERR_DTYPE;
    if (state_dtype == FSM_STATE_U16 && Q > 65535) return FSM_ERR_DTYPE;
    if (dead_state < 0 || dead_state >= Q) return FSM_ERR_RANGE;
    if (eos_id < -1 || eos_id >= N) return FSM_ERR_RANGE;
    if (q_begin < 0 || q_end > Q || q_begin > q_end) return FSM_ERR_RANGE;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(dfa_trans, 4) || misaligned(vocab_offsets, 4) || misaligned(allowed_mask, 4) ||
        misaligned(status_word, 4))
        return FSM_ERR_ALIGN;
    if (next_state && misaligned(next_state, state_dtype == FSM_STATE_U16 ? 2 : 4))
        return FSM_ERR_ALIGN;
    const Workspace sizes = carve(nullptr, Q, N);
    const size_t need = dense_only ? sizes.dense_bytes : sizes.bytes;
    if (!workspace || workspace_bytes < need) return FSM_ERR_WORKSPACE;
    if (misaligned(workspace, 256)) return FSM_ERR_ALIGN;
    if (q_begin == q_end) return FSM_OK;

    const DeviceInfo& dev = device_info();
    if (!dev.ok) return FSM_ERR_CUDA;
    if (dev.cc_major != 10) return FSM_ERR_DEVICE;
    const Tunables& tune = tunables();
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    Workspace ws = carve(workspace, Q, N);
    const bool wide = Q > 65535;
    const int G = (N + 31) / 32;
    int cap = dev.smem_optin - kStaticSmemSlack;  // static shared memory and alignment slack
    if (tune.smem_table_cap > 0 && tune.smem_table_cap < cap) cap = tune.smem_table_cap;
    // Automatic choice: the work-avoiding walks work row by row (or window by window) with
    // one CTA per SM, so they need at least one row per SM to fill the device; small automata
    // take the dense walk.  With a next-state table: the row-wise fill-and-patch walk;
    // bitmask-only builds: the bucket walk.
    const bool enough_rows = q_end - q_begin >= dev.sm_count;
    const bool rows_fits =
        !dense_only && rows_min_smem<int32_t>() <= static_cast<size_t>(dev.smem_optin - kStaticSmemSlack);
    const bool bucket = next_state == nullptr && !dense_only &&
                        (tune.walk_algo == 3 || (tune.walk_algo == 0 && enough_rows));
    const bool rows = !bucket && rows_fits &&
                      (tune.walk_algo == 2 || tune.walk_algo == 3 || (tune.walk_algo == 0 && enough_rows));
    const bool sparse = bucket || rows;  // tokens sorted by bucket key

    // ---- preparation: one cooperative launch, one block per SM
    int32_t* row_order = sparse && !bucket ? ws.row_order : nullptr;
    // (the ranking of the windows counts them in kKeys words of shared memory)
    int32_t* win_order = bucket && (N + 31) / 32 <= kKeys ? ws.win_order : nullptr;
    {
        PrepParams a = {};
        a.trans = dfa_trans;
        a.vocab_bytes = vocab_bytes;
        a.vocab_offsets = vocab_offsets;
        a.vocab_nbytes = vocab_nbytes;
        a.Q = Q;
        a.N = N;
        a.dead = dead_state;
        a.eos_id = eos_id;
        a.q_begin = q_begin;
        a.q_end = q_end;
        a.nparts = Q < kHashBlocks ? Q : kHashBlocks;
        a.weak = tune.weak_hash;
        a.sorted = sparse ? 1 : 0;
        a.partial = ws.partial;
        a.meta = ws.meta;
        a.cls = ws.cls;
        a.table = ws.table;
        a.tok_cls = ws.tok_cls;  // dense walk: token records
        a.tok_len = ws.tok_len;
        a.live = sparse ? ws.live : nullptr;  // bucket walk; row order of the row-wise walk
        a.count2 = ws.count2;
        a.cursor2 = ws.cursor2;
        a.start2 = ws.start2;
        a.gstart = ws.gstart;
        a.row_ctr = ws.row_ctr;
        a.planes = bucket || rows ? ws.planes : nullptr;
        a.tok_head = want_tok_head ? ws.tok_head : nullptr;
        a.tok_c1 = rows ? ws.tok_c1 : nullptr;
        a.srec = ws.srec;
        a.row_order = row_order;
        a.win_order = win_order;
        a.status = status_word;
        const size_t prep_smem = (sparse ? kKeysPad + kKeys : 0) * sizeof(int);
        int prep_blocks = dev.sm_count;
        if (tune.walk_ctas > 0 && tune.walk_ctas < prep_blocks) prep_blocks = tune.walk_ctas;
        if (prep_blocks < a.nparts) a.nparts = prep_blocks;
        cudaError_t e;
        if (wide) {
            auto k = prepare_fused<int32_t>;
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(prep_smem));
            if (e == cudaSuccess)
                e = launch_cooperative(k, dim3(prep_blocks), dim3(kPrepThreads), prep_smem, stream, a);
        } else {
            auto k = prepare_fused<uint16_t>;
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(prep_smem));
            if (e == cudaSuccess)
                e = launch_cooperative(k, dim3(prep_blocks), dim3(kPrepThreads), prep_smem, stream, a);
        }
        if (e != cudaSuccess) return FSM_ERR_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return FSM_ERR_CUDA;

    WalkParams p;
    p.table = ws.table;
    p.meta = ws.meta;
    p.trans = dfa_trans;
    p.accept = accept;
    p.vocab_bytes = vocab_bytes;
    p.vocab_offsets = vocab_offsets;
    p.vocab_nbytes = vocab_nbytes;
    p.Q = Q;
    p.N = N;
    p.G = G;
    p.dead = dead_state;
    p.eos_id = eos_id;
    p.q_begin = q_begin;
    p.q_end = q_end;
    p.tok_cls = ws.tok_cls;
    p.tok_len = ws.tok_len;
    p.srec = ws.srec;
    p.planes = ws.planes;
    p.tok_c1 = ws.tok_c1;
    p.live = ws.live;
    p.row_order = row_order;
    p.chunk = kChunk;
    p.wait_probe = tune.wait_probe;
    p.win_order = win_order;
    p.gstart = ws.gstart;
    p.count2 = ws.count2;
    p.start2 = ws.start2;
    p.row_ctr = ws.row_ctr;
    p.mask = allowed_mask;
    p.next = next_state;
    p.status = status_word;
    const int min_cap = rows ? static_cast<int>(rows_min_smem<int32_t>())
                             : (kChunk + 4) * kMaxCs * 4;
    if (cap < min_cap) cap = min_cap;
    p.smem_cap = static_cast<uint32_t>(cap) / 128 * 128;

    int64_t grid;
    if (sparse) {
        grid = q_end - q_begin;
    } else {
        // States per warp task: fewer for a small build, until every warp of the device has
        // two tasks (a task walks its states one after the other, so its length is latency).
        auto tasks_with = [&](int c) { return static_cast<int64_t>((q_end - q_begin + c - 1) / c) * G; };
        p.chunk = tasks_with(kChunk) < 2LL * dev.sm_count * kWalkWarps ? kSmallChunk : kChunk;
        const int64_t tasks = tasks_with(p.chunk);
        grid = tasks;  // capped at one CTA per SM below; its warps take the tasks round-robin
    }
    if (grid > dev.sm_count) grid = dev.sm_count;
    if (tune.walk_ctas > 0 && tune.walk_ctas < grid) grid = tune.walk_ctas;
    const int prof = profile_begin(stream);
    cudaError_t e;
    if (bucket)
        e = wide ? launch_bucket<int32_t>(p, dev.sm_count, stream)
                 : launch_bucket<uint16_t>(p, dev.sm_count, stream);
    else if (rows)
        e = wide ? launch_rows_for<int32_t>(p, static_cast<int>(grid), state_dtype,
                                            next_state != nullptr, stream)
                 : launch_rows_for<uint16_t>(p, static_cast<int>(grid), state_dtype,
                                             next_state != nullptr, stream);
    else
        e = wide ? launch_walk_for<int32_t>(p, static_cast<int>(grid), state_dtype,
                                            next_state != nullptr, stream)
                 : launch_walk_for<uint16_t>(p, static_cast<int>(grid), state_dtype,
                                             next_state != nullptr, stream);
    profile_end(prof, stream);
    return e == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
}
}  // namespace

extern "C" int fsm_index_build_rows(const int32_t* dfa_trans, const uint8_t* accept,
                                    const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                    int64_t vocab_nbytes, int32_t Q, int32_t N,
                                    int32_t dead_state, int32_t eos_id, int32_t q_begin,
                                    int32_t q_end, uint32_t* allowed_mask, void* next_state,
                                    int32_t state_dtype, void* workspace, size_t workspace_bytes,
                                    int32_t* status_word, void* cuda_stream) {
    return build_rows_impl(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                           dead_state, eos_id, q_begin, q_end, allowed_mask, next_state,
                           state_dtype, workspace, workspace_bytes, status_word, cuda_stream, false);
}

extern "C" int fsm_index_build(const int32_t* dfa_trans, const uint8_t* accept,
                               const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                               int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                               int32_t eos_id, uint32_t* allowed_mask, void* next_state,
                               int32_t state_dtype, void* workspace, size_t workspace_bytes,
                               int32_t* status_word, void* cuda_stream) {
    return fsm_index_build_rows(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                                dead_state, eos_id, 0, Q, allowed_mask, next_state, state_dtype,
                                workspace, workspace_bytes, status_word, cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant: the scratch of the build's kernels lives in this array inside the
// library's device image instead of in a caller-provided workspace.  In host code the name
// `g_static_scratch` is only a handle for the runtime, not a device address: the address the
// kernels need comes from cudaGetSymbolAddress, looked up once per device.
namespace fsm {
namespace {
static __device__ __align__(256) unsigned char g_static_scratch[FSM_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device, or nullptr on failure.
void* static_scratch_address() {
    constexpr int kMaxDevices = 64;
    static void* cached[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (cached[dev] == nullptr) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        cached[dev] = ptr;
    }
    return cached[dev];
}
}  // namespace
}  // namespace fsm

extern "C" int fsm_index_build_static(const int32_t* dfa_trans, const uint8_t* accept,
                                      const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                      int64_t vocab_nbytes, int32_t Q, int32_t N,
                                      int32_t dead_state, int32_t eos_id, uint32_t* allowed_mask,
                                      void* next_state, int32_t state_dtype, int32_t* status_word,
                                      void* cuda_stream) {
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0) return FSM_ERR_SHAPE;
    // The built-in array is sized for the dense walk's scratch (no survivor lists).
    const size_t need = fsm::carve(nullptr, Q, N).dense_bytes;
    if (need > FSM_STATIC_SCRATCH_BYTES) return FSM_ERR_WORKSPACE;
    if (!fsm::device_info().ok) return FSM_ERR_CUDA;
    void* scratch = fsm::static_scratch_address();
    if (scratch == nullptr) return FSM_ERR_CUDA;
    // Every part of the scratch that the build reads is written earlier in the same build,
    // so the previous call's leftovers need no clearing.
    return build_rows_impl(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                           dead_state, eos_id, 0, Q, allowed_mask, next_state, state_dtype, scratch,
                           FSM_STATIC_SCRATCH_BYTES, status_word, cuda_stream, true);
}

// ---------------------------------------------------------------------------------------------
// Compressed rows: a bitmask-only build, then the rows are cut out of the bitmask.
extern "C" int fsm_index_build_csr(const int32_t* dfa_trans, const uint8_t* accept,
                                   const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                   int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                                   int32_t eos_id, uint32_t* allowed_mask, int64_t* row_offsets,
                                   int32_t* csr_tokens, int32_t* csr_next, int64_t capacity,
                                   void* workspace, size_t workspace_bytes, int32_t* status_word,
                                   void* cuda_stream) {
    using namespace fsm;
    if (!row_offsets || (capacity > 0 && (!csr_tokens || !csr_next))) return FSM_ERR_NULL;
    if (capacity < 0) return FSM_ERR_SHAPE;
    auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
    if (misaligned(row_offsets, 8) || misaligned(csr_tokens, 4) || misaligned(csr_next, 4))
        return FSM_ERR_ALIGN;
    if (Q <= 0 || N <= 0) return FSM_ERR_SHAPE;
    Workspace ws = carve(workspace, Q, N);
    uint16_t* dense_next = Q < kCsrDenseRows ? ws.csr_dense : nullptr;
    const int rc = build_rows_impl(dfa_trans, accept, vocab_bytes, vocab_offsets, vocab_nbytes, Q, N,
                                   dead_state, eos_id, 0, Q, allowed_mask, dense_next,
                                   dense_next ? FSM_STATE_U16 : FSM_STATE_I32, workspace,
                                   workspace_bytes, status_word, cuda_stream, false,
                                   /*want_tok_head=*/dense_next == nullptr);
    if (rc != FSM_OK) return rc;
    const DeviceInfo& dev = device_info();
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    WalkParams p = {};
    p.trans = dfa_trans;
    p.accept = accept;
    p.vocab_bytes = vocab_bytes;
    p.vocab_offsets = vocab_offsets;
    p.vocab_nbytes = vocab_nbytes;
    p.Q = Q;
    p.N = N;
    p.G = (N + 31) / 32;
    p.dead = dead_state;
    p.eos_id = eos_id;
    p.q_begin = 0;
    p.q_end = Q;
    p.mask = allowed_mask;
    p.status = status_word;
    const int blocks = Q < 8 * dev.sm_count ? Q : 8 * dev.sm_count;
    csr_count<<<blocks, kCsrThreads, 0, stream>>>(allowed_mask, p.G, Q, ws.row_count);
    csr_scan<<<1, 1024, 0, stream>>>(ws.row_count, Q, row_offsets, capacity, N, ws.row_order, status_word);
    const int fill_blocks = Q < 16 * dev.sm_count ? Q : 16 * dev.sm_count;
    const int fill_parts = p.G >= 8 * 32 * kFillWarps ? 8 : (p.G >= 4 * 32 * kFillWarps ? 4 : 1);
    csr_fill<<<dim3(fill_blocks, fill_parts), kFillThreads, 0, stream>>>(
        p, ws.tok_head, dense_next, ws.row_order, row_offsets, csr_tokens, csr_next, capacity);
    return cudaGetLastError() == cudaSuccess ? FSM_OK : FSM_ERR_CUDA;
}
