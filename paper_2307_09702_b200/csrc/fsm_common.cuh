// Shared host/device helpers for the fsmguide kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fsmguide.h"

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "fsmguide kernels are written for sm_100a"
#endif

namespace fsm {

constexpr uint32_t kFullWarp = 0xFFFFFFFFu;

// Process-wide knobs behind fsm_debug_set.
struct Tunables {
    int weak_hash = 0;
    int mask_cluster = 0;
    int walk_ctas = 0;
    int smem_table_cap = 0;
    int profile_walk = 0;
    int walk_algo = 0;
    int wait_probe = 0;
};
Tunables& tunables();

struct DeviceInfo {
    int ok;          // 1 when the query succeeded
    int cc_major;
    int sm_count;
    int smem_optin;  // max dynamic shared memory per block (opt-in), bytes
};
// Properties of the current device (queried once per device index, cached).
const DeviceInfo& device_info();

// Event pairs behind FSM_PROFILE_WALK.  profile_begin returns a slot (or -1 when
// profiling is off or the ring is full) after recording the first event.
int profile_begin(cudaStream_t stream);
void profile_end(int slot, cudaStream_t stream);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#ifdef __CUDACC__
// Plain launch on `stream` through the extensible launch API.
template <typename... KArgs, typename... Args>
cudaError_t launch_on(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                      cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Cooperative launch: every block of the grid is resident at once (the launch fails
// otherwise), so the kernel may use grid-wide barriers.
template <typename... KArgs, typename... Args>
cudaError_t launch_cooperative(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                               cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

#ifdef __CUDACC__
__device__ __forceinline__ void raise_flag(int32_t* status_word, int flag) {
    if (status_word != nullptr) atomicOr(status_word, flag);
}

// Range-checked build (-DFSM_CHECKED, a second library that is never the default): every
// index that depends on data read from memory - a token id out of a sorted record, a state
// out of a table, a position out of a counter - is compared with the size of the array it
// goes into.  A violation raises FSM_FLAG_INDEX and the access is skipped; nothing traps.
// In the regular build the test is constant-true and folds away.
#ifdef FSM_CHECKED
constexpr bool kChecked = true;
#else
constexpr bool kChecked = false;
#endif

template <typename I, typename B>
__device__ __forceinline__ bool idx_ok(I i, B n, int32_t* status_word) {
    if constexpr (kChecked) {
        if (static_cast<long long>(i) < 0 || static_cast<long long>(i) >= static_cast<long long>(n)) {
            raise_flag(status_word, FSM_FLAG_INDEX);
            return false;
        }
    }
    return true;
}

// ----------------------------------------------------------------------------
// mbarrier + bulk async copy (the non-tensor form of TMA), CTA-local, no multicast.
// ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count)
                 : "memory");
}

__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)),
                 "r"(bytes)
                 : "memory");
}

// dst (shared) and src (global) 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes,
                                              uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_addr(dst)), "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

// Bounded wait: gives up after `limit` polls (each poll may itself suspend for a
// hardware-defined time).  Returns false on give-up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity,
                                                  uint32_t limit = (1u << 20)) {
    for (uint32_t it = 0; it < limit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

// ----------------------------------------------------------------------------
// 256-bit global loads / stores (sm_100).
// ----------------------------------------------------------------------------
struct alignas(32) Vec32B {
    uint32_t w[8];
};

__device__ __forceinline__ Vec32B ldg_stream_32B(const void* p) {
    Vec32B v;
    asm volatile("ld.global.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]),
                   "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void stg_32B(void* p, const Vec32B& v) {
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.w[0]),
                 "r"(v.w[1]), "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]),
                 "r"(v.w[7])
                 : "memory");
}
#endif  // __CUDACC__

}  // namespace fsm
