// Status strings, device query and process-wide knobs of the fsmguide C ABI.
#include <vector>

#include "fsm_common.cuh"

namespace fsm {

Tunables& tunables() {
    static Tunables t;
    return t;
}

const DeviceInfo& device_info() {
    constexpr int kMaxDevices = 64;
    static DeviceInfo cache[kMaxDevices] = {};
    static DeviceInfo bad = {0, 0, 0, 0};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return bad;
    }
    DeviceInfo& d = cache[dev];
    if (!d.ok) {
        int major = 0, sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) !=
                cudaSuccess) {
            (void)cudaGetLastError();
            return bad;
        }
        d.cc_major = major;
        d.sm_count = sms;
        d.smem_optin = smem;
        d.ok = 1;
    }
    return d;
}

namespace {
constexpr int kProfileRing = 4096;
struct EventPair {
    cudaEvent_t begin, end;
};
std::vector<EventPair>& ring() {
    static std::vector<EventPair> r;
    return r;
}
int g_profile_used = 0;
}  // namespace

int profile_begin(cudaStream_t stream) {
    if (!tunables().profile_walk || g_profile_used >= kProfileRing) return -1;
    std::vector<EventPair>& r = ring();
    if (g_profile_used >= static_cast<int>(r.size())) {
        EventPair e;
        if (cudaEventCreate(&e.begin) != cudaSuccess) return -1;
        if (cudaEventCreate(&e.end) != cudaSuccess) {
            cudaEventDestroy(e.begin);
            return -1;
        }
        r.push_back(e);
    }
    const int slot = g_profile_used++;
    cudaEventRecord(r[slot].begin, stream);
    return slot;
}

void profile_end(int slot, cudaStream_t stream) {
    if (slot >= 0) cudaEventRecord(ring()[slot].end, stream);
}

}  // namespace fsm

extern "C" int fsm_profile_read(float* ms_out, int32_t capacity) {
    using namespace fsm;
    int n = 0;
    int rc = 0;
    for (int i = 0; i < g_profile_used; ++i) {
        float ms = 0.f;
        if (cudaEventSynchronize(ring()[i].end) != cudaSuccess ||
            cudaEventElapsedTime(&ms, ring()[i].begin, ring()[i].end) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = FSM_ERR_CUDA;
            break;
        }
        if (ms_out && n < capacity) ms_out[n++] = ms;
    }
    g_profile_used = 0;
    return rc ? rc : n;
}

extern "C" const char* fsm_status_string(int status) {
    switch (status) {
        case FSM_OK: return "FSM_OK";
        case FSM_ERR_NULL: return "FSM_ERR_NULL: a required pointer is NULL";
        case FSM_ERR_SHAPE: return "FSM_ERR_SHAPE: a size is non-positive or inconsistent";
        case FSM_ERR_ALIGN: return "FSM_ERR_ALIGN: a pointer or stride is misaligned";
        case FSM_ERR_DTYPE: return "FSM_ERR_DTYPE: unknown dtype, or u16 states with Q > 65535";
        case FSM_ERR_WORKSPACE: return "FSM_ERR_WORKSPACE: workspace missing or too small";
        case FSM_ERR_RANGE: return "FSM_ERR_RANGE: dead_state, eos_id, row range or key out of range";
        case FSM_ERR_CUDA: return "FSM_ERR_CUDA: a CUDA runtime call failed";
        case FSM_ERR_DEVICE: return "FSM_ERR_DEVICE: current device is not compute capability 10.x";
        case FSM_ERR_IO: return "FSM_ERR_IO: index file cannot be opened, read or written, or is truncated";
        case FSM_ERR_FORMAT: return "FSM_ERR_FORMAT: not an index file of this version, for another problem, or damaged";
        default: return "FSM_ERR_UNKNOWN";
    }
}

extern "C" int fsm_device_check(void) {
    const fsm::DeviceInfo& d = fsm::device_info();
    if (!d.ok) return FSM_ERR_CUDA;
    return d.cc_major == 10 ? FSM_OK : FSM_ERR_DEVICE;
}

extern "C" int fsm_debug_set(int32_t key, int32_t value) {
    fsm::Tunables& t = fsm::tunables();
    int* slot = nullptr;
    switch (key) {
        case FSM_DEBUG_WEAK_HASH: slot = &t.weak_hash; break;
        case FSM_TUNE_MASK_CLUSTER: slot = &t.mask_cluster; break;
        case FSM_TUNE_WALK_CTAS: slot = &t.walk_ctas; break;
        case FSM_TUNE_SMEM_TABLE_BYTES: slot = &t.smem_table_cap; break;
        case FSM_PROFILE_WALK: slot = &t.profile_walk; break;
        case FSM_TUNE_WALK_ALGO: slot = &t.walk_algo; break;
        case FSM_DEBUG_WAIT_PROBE: slot = &t.wait_probe; break;
        default: return FSM_ERR_RANGE;
    }
    int old = *slot;
    *slot = value;
    return old;
}
