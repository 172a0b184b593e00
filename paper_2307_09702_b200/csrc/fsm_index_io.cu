// Index files: a built index written to and read back from one flat file (paper
// Section 3.2: the index is built once per automaton and vocabulary and reused).
// Host code only; device arrays travel through two pinned staging buffers.
#include <stdio.h>
#include <string.h>

#include "fsm_common.cuh"

namespace fsm {
namespace {

constexpr char kMagic[8] = {'F', 'S', 'M', 'G', 'I', 'D', 'X', '1'};
constexpr uint32_t kVersion = 1;
constexpr size_t kHeaderBytes = 128;
constexpr size_t kStageBytes = 16u << 20;

// ---------------------------------------------------------------------------- SHA-256
// FIPS 180-4, section 6.2.  The round constants are the first 32 bits of the fractional
// parts of the cube roots of the first 64 primes, the initial hash value those of the
// square roots of the first 8 primes; both are computed here (integer roots by Newton's
// method on 128-bit integers) rather than typed in.
struct Sha256Tables {
    uint32_t k[64];
    uint32_t h0[8];
};

unsigned __int128 iroot(unsigned __int128 x, int n) {  // floor of the n-th root, n = 2 or 3
    unsigned __int128 lo = 0, hi = (static_cast<unsigned __int128>(1) << (n == 2 ? 62 : 41));
    while (lo < hi) {
        const unsigned __int128 mid = lo + (hi - lo + 1) / 2;
        unsigned __int128 p = mid * mid;
        bool over = false;
        if (n == 3) {
            if (p != 0 && mid > (~static_cast<unsigned __int128>(0)) / p) over = true;
            else p *= mid;
        }
        if (!over && p <= x) lo = mid;
        else hi = mid - 1;
    }
    return lo;
}

const Sha256Tables& sha_tables() {
    static Sha256Tables t;
    static bool ready = false;
    if (!ready) {
        int primes[64], np = 0;
        for (int c = 2; np < 64; ++c) {
            bool prime = true;
            for (int d = 2; d * d <= c; ++d)
                if (c % d == 0) prime = false;
            if (prime) primes[np++] = c;
        }
        // frac(root(p)) * 2^32 = floor(root(p * 2^(32 n))) mod 2^32
        for (int i = 0; i < 64; ++i)
            t.k[i] = static_cast<uint32_t>(iroot(static_cast<unsigned __int128>(primes[i]) << 96, 3));
        for (int i = 0; i < 8; ++i)
            t.h0[i] = static_cast<uint32_t>(iroot(static_cast<unsigned __int128>(primes[i]) << 64, 2));
        ready = true;
    }
    return t;
}

inline uint32_t rotr(uint32_t x, int n) { return (x >> n) | (x << (32 - n)); }

struct Sha256 {
    uint32_t h[8];
    uint8_t block[64];
    size_t fill = 0;
    uint64_t total = 0;

    Sha256() { memcpy(h, sha_tables().h0, sizeof(h)); }

    void compress(const uint8_t* b) {
        const uint32_t* K = sha_tables().k;
        uint32_t w[64];
        for (int t = 0; t < 16; ++t)
            w[t] = (uint32_t(b[4 * t]) << 24) | (uint32_t(b[4 * t + 1]) << 16) | (uint32_t(b[4 * t + 2]) << 8) |
                   uint32_t(b[4 * t + 3]);
        for (int t = 16; t < 64; ++t) {
            const uint32_t s0 = rotr(w[t - 15], 7) ^ rotr(w[t - 15], 18) ^ (w[t - 15] >> 3);
            const uint32_t s1 = rotr(w[t - 2], 17) ^ rotr(w[t - 2], 19) ^ (w[t - 2] >> 10);
            w[t] = w[t - 16] + s0 + w[t - 7] + s1;
        }
        uint32_t a = h[0], bb = h[1], c = h[2], d = h[3], e = h[4], f = h[5], g = h[6], hh = h[7];
        for (int t = 0; t < 64; ++t) {
            const uint32_t S1 = rotr(e, 6) ^ rotr(e, 11) ^ rotr(e, 25);
            const uint32_t ch = (e & f) ^ (~e & g);
            const uint32_t t1 = hh + S1 + ch + K[t] + w[t];
            const uint32_t S0 = rotr(a, 2) ^ rotr(a, 13) ^ rotr(a, 22);
            const uint32_t maj = (a & bb) ^ (a & c) ^ (bb & c);
            const uint32_t t2 = S0 + maj;
            hh = g; g = f; f = e; e = d + t1; d = c; c = bb; bb = a; a = t1 + t2;
        }
        h[0] += a; h[1] += bb; h[2] += c; h[3] += d; h[4] += e; h[5] += f; h[6] += g; h[7] += hh;
    }

    void update(const void* data, size_t n) {
        const uint8_t* p = static_cast<const uint8_t*>(data);
        total += n;
        while (n > 0) {
            if (fill == 0 && n >= 64) {
                compress(p);
                p += 64;
                n -= 64;
                continue;
            }
            const size_t take = n < 64 - fill ? n : 64 - fill;
            memcpy(block + fill, p, take);
            fill += take;
            p += take;
            n -= take;
            if (fill == 64) {
                compress(block);
                fill = 0;
            }
        }
    }

    void finish(uint8_t* out32) {
        const uint64_t bits = total * 8;
        const uint8_t one = 0x80, zero = 0;
        update(&one, 1);
        while (fill != 56) update(&zero, 1);
        uint8_t len[8];
        for (int i = 0; i < 8; ++i) len[i] = static_cast<uint8_t>(bits >> (56 - 8 * i));
        update(len, 8);
        for (int i = 0; i < 8; ++i)
            for (int j = 0; j < 4; ++j) out32[4 * i + j] = static_cast<uint8_t>(h[i] >> (24 - 8 * j));
    }
};

// ---------------------------------------------------------------------------- checksum
inline uint64_t mix_word(uint64_t x) {  // splitmix64 finaliser
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

uint64_t checksum64(const void* data, size_t nbytes, uint64_t first) {
    const uint8_t* p = static_cast<const uint8_t*>(data);
    uint64_t sum = 0;
    for (size_t i = 0; i + 8 <= nbytes; i += 8) {
        uint64_t w;
        memcpy(&w, p + i, 8);
        sum += mix_word(w + (first + i / 8 + 1) * 0x9E3779B97F4A7C15ull);
    }
    return sum;
}

// ---------------------------------------------------------------------------- layout
struct Array {
    void* dev;
    size_t bytes;
};

inline size_t pad8(size_t n) { return (n + 7) / 8 * 8; }

// Checks the scalar part of a descriptor; fills the array list (device pointers as given).
int describe(const fsm_index_desc* d, Array (&arrays)[4], int* count, size_t* payload) {
    if (d == nullptr) return FSM_ERR_NULL;
    if (d->Q <= 0 || d->N <= 0) return FSM_ERR_SHAPE;
    if (d->form != FSM_INDEX_DENSE && d->form != FSM_INDEX_BITMASK && d->form != FSM_INDEX_CSR)
        return FSM_ERR_DTYPE;
    if (d->dead_state < 0 || d->dead_state >= d->Q || d->eos_id < -1 || d->eos_id >= d->N) return FSM_ERR_RANGE;
    const size_t Q = d->Q, N = d->N, W = (N + 31) / 32;
    int n = 0;
    arrays[n++] = {d->allowed_mask, Q * W * 4};
    if (d->form == FSM_INDEX_DENSE) {
        if (d->state_dtype != FSM_STATE_I32 && d->state_dtype != FSM_STATE_U16) return FSM_ERR_DTYPE;
        if (d->state_dtype == FSM_STATE_U16 && d->Q > 65535) return FSM_ERR_DTYPE;
        if (d->nnz != 0) return FSM_ERR_SHAPE;
        arrays[n++] = {d->next_state, Q * N * (d->state_dtype == FSM_STATE_U16 ? 2u : 4u)};
    } else if (d->form == FSM_INDEX_CSR) {
        if (d->state_dtype != 0) return FSM_ERR_DTYPE;
        if (d->nnz < 0 || static_cast<uint64_t>(d->nnz) > static_cast<uint64_t>(Q) * N) return FSM_ERR_SHAPE;
        arrays[n++] = {d->row_offsets, (Q + 1) * 8};
        arrays[n++] = {d->csr_tokens, static_cast<size_t>(d->nnz) * 4};
        arrays[n++] = {d->csr_next, static_cast<size_t>(d->nnz) * 4};
    } else {
        if (d->state_dtype != 0 || d->nnz != 0) return FSM_ERR_DTYPE;
    }
    size_t total = 0;
    for (int i = 0; i < n; ++i) total += pad8(arrays[i].bytes);
    *count = n;
    *payload = total;
    return FSM_OK;
}

void put32(uint8_t* p, uint32_t v) { memcpy(p, &v, 4); }
void put64(uint8_t* p, uint64_t v) { memcpy(p, &v, 8); }
uint32_t get32(const uint8_t* p) { uint32_t v; memcpy(&v, p, 4); return v; }
uint64_t get64(const uint8_t* p) { uint64_t v; memcpy(&v, p, 8); return v; }

void write_header(uint8_t (&h)[kHeaderBytes], const fsm_index_desc* d, uint64_t payload, uint64_t check) {
    memset(h, 0, kHeaderBytes);
    memcpy(h, kMagic, 8);
    put32(h + 8, kVersion);
    put32(h + 12, static_cast<uint32_t>(d->form));
    put32(h + 16, static_cast<uint32_t>(d->Q));
    put32(h + 20, static_cast<uint32_t>(d->N));
    put32(h + 24, static_cast<uint32_t>(d->state_dtype));
    put32(h + 28, static_cast<uint32_t>(d->dead_state));
    put32(h + 32, static_cast<uint32_t>(d->eos_id));
    put64(h + 40, static_cast<uint64_t>(d->nnz));
    put64(h + 48, payload);
    put64(h + 56, check);
    memcpy(h + 64, d->input_digest, 32);
}

// Reads and validates a header; returns the file's size through *file_bytes.
int read_header(FILE* f, fsm_index_desc* out, uint64_t* payload, uint64_t* check, uint64_t* file_bytes) {
    uint8_t h[kHeaderBytes];
    if (fread(h, 1, kHeaderBytes, f) != kHeaderBytes) return FSM_ERR_IO;
    if (memcmp(h, kMagic, 8) != 0 || get32(h + 8) != kVersion) return FSM_ERR_FORMAT;
    out->form = static_cast<int32_t>(get32(h + 12));
    out->Q = static_cast<int32_t>(get32(h + 16));
    out->N = static_cast<int32_t>(get32(h + 20));
    out->state_dtype = static_cast<int32_t>(get32(h + 24));
    out->dead_state = static_cast<int32_t>(get32(h + 28));
    out->eos_id = static_cast<int32_t>(get32(h + 32));
    out->nnz = static_cast<int64_t>(get64(h + 40));
    *payload = get64(h + 48);
    *check = get64(h + 56);
    memcpy(out->input_digest, h + 64, 32);
    if (fseek(f, 0, SEEK_END) != 0) return FSM_ERR_IO;
    const long end = ftell(f);
    if (end < 0) return FSM_ERR_IO;
    *file_bytes = static_cast<uint64_t>(end);
    if (fseek(f, static_cast<long>(kHeaderBytes), SEEK_SET) != 0) return FSM_ERR_IO;
    return FSM_OK;
}

// Two pinned staging buffers and the events that say when each is free again.
struct Staging {
    uint8_t* buf[2] = {nullptr, nullptr};
    cudaEvent_t done[2] = {nullptr, nullptr};
    bool ok = false;
    Staging() {
        ok = cudaMallocHost(reinterpret_cast<void**>(&buf[0]), kStageBytes) == cudaSuccess &&
             cudaMallocHost(reinterpret_cast<void**>(&buf[1]), kStageBytes) == cudaSuccess &&
             cudaEventCreateWithFlags(&done[0], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&done[1], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) (void)cudaGetLastError();
    }
    ~Staging() {
        for (int i = 0; i < 2; ++i) {
            if (done[i]) cudaEventDestroy(done[i]);
            if (buf[i]) cudaFreeHost(buf[i]);
        }
    }
};

}  // namespace
}  // namespace fsm

using namespace fsm;

extern "C" int fsm_sha256(const void* data, size_t nbytes, uint8_t* out32) {
    if ((data == nullptr && nbytes != 0) || out32 == nullptr) return FSM_ERR_NULL;
    Sha256 s;
    s.update(data, nbytes);
    s.finish(out32);
    return FSM_OK;
}

extern "C" uint64_t fsm_checksum64(const void* data, size_t nbytes, uint64_t first_word_index) {
    if (data == nullptr) return 0;
    return checksum64(data, nbytes, first_word_index);
}

extern "C" size_t fsm_index_serialized_bytes(const fsm_index_desc* desc) {
    Array arrays[4];
    int n = 0;
    size_t payload = 0;
    if (describe(desc, arrays, &n, &payload) != FSM_OK) return 0;
    return kHeaderBytes + payload;
}

extern "C" int fsm_index_peek(const char* path, fsm_index_desc* desc) {
    if (path == nullptr || desc == nullptr) return FSM_ERR_NULL;
    FILE* f = fopen(path, "rb");
    if (f == nullptr) return FSM_ERR_IO;
    fsm_index_desc got = *desc;
    uint64_t payload = 0, check = 0, file_bytes = 0;
    int rc = read_header(f, &got, &payload, &check, &file_bytes);
    fclose(f);
    if (rc != FSM_OK) return rc;
    Array arrays[4];
    int n = 0;
    size_t want = 0;
    if (describe(&got, arrays, &n, &want) != FSM_OK || want != payload) return FSM_ERR_FORMAT;
    if (file_bytes < kHeaderBytes + payload) return FSM_ERR_IO;
    if (file_bytes != kHeaderBytes + payload) return FSM_ERR_FORMAT;
    *desc = got;  // (the pointers were copied from *desc above)
    return FSM_OK;
}

extern "C" int fsm_index_save(const char* path, const fsm_index_desc* desc, void* cuda_stream) {
    if (path == nullptr) return FSM_ERR_NULL;
    Array arrays[4];
    int n = 0;
    size_t payload = 0;
    int rc = describe(desc, arrays, &n, &payload);
    if (rc != FSM_OK) return rc;
    for (int i = 0; i < n; ++i)
        if (arrays[i].bytes != 0 && arrays[i].dev == nullptr) return FSM_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    FILE* f = fopen(path, "wb");
    if (f == nullptr) return FSM_ERR_IO;
    Staging st;
    uint8_t header[kHeaderBytes];
    write_header(header, desc, payload, 0);
    bool io_ok = st.ok && fwrite(header, 1, kHeaderBytes, f) == kHeaderBytes;
    bool cuda_ok = st.ok;
    uint64_t check = 0, word = 0;
    // pieces of at most kStageBytes, alternating between the two buffers: the copy of piece
    // i+1 runs while piece i is summed and written
    struct Piece { int buf; size_t bytes, padded; };
    Piece inflight = {0, 0, 0};
    bool have = false;
    int next_buf = 0;
    auto drain = [&]() {
        if (!have) return;
        if (cudaEventSynchronize(st.done[inflight.buf]) != cudaSuccess) cuda_ok = false;
        uint8_t* b = st.buf[inflight.buf];
        memset(b + inflight.bytes, 0, inflight.padded - inflight.bytes);
        check += checksum64(b, inflight.padded, word);
        word += inflight.padded / 8;
        if (io_ok && fwrite(b, 1, inflight.padded, f) != inflight.padded) io_ok = false;
        have = false;
    };
    for (int i = 0; i < n && io_ok && cuda_ok; ++i) {
        const uint8_t* src = static_cast<const uint8_t*>(arrays[i].dev);
        size_t left = arrays[i].bytes;
        while (left > 0 && io_ok && cuda_ok) {
            const size_t take = left < kStageBytes ? left : kStageBytes;  // (kStageBytes is a multiple of 8)
            const int b = next_buf;
            next_buf ^= 1;
            if (cudaMemcpyAsync(st.buf[b], src, take, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
                cudaEventRecord(st.done[b], stream) != cudaSuccess)
                cuda_ok = false;
            drain();  // the piece before this one
            inflight = {b, take, left == take ? pad8(take) : take};
            have = true;
            src += take;
            left -= take;
        }
    }
    drain();
    if (cudaStreamSynchronize(stream) != cudaSuccess) cuda_ok = false;
    if (io_ok && cuda_ok) {
        write_header(header, desc, payload, check);
        io_ok = fseek(f, 0, SEEK_SET) == 0 && fwrite(header, 1, kHeaderBytes, f) == kHeaderBytes;
    }
    if (fclose(f) != 0) io_ok = false;
    if (!cuda_ok) {
        (void)cudaGetLastError();
        remove(path);
        return FSM_ERR_CUDA;
    }
    if (!io_ok) {
        remove(path);
        return FSM_ERR_IO;
    }
    return FSM_OK;
}

extern "C" int fsm_index_load(const char* path, const fsm_index_desc* desc, void* cuda_stream) {
    if (path == nullptr) return FSM_ERR_NULL;
    Array arrays[4];
    int n = 0;
    size_t payload = 0;
    int rc = describe(desc, arrays, &n, &payload);
    if (rc != FSM_OK) return rc;
    for (int i = 0; i < n; ++i)
        if (arrays[i].bytes != 0 && arrays[i].dev == nullptr) return FSM_ERR_NULL;
    FILE* f = fopen(path, "rb");
    if (f == nullptr) return FSM_ERR_IO;
    fsm_index_desc got = {};
    uint64_t file_payload = 0, want_check = 0, file_bytes = 0;
    rc = read_header(f, &got, &file_payload, &want_check, &file_bytes);
    if (rc == FSM_OK) {
        static const uint8_t zero[32] = {0};
        const bool any_digest = memcmp(desc->input_digest, zero, 32) == 0;
        if (got.form != desc->form || got.Q != desc->Q || got.N != desc->N ||
            got.state_dtype != desc->state_dtype || got.dead_state != desc->dead_state ||
            got.eos_id != desc->eos_id || got.nnz != desc->nnz || file_payload != payload ||
            (!any_digest && memcmp(got.input_digest, desc->input_digest, 32) != 0))
            rc = FSM_ERR_FORMAT;
        else if (file_bytes < kHeaderBytes + payload)
            rc = FSM_ERR_IO;  // truncated
        else if (file_bytes != kHeaderBytes + payload)
            rc = FSM_ERR_FORMAT;
    }
    if (rc != FSM_OK) {
        fclose(f);
        return rc;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    Staging st;
    bool io_ok = true, cuda_ok = st.ok;
    uint64_t check = 0, word = 0;
    int next_buf = 0;
    bool used[2] = {false, false};
    for (int i = 0; i < n && io_ok && cuda_ok; ++i) {
        uint8_t* dst = static_cast<uint8_t*>(arrays[i].dev);
        size_t left = arrays[i].bytes;
        while (left > 0 && io_ok && cuda_ok) {
            const size_t take = left < kStageBytes ? left : kStageBytes;
            const size_t padded = left == take ? pad8(take) : take;
            const int b = next_buf;
            next_buf ^= 1;
            if (used[b] && cudaEventSynchronize(st.done[b]) != cudaSuccess) cuda_ok = false;  // buffer free again
            if (fread(st.buf[b], 1, padded, f) != padded) {
                io_ok = false;
                break;
            }
            check += checksum64(st.buf[b], padded, word);
            word += padded / 8;
            if (cudaMemcpyAsync(dst, st.buf[b], take, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
                cudaEventRecord(st.done[b], stream) != cudaSuccess)
                cuda_ok = false;
            used[b] = true;
            dst += take;
            left -= take;
        }
    }
    fclose(f);
    if (cudaStreamSynchronize(stream) != cudaSuccess) cuda_ok = false;
    if (!cuda_ok) {
        (void)cudaGetLastError();
        return FSM_ERR_CUDA;
    }
    if (!io_ok) return FSM_ERR_IO;
    return check == want_check ? FSM_OK : FSM_ERR_FORMAT;
}

extern "C" int fsm_index_input_digest(const int32_t* dfa_trans, const uint8_t* accept,
                                      const uint8_t* vocab_bytes, const int32_t* vocab_offsets,
                                      int64_t vocab_nbytes, int32_t Q, int32_t N, int32_t dead_state,
                                      int32_t eos_id, uint8_t* out32, void* cuda_stream) {
    if (!dfa_trans || !accept || !vocab_offsets || !out32 || (!vocab_bytes && vocab_nbytes > 0))
        return FSM_ERR_NULL;
    if (Q <= 0 || N <= 0 || vocab_nbytes < 0) return FSM_ERR_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    Sha256 sha;
    const int32_t scalars[4] = {Q, N, dead_state, eos_id};
    sha.update(scalars, sizeof(scalars));
    sha.update(&vocab_nbytes, sizeof(vocab_nbytes));
    Staging st;
    if (!st.ok) return FSM_ERR_CUDA;
    const Array arrays[4] = {{const_cast<int32_t*>(dfa_trans), static_cast<size_t>(Q) * 256 * 4},
                             {const_cast<uint8_t*>(accept), static_cast<size_t>(Q)},
                             {const_cast<int32_t*>(vocab_offsets), (static_cast<size_t>(N) + 1) * 4},
                             {const_cast<uint8_t*>(vocab_bytes), static_cast<size_t>(vocab_nbytes)}};
    for (const Array& a : arrays) {
        const uint8_t* src = static_cast<const uint8_t*>(a.dev);
        for (size_t left = a.bytes; left > 0;) {
            const size_t take = left < kStageBytes ? left : kStageBytes;
            if (cudaMemcpyAsync(st.buf[0], src, take, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
                cudaStreamSynchronize(stream) != cudaSuccess) {
                (void)cudaGetLastError();
                return FSM_ERR_CUDA;
            }
            sha.update(st.buf[0], take);
            src += take;
            left -= take;
        }
    }
    sha.finish(out32);
    return FSM_OK;
}
