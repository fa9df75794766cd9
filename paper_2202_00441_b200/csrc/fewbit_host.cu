// HOST-pointer entry points: the hot path for callers whose tensors live in
// host memory.  The tensor is streamed through a caller-owned device
// workspace in chunks; chunk c uses pipeline stage c % 3, each stage has its
// own stream, so the host->device copy of one chunk, the kernel of the
// previous one and the device->host copy of the one before overlap.  The
// streams are created on first use and reused by later calls.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <mutex>
#include <vector>

#include "fewbit_internal.h"

namespace fewbit {
namespace {

constexpr int kStages = 3;
constexpr size_t kChunkQuantum = 1024;   // elements; keeps every chunk's packed words whole and 16-byte aligned
constexpr size_t kSlotAlign = 256;

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t elem_bytes(fewbit_dtype d) { return d == FEWBIT_F32 ? 4 : 2; }

// per stage: two dtype buffers (input and output of the kernel) and the packed words
inline size_t stage_bytes(size_t chunk, fewbit_dtype d, int bits) {
    return 2 * round_up(chunk * elem_bytes(d), kSlotAlign) + round_up(chunk * bits / 8, kSlotAlign);
}

// The three non-blocking streams of one call.  They are created once and kept: a call takes a free
// triple of the current device from a small per-device pool (or creates one when all are in use by
// concurrent calls of other host threads) and hands it back when it returns; nothing is destroyed
// before the process ends.  A call only returns after its streams have drained, so a triple taken
// from the pool is idle.
constexpr int kMaxDevices = 64;
struct StreamTriple { cudaStream_t s[kStages] = {nullptr, nullptr, nullptr}; };
std::mutex g_pool_mutex;
std::vector<StreamTriple> g_pool[kMaxDevices];

struct Pipeline {
    cudaStream_t stream[kStages] = {nullptr, nullptr, nullptr};
    cudaError_t err = cudaSuccess;
    int dev = -1;
    bool pooled = false;
    bool ok(cudaError_t e) { if (e != cudaSuccess && err == cudaSuccess) err = e; return e == cudaSuccess; }
    bool open() {
        if (!ok(cudaGetDevice(&dev))) return false;
        pooled = dev >= 0 && dev < kMaxDevices;
        if (pooled) {
            std::lock_guard<std::mutex> lock(g_pool_mutex);
            if (!g_pool[dev].empty()) {
                for (int s = 0; s < kStages; ++s) stream[s] = g_pool[dev].back().s[s];
                g_pool[dev].pop_back();
                return true;
            }
        }
        for (int s = 0; s < kStages; ++s)
            if (!ok(cudaStreamCreateWithFlags(&stream[s], cudaStreamNonBlocking))) return false;
        return true;
    }
    void close() {
        bool complete = true;
        for (int s = 0; s < kStages; ++s) {
            if (stream[s]) ok(cudaStreamSynchronize(stream[s])); else complete = false;
        }
        if (pooled && complete) {
            StreamTriple t;
            for (int s = 0; s < kStages; ++s) { t.s[s] = stream[s]; stream[s] = nullptr; }
            std::lock_guard<std::mutex> lock(g_pool_mutex);
            g_pool[dev].push_back(t);
            return;
        }
        for (int s = 0; s < kStages; ++s)
            if (stream[s]) { cudaStreamDestroy(stream[s]); stream[s] = nullptr; }
    }
};

inline size_t chunk_for(size_t workspace_bytes, fewbit_dtype d, int bits) {
    // largest multiple of the quantum whose three stages fit
    size_t lo = 0, hi = workspace_bytes / (kStages * 2 * elem_bytes(d)) / kChunkQuantum + 1;
    while (lo < hi) {
        const size_t mid = (lo + hi + 1) / 2;
        if (kStages * stage_bytes(mid * kChunkQuantum, d, bits) <= workspace_bytes) lo = mid; else hi = mid - 1;
    }
    return lo * kChunkQuantum;
}

}  // namespace
}  // namespace fewbit

extern "C" {

size_t fewbit_host_workspace_bytes(size_t chunk_elems, fewbit_dtype dtype, int bits) {
    using namespace fewbit;
    if (bits < 1 || bits > kMaxBits || !valid_dtype(dtype)) return 0;
    const size_t chunk = round_up(std::max<size_t>(chunk_elems, 1), kChunkQuantum);
    return kStages * stage_bytes(chunk, dtype, bits);
}

fewbit_status fewbit_fwd_host(const fewbit_table *table, const void *x_host, void *y_host, uint32_t *packed_host,
                              size_t n, fewbit_dtype dtype, void *workspace, size_t workspace_bytes) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (x_host == nullptr || y_host == nullptr || packed_host == nullptr || workspace == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kSlotAlign) return FEWBIT_ERR_ALIGNMENT;
    const int bits = table->bits;
    const size_t eb = elem_bytes(dtype);
    const size_t chunk = std::min(chunk_for(workspace_bytes, dtype, bits), round_up(n, kChunkQuantum));
    if (chunk == 0) return FEWBIT_ERR_ALLOC;
    const size_t sb = stage_bytes(chunk, dtype, bits), db = round_up(chunk * eb, kSlotAlign);
    Pipeline pipe;
    fewbit_status st = FEWBIT_OK;
    if (pipe.open()) {
        size_t c = 0;
        for (size_t e0 = 0; e0 < n && st == FEWBIT_OK; e0 += chunk, ++c) {
            const size_t m = std::min(chunk, n - e0);
            const int s = static_cast<int>(c % kStages);
            char *slot = static_cast<char *>(workspace) + s * sb;
            void *dx = slot, *dy = slot + db;
            uint32_t *dp = reinterpret_cast<uint32_t *>(slot + 2 * db);
            const char *hx = static_cast<const char *>(x_host) + e0 * eb;
            char *hy = static_cast<char *>(y_host) + e0 * eb;
            char *hp = reinterpret_cast<char *>(packed_host) + e0 / 32 * bits * 4;
            if (!pipe.ok(cudaMemcpyAsync(dx, hx, m * eb, cudaMemcpyHostToDevice, pipe.stream[s]))) break;
            st = fewbit_fwd(table, dx, dy, dp, m, dtype, pipe.stream[s]);
            if (st != FEWBIT_OK) break;
            if (!pipe.ok(cudaMemcpyAsync(hy, dy, m * eb, cudaMemcpyDeviceToHost, pipe.stream[s]))) break;
            if (!pipe.ok(cudaMemcpyAsync(hp, dp, fewbit_packed_bytes(m, bits), cudaMemcpyDeviceToHost, pipe.stream[s]))) break;
        }
    }
    pipe.close();
    if (st == FEWBIT_OK && pipe.err != cudaSuccess) { t_last_cuda_error = static_cast<int>(pipe.err); st = FEWBIT_ERR_CUDA; }
    return st;
}

fewbit_status fewbit_bwd_host(const fewbit_table *table, const uint32_t *packed_host, const void *grad_out_host,
                              void *grad_in_host, size_t n, fewbit_dtype dtype, void *workspace, size_t workspace_bytes) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (packed_host == nullptr || grad_out_host == nullptr || grad_in_host == nullptr || workspace == nullptr)
        return FEWBIT_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) % kSlotAlign) return FEWBIT_ERR_ALIGNMENT;
    const int bits = table->bits;
    const size_t eb = elem_bytes(dtype);
    const size_t chunk = std::min(chunk_for(workspace_bytes, dtype, bits), round_up(n, kChunkQuantum));
    if (chunk == 0) return FEWBIT_ERR_ALLOC;
    const size_t sb = stage_bytes(chunk, dtype, bits), db = round_up(chunk * eb, kSlotAlign);
    Pipeline pipe;
    fewbit_status st = FEWBIT_OK;
    if (pipe.open()) {
        size_t c = 0;
        for (size_t e0 = 0; e0 < n && st == FEWBIT_OK; e0 += chunk, ++c) {
            const size_t m = std::min(chunk, n - e0);
            const int s = static_cast<int>(c % kStages);
            char *slot = static_cast<char *>(workspace) + s * sb;
            void *dg = slot, *di = slot + db;
            uint32_t *dp = reinterpret_cast<uint32_t *>(slot + 2 * db);
            const char *hg = static_cast<const char *>(grad_out_host) + e0 * eb;
            char *hi = static_cast<char *>(grad_in_host) + e0 * eb;
            const char *hp = reinterpret_cast<const char *>(packed_host) + e0 / 32 * bits * 4;
            if (!pipe.ok(cudaMemcpyAsync(dp, hp, fewbit_packed_bytes(m, bits), cudaMemcpyHostToDevice, pipe.stream[s]))) break;
            if (!pipe.ok(cudaMemcpyAsync(dg, hg, m * eb, cudaMemcpyHostToDevice, pipe.stream[s]))) break;
            st = fewbit_bwd(table, dp, dg, di, m, dtype, pipe.stream[s]);
            if (st != FEWBIT_OK) break;
            if (!pipe.ok(cudaMemcpyAsync(hi, di, m * eb, cudaMemcpyDeviceToHost, pipe.stream[s]))) break;
        }
    }
    pipe.close();
    if (st == FEWBIT_OK && pipe.err != cudaSuccess) { t_last_cuda_error = static_cast<int>(pipe.err); st = FEWBIT_ERR_CUDA; }
    return st;
}

}  // extern "C"
