// fewbit_fwd_host_static: the forward half on HOST buffers for callers that
// cannot allocate device memory.  The device staging area that
// fewbit_fwd_host takes from its caller lives here in a fixed array that is
// part of the library image, so the call needs no cudaMalloc from anyone.
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <mutex>

#include "fewbit_internal.h"

namespace fewbit {
namespace {

constexpr size_t kStaticMaxElems = FEWBIT_STATIC_MAX_ELEMS;
constexpr size_t kSlotAlign = 256;
// x, y (4 bytes per element at most) and the packed words (4 bits per element at most), each
// rounded up to the alignment unit
constexpr size_t kStaticBytes = 2 * (kStaticMaxElems * 4) + kStaticMaxElems / 2 + 3 * kSlotAlign;

// The staging area.  In host code this name is only a handle for the runtime, NOT a device
// address: it must never be handed to a kernel or a copy as a pointer.  The device address is
// obtained once per device with cudaGetSymbolAddress (below).
static __device__ __align__(256) unsigned char g_static_stage[kStaticBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char *g_stage_ptr[kMaxDevices] = {};       // device address of g_static_stage, per device
std::atomic<bool> g_stage_ready[kMaxDevices];

// Device address of the staging area on the current device; resolved on the first call per device.
cudaError_t stage_address(unsigned char **out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_stage_ready[dev].load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_stage_ready[dev].load(std::memory_order_relaxed)) {
            void *p = nullptr;
            err = cudaGetSymbolAddress(&p, g_static_stage);     // with `dev` current: that device's copy
            if (err != cudaSuccess) return err;
            g_stage_ptr[dev] = static_cast<unsigned char *>(p);
            g_stage_ready[dev].store(true, std::memory_order_release);
        }
    }
    *out = g_stage_ptr[dev];
    return cudaSuccess;
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace
}  // namespace fewbit

extern "C" {

size_t fewbit_static_max_elements(void) { return fewbit::kStaticMaxElems; }

fewbit_status fewbit_fwd_host_static(const fewbit_table *table, const void *x_host, void *y_host,
                                     uint32_t *packed_host, size_t n, fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (x_host == nullptr || y_host == nullptr || packed_host == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (n > kStaticMaxElems) return FEWBIT_ERR_TOO_LARGE;
    unsigned char *stage = nullptr;
    cudaError_t err = stage_address(&stage);
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    const size_t eb = dtype == FEWBIT_F32 ? 4 : 2;
    const size_t data_bytes = n * eb, slot = round_up(data_bytes, kSlotAlign);
    const size_t packed_bytes = fewbit_packed_bytes(n, table->bits);
    void *dx = stage, *dy = stage + slot;
    uint32_t *dp = reinterpret_cast<uint32_t *>(stage + 2 * slot);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // Every byte of the three regions that is read below is written first (x by the copy, y and the
    // packed words -- padding bits included -- by the kernel), so nothing has to be cleared even
    // though the array still holds the previous call's data.
    err = cudaMemcpyAsync(dx, x_host, data_bytes, cudaMemcpyHostToDevice, st);
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    const fewbit_status fs = fewbit_fwd(table, dx, dy, dp, n, dtype, stream);
    if (fs != FEWBIT_OK) { cudaStreamSynchronize(st); return fs; }
    err = cudaMemcpyAsync(y_host, dy, data_bytes, cudaMemcpyDeviceToHost, st);
    if (err == cudaSuccess) err = cudaMemcpyAsync(packed_host, dp, packed_bytes, cudaMemcpyDeviceToHost, st);
    const cudaError_t sync_err = cudaStreamSynchronize(st);
    if (err == cudaSuccess) err = sync_err;
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    return FEWBIT_OK;
}

}  // extern "C"
