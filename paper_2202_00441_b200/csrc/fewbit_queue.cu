// Leases of work-counter sets for the dynamically scheduled forward variants.
//
// The counters are a file-scope __device__ array (no allocation at call time; the device address
// is resolved once per device with cudaGetSymbolAddress).  What is created lazily is one CUDA event
// per set and device, used to learn whether the last kernel that used the set has finished.
// A set is handed out again
//   * to the stream that used it last without any wait (stream order puts the new kernel after the
//     previous one, whose last CTA has zeroed the counters; streams are told apart by
//     cudaStreamGetId, which is never reused), or
//   * to any stream once its event has completed.
// While a stream is being captured no set is leased (an event query is not allowed there): the
// caller then uses the static partition.
#include <cuda_runtime.h>

#include <mutex>

#include "fewbit_internal.h"

namespace fewbit {
namespace {

constexpr int kMaxDevices = 64;
constexpr size_t kSetWords = static_cast<size_t>(kQueues) * kQueueStride;

// In host code this name is only a handle for the runtime, never a device address.
// The word behind the last set is the diagnostic tail counter.
static __device__ __align__(256) uint32_t g_counters[kQueueSlots * kSetWords + kQueueStride];

struct Slot {
    cudaEvent_t done = nullptr;          // recorded after the last launch that used the set
    unsigned long long stream_id = 0;    // of that launch
    bool used = false;                   // `done` has been recorded at least once
    bool leased = false;                 // between queue_acquire and queue_release
};
struct DeviceState {
    uint32_t *base = nullptr;            // device address of g_counters on this device
    Slot slot[kQueueSlots];
};
DeviceState g_state[kMaxDevices];
std::mutex g_mutex;

// Device address of g_counters on the current device (resolved once per device, under g_mutex).
cudaError_t counters_base(int *dev_out, uint32_t **base) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    DeviceState &st = g_state[dev];
    if (st.base == nullptr) {
        void *p = nullptr;
        err = cudaGetSymbolAddress(&p, g_counters);        // with `dev` current: that device's copy
        if (err != cudaSuccess) return err;
        st.base = static_cast<uint32_t *>(p);
    }
    *dev_out = dev;
    *base = st.base;
    return cudaSuccess;
}

}  // namespace

cudaError_t tail_counter_address(unsigned int **out) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int dev = 0;
    uint32_t *base = nullptr;
    const cudaError_t err = counters_base(&dev, &base);
    if (err != cudaSuccess) return err;
    *out = base + static_cast<size_t>(kQueueSlots) * kSetWords;
    return cudaSuccess;
}

cudaError_t tail_counter_read(uint64_t *count, bool reset) {
    unsigned int *p = nullptr;
    cudaError_t err = tail_counter_address(&p);
    if (err != cudaSuccess) return err;
    err = cudaDeviceSynchronize();
    if (err != cudaSuccess) return err;
    unsigned int v = 0;
    err = cudaMemcpy(&v, p, sizeof(v), cudaMemcpyDeviceToHost);
    if (err != cudaSuccess) return err;
    *count = v;
    return reset ? cudaMemset(p, 0, sizeof(v)) : cudaSuccess;
}

cudaError_t queue_acquire(cudaStream_t stream, QueueLease *lease) {
    *lease = QueueLease{};
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    cudaError_t err = cudaStreamIsCapturing(stream, &capturing);
    if (err != cudaSuccess) return err;
    if (capturing != cudaStreamCaptureStatusNone) return cudaSuccess;
    unsigned long long id = 0;
    err = cudaStreamGetId(stream, &id);
    if (err != cudaSuccess) return err;
    // Another host thread may be capturing a stream in the global capture mode, under which an event
    // query or creation from any thread is refused and would invalidate that capture: what follows
    // runs in the relaxed mode, which exempts this thread (none of it touches a capturing stream).
    cudaStreamCaptureMode mode = cudaStreamCaptureModeRelaxed;
    err = cudaThreadExchangeStreamCaptureMode(&mode);
    if (err != cudaSuccess) return err;
    struct Restore {
        cudaStreamCaptureMode m;
        ~Restore() { cudaThreadExchangeStreamCaptureMode(&m); }
    } restore{mode};
    std::lock_guard<std::mutex> lock(g_mutex);
    int dev = 0;
    uint32_t *base = nullptr;
    err = counters_base(&dev, &base);
    if (err == cudaErrorInvalidDevice) return cudaSuccess;  // more devices than the table holds: static partition
    if (err != cudaSuccess) return err;
    DeviceState &st = g_state[dev];
    int pick = -1;
    for (int i = 0; i < kQueueSlots && pick < 0; ++i)       // 1. last used by this stream: ordered behind that use
        if (!st.slot[i].leased && st.slot[i].used && st.slot[i].stream_id == id) pick = i;
    for (int i = 0; i < kQueueSlots && pick < 0; ++i)       // 2. never used
        if (!st.slot[i].leased && !st.slot[i].used) pick = i;
    for (int i = 0; i < kQueueSlots && pick < 0; ++i) {     // 3. its last use has completed
        if (st.slot[i].leased) continue;
        const cudaError_t q = cudaEventQuery(st.slot[i].done);
        if (q == cudaSuccess) pick = i;
        else if (q != cudaErrorNotReady) return q;
        else (void)cudaGetLastError();       // "not ready" is an answer, not an error: do not leave it behind for a later cudaGetLastError
    }
    if (pick < 0) return cudaSuccess;
    Slot &s = st.slot[pick];
    if (s.done == nullptr) {
        err = cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming);
        if (err != cudaSuccess) { s.done = nullptr; return err; }
    }
    uint32_t *set = st.base + static_cast<size_t>(pick) * kSetWords;     // all zero: never used, or reset by its last kernel
    s.leased = true;
    s.stream_id = id;
    lease->counters = set;
    lease->slot = pick;
    return cudaSuccess;
}

cudaError_t queue_release(const QueueLease &lease, cudaStream_t stream) {
    if (lease.counters == nullptr) return cudaSuccess;
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(g_mutex);
    if (err != cudaSuccess || dev < 0 || dev >= kMaxDevices) return err;
    Slot &s = g_state[dev].slot[lease.slot];
    err = cudaEventRecord(s.done, stream);
    if (err != cudaSuccess) return err;      // the set stays leased for good: nothing tells when its kernel ends
    s.used = true;
    s.leased = false;
    return cudaSuccess;
}

}  // namespace fewbit
