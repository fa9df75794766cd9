// Definitions shared by the translation units of the library (not installed).
#pragma once

#include <cstdint>

#include "fewbit.h"

#include <atomic>

namespace fewbit {
constexpr int kMaxBits = 4;
constexpr int kMaxLevels = 1 << kMaxBits;   // K <= 16

inline bool valid_dtype(int d) { return d == FEWBIT_F32 || d == FEWBIT_BF16 || d == FEWBIT_F16; }

extern std::atomic<uint64_t> g_launches;     // kernels launched by the library in this process
extern thread_local int t_last_cuda_error;   // cudaError_t behind this thread's last FEWBIT_ERR_CUDA
}  // namespace fewbit

namespace fewbit {

// Run-length form of a code look-up table over the top bits of an element's
// bit pattern ("cells").  Run i covers cells [start_i, start_{i+1}) and holds
// one byte value; entry = start | value << 24.  The forward kernel expands it
// into shared memory.
//   bf16 / f16 table: one cell per 16-bit pattern (65 536 cells), value = code.
//   fp32 table: one cell per top-13-bit pattern (8 192 cells), value = the
//               smallest code m in the cell when the cell holds at most one
//               boundary (then code(x) = m + (s[m] < x)), else kCellDense.
constexpr int kMaxRuns = 120;
constexpr int kCellBitsBf16 = 16;
constexpr int kCellBitsF32 = 13;
constexpr unsigned kCellDense = 0xffu;

struct CodeRuns {
    uint32_t count;                    // 0: table not expressible, use the search kernel
    uint32_t run[kMaxRuns];
};

void build_code_runs(const float *s, int bits, bool folded, CodeRuns *bf16_runs, CodeRuns *f32_runs, CodeRuns *f16_runs);
void build_bf16_thresholds(const float *s, uint32_t *s_bf16x2);
void build_f16_thresholds(const float *s, uint32_t *s_f16x2);
float f16_bits_to_float(uint32_t h);

}  // namespace fewbit

// ---- work counters of the dynamically scheduled forward variants (fewbit_queue.cu) ----------
// A launch that distributes warp-blocks dynamically needs kQueues zeroed 32-bit counters,
// kQueueStride words apart, that no other running kernel uses.  They live in a file-scope
// __device__ pool of kQueueSlots sets (zero-initialised); a set is leased per launch and the
// kernel itself puts it back to zero when its last CTA finishes.
#include <cuda_runtime_api.h>
namespace fewbit {
constexpr uint32_t kQueues = 16;
constexpr uint32_t kQueueStride = 64;               // 32-bit words (256 bytes)
constexpr int kQueueSlots = 16;
constexpr uint32_t kQueueDoneWord = kQueueStride / 2;   // in the padding behind counter 0: CTAs that have finished

struct QueueLease {
    uint32_t *counters = nullptr;                   // device address; nullptr: no set free, use the static partition
    int slot = -1;
};
// Picks a set that is safe to reuse (last used on this very stream, or by work that has completed).
// Leaves the lease empty while `stream` is being captured or when every set is still in use by
// other streams.
cudaError_t queue_acquire(cudaStream_t stream, QueueLease *lease);
// After the kernel launch (also after a failed one): records the point of `stream` up to which
// the set is in use.
cudaError_t queue_release(const QueueLease &lease, cudaStream_t stream);
// Diagnostic counter of the warps that ran the forward kernel's ragged-tail path (one word of the
// same file-scope device array): its device address on the current device, and a synchronising read.
cudaError_t tail_counter_address(unsigned int **out);
cudaError_t tail_counter_read(uint64_t *count, bool reset);
}  // namespace fewbit

// The parameters s and y of Eq. 2, as binary32.  Unused boundary slots hold
// +inf (never below any x), unused level slots 0.
struct fewbit_table {
    fewbit_act act;
    int bits;
    int folded;                        // 1: even f', the code is the position of |x| (table on [0, B])
    double objective;                  // value of Eq. 3 reached by the solver
    float s[fewbit::kMaxLevels];       // s[0 .. K-2]
    float lev[fewbit::kMaxLevels];     // lev[0 .. K-1]
    uint32_t s_bf16x2[fewbit::kMaxLevels];   // derived from s: largest bfloat16 <= s[j], in both halves of a word
    uint32_t s_f16x2[fewbit::kMaxLevels];    // the same for IEEE binary16
    fewbit::CodeRuns runs_bf16;        // derived from s: the bucketize step as a look-up table
    fewbit::CodeRuns runs_f16;
    fewbit::CodeRuns runs_f32;
};
