// Diagnostics: the binary32 evaluation of an activation against its binary64 form, on the device,
// over a range of input bit patterns (all 2^32 of them in a few seconds).
#include <cuda_runtime.h>

#include <cstdint>

#include "fewbit.h"
#include "fewbit_internal.h"
#include "fewbit_math.cuh"

namespace fewbit {
namespace {

// position of a binary32 value on the line of representable numbers (-0 and +0 coincide)
__device__ __forceinline__ long long ordered(float f) {
    const uint32_t u = __float_as_uint(f);
    const long long m = u & 0x7fffffffu;
    return (u >> 31) ? -m : m;
}

__device__ __forceinline__ unsigned long long distance(float got, float want) {
    if (isnan(got) || isnan(want)) return (isnan(got) && isnan(want)) ? 0ull : 0x7fffffffull;
    const long long d = ordered(got) - ordered(want);
    const unsigned long long a = static_cast<unsigned long long>(d < 0 ? -d : d);
    return a > 0x7fffffffull ? 0x7fffffffull : a;
}

// result[0..2]: inputs whose value is 0 / 1 / 2 ulp from the binary64 form rounded once;
// result[3]: inputs further away; result[4]: (largest distance << 32) | an input pattern with it
template <int ACT>
__global__ void __launch_bounds__(256) scan_kernel(unsigned long long first, unsigned long long count,
                                                    unsigned long long *result) {
    unsigned long long hist[4] = {0, 0, 0, 0};
    unsigned long long worst = 0;
    const unsigned long long pairs = (count + 1) / 2;
    for (unsigned long long i = static_cast<unsigned long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < pairs;
         i += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const uint32_t b0 = static_cast<uint32_t>(first + 2 * i);
        const bool two = 2 * i + 1 < count;
        const uint32_t b1 = two ? b0 + 1 : b0;
        const float x0 = __uint_as_float(b0), x1 = __uint_as_float(b1);
        const float2 y = act_f32<ACT>(make_float2(x0, x1));
        if (isfinite(x0)) {
            const unsigned long long d = distance(y.x, act_f64<ACT>(x0));
            hist[d < 3 ? d : 3] += 1;
            const unsigned long long key = (d << 32) | b0;
            worst = key > worst ? key : worst;
        }
        if (two && isfinite(x1)) {
            const unsigned long long d = distance(y.y, act_f64<ACT>(x1));
            hist[d < 3 ? d : 3] += 1;
            const unsigned long long key = (d << 32) | b1;
            worst = key > worst ? key : worst;
        }
    }
    for (int k = 0; k < 4; ++k) {
        unsigned long long v = hist[k];
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        if ((threadIdx.x & 31) == 0 && v) atomicAdd(&result[k], v);
    }
    for (int off = 16; off > 0; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, worst, off);
        worst = o > worst ? o : worst;
    }
    if ((threadIdx.x & 31) == 0) atomicMax(&result[4], worst);
}

using ScanLaunch = void (*)(unsigned long long, unsigned long long, unsigned long long *, int, cudaStream_t);

template <int ACT>
void launch_scan(unsigned long long first, unsigned long long count, unsigned long long *result, int grid, cudaStream_t st) {
    scan_kernel<ACT><<<grid, 256, 0, st>>>(first, count, result);
}

constexpr ScanLaunch kScan[FEWBIT_NUM_ACTS] = {
    launch_scan<0>, launch_scan<1>, launch_scan<2>, launch_scan<3>, launch_scan<4>,
    launch_scan<5>, launch_scan<6>, launch_scan<7>, launch_scan<8>};

}  // namespace
}  // namespace fewbit

extern "C" fewbit_status fewbit_f32_activation_scan(fewbit_act act, uint64_t first_pattern, uint64_t count,
                                                    uint64_t *result_device, void *stream) {
    using namespace fewbit;
    if (static_cast<int>(act) < 0 || static_cast<int>(act) >= FEWBIT_NUM_ACTS || result_device == nullptr)
        return FEWBIT_ERR_INVALID_ARG;
    if (first_pattern > (1ull << 32) || count > (1ull << 32) - first_pattern) return FEWBIT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(result_device) & 7u) != 0) return FEWBIT_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t err = cudaMemsetAsync(result_device, 0, 5 * sizeof(uint64_t), st);
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    if (count == 0) return FEWBIT_OK;
    const unsigned long long pairs = (count + 1) / 2;
    const unsigned long long want = (pairs + 255) / 256;
    const int grid = static_cast<int>(want < 148ull * 16 ? want : 148ull * 16);
    kScan[act](first_pattern, count, reinterpret_cast<unsigned long long *>(result_device), grid, st);
    err = cudaGetLastError();
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FEWBIT_OK;
}
