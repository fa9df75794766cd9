// Device side of the library: the fused forward (activation + bucketize +
// bit-pack) and backward (unpack + level lookup + multiply) kernels of
// Listing 1 for sm_100a, and the two DEVICE-pointer entry points.
//
// Work decomposition (both kernels)
//   lane-chunk : 8 consecutive elements, one 128-bit (bf16) or 256-bit (fp32)
//                global access per lane;
//   tile       : 32 lane-chunks = 256 consecutive elements, one fully
//                coalesced warp access;
//   warp-block : 4 consecutive tiles = 1024 elements = 32*bits packed words.
// A lane computes the 8 codes of its chunk in each of the 4 tiles (an
// 8*bits-bit group per tile).  A 4x4 transpose of those groups inside each
// quad of lanes (two shuffle rounds) leaves lane (4q + r) with the four
// groups of lanes 4q..4q+3 for tile r, i.e. with 32 consecutive codes =
// exactly `bits` whole words, written with one vector store.  The backward
// kernel runs the same transpose the other way round.
// The last n % 1024 elements take a scalar path (one lane = 32 consecutive
// elements = `bits` words, zero padded).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "fewbit_internal.h"
#include "fewbit_math.cuh"

namespace fewbit {

struct Boundaries { float s[kMaxLevels]; };
struct Levels { float lev[kMaxLevels]; };

constexpr int kLaneElems = 8;
constexpr int kTileElems = 32 * kLaneElems;               // 256
constexpr int kTilesPerWarp = 4;
constexpr int kWarpElems = kTilesPerWarp * kTileElems;    // 1024
constexpr int kThreads = 256;
constexpr int kWarpsPerCta = kThreads / 32;

std::atomic<uint64_t> g_launches{0};
thread_local int t_last_cuda_error = 0;

// ---------------------------------------------------------------------------
// global memory access: 8 elements per lane, widened to binary32
// ---------------------------------------------------------------------------
__device__ __forceinline__ void load8(const float *p, float (&v)[8]) {
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                 : "l"(p) : "memory");
}

__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8]) {
    uint32_t r[4];
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p) : "memory");
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(r[i] << 16);                // exact widening
        v[2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ void store8(float *p, const float (&v)[8]) {
    asm volatile("st.global.v8.f32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 :: "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "l"(p)
                 : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));   // round-to-nearest-even
    return d;
}

__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float (&v)[8]) {
    const uint32_t a = pack_bf16x2(v[0], v[1]), b = pack_bf16x2(v[2], v[3]);
    const uint32_t c = pack_bf16x2(v[4], v[5]), d = pack_bf16x2(v[6], v[7]);
    asm volatile("st.global.v4.u32 [%4], {%0,%1,%2,%3};" :: "r"(a), "r"(b), "r"(c), "r"(d), "l"(p) : "memory");
}

__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store1(float *p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------
// Eq. 2 / "sortedsearch": code = #{ j : s[j] < x }, a branch-free binary
// search over the 2^BITS - 1 sorted boundaries.  Every comparison is
// `s < x` in binary32, so NaN compares false everywhere (code 0).
// ---------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ uint32_t bucketize(const Boundaries &tb, float x) {
    const float *s = tb.s;
    if constexpr (BITS == 1) {
        return s[0] < x ? 1u : 0u;
    } else if constexpr (BITS == 2) {
        const bool p1 = s[1] < x;
        const float t0 = p1 ? s[2] : s[0];
        return (p1 ? 2u : 0u) + (t0 < x ? 1u : 0u);
    } else if constexpr (BITS == 3) {
        const bool p2 = s[3] < x;
        const float t1 = p2 ? s[5] : s[1];
        const bool p1 = t1 < x;
        const float a = p2 ? s[6] : s[2], b = p2 ? s[4] : s[0];
        const float t0 = p1 ? a : b;
        return (p2 ? 4u : 0u) + (p1 ? 2u : 0u) + (t0 < x ? 1u : 0u);
    } else {
        const bool p3 = s[7] < x;
        const float t2 = p3 ? s[11] : s[3];
        const bool p2 = t2 < x;
        const float a1 = p3 ? s[13] : s[5], b1 = p3 ? s[9] : s[1];
        const float t1 = p2 ? a1 : b1;
        const bool p1 = t1 < x;
        const float e0 = p3 ? s[8] : s[0], e1 = p3 ? s[10] : s[2];
        const float e2 = p3 ? s[12] : s[4], e3 = p3 ? s[14] : s[6];
        const float f0 = p2 ? e2 : e0, f1 = p2 ? e3 : e1;
        const float t0 = p1 ? f1 : f0;
        return (p3 ? 8u : 0u) + (p2 ? 4u : 0u) + (p1 ? 2u : 0u) + (t0 < x ? 1u : 0u);
    }
}

// ---------------------------------------------------------------------------
// 4x4 transpose inside each quad of lanes: on return a[j] of lane 4q+i holds
// what a[i] of lane 4q+j held.  Two butterfly rounds, four shuffles.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void quad_transpose(uint32_t (&a)[4], int lane) {
    const bool b0 = lane & 1, b1 = lane & 2;
    {
        const uint32_t s0 = b0 ? a[0] : a[1], s1 = b0 ? a[2] : a[3];
        const uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
        if (b0) { a[0] = r0; a[2] = r1; } else { a[1] = r0; a[3] = r1; }
    }
    {
        const uint32_t s0 = b1 ? a[0] : a[2], s1 = b1 ? a[1] : a[3];
        const uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 2), r1 = __shfl_xor_sync(0xffffffffu, s1, 2);
        if (b1) { a[0] = r0; a[1] = r1; } else { a[2] = r0; a[3] = r1; }
    }
}

// Four consecutive groups of 8*BITS bits  <->  BITS whole words.
template <int BITS>
__device__ __forceinline__ void groups_to_words(const uint32_t (&g)[4], uint32_t (&w)[BITS]) {
    if constexpr (BITS == 1) {
        w[0] = g[0] | (g[1] << 8) | (g[2] << 16) | (g[3] << 24);
    } else if constexpr (BITS == 2) {
        w[0] = g[0] | (g[1] << 16);
        w[1] = g[2] | (g[3] << 16);
    } else if constexpr (BITS == 3) {
        w[0] = g[0] | (g[1] << 24);
        w[1] = (g[1] >> 8) | (g[2] << 16);
        w[2] = (g[2] >> 16) | (g[3] << 8);
    } else {
        w[0] = g[0]; w[1] = g[1]; w[2] = g[2]; w[3] = g[3];
    }
}

template <int BITS>
__device__ __forceinline__ void words_to_groups(const uint32_t (&w)[BITS], uint32_t (&g)[4]) {
    if constexpr (BITS == 1) {
        g[0] = w[0] & 0xffu; g[1] = (w[0] >> 8) & 0xffu; g[2] = (w[0] >> 16) & 0xffu; g[3] = w[0] >> 24;
    } else if constexpr (BITS == 2) {
        g[0] = w[0] & 0xffffu; g[1] = w[0] >> 16; g[2] = w[1] & 0xffffu; g[3] = w[1] >> 16;
    } else if constexpr (BITS == 3) {
        g[0] = w[0] & 0xffffffu;
        g[1] = ((w[0] >> 24) | (w[1] << 8)) & 0xffffffu;
        g[2] = ((w[1] >> 16) | (w[2] << 16)) & 0xffffffu;
        g[3] = w[2] >> 8;
    } else {
        g[0] = w[0]; g[1] = w[1]; g[2] = w[2]; g[3] = w[3];
    }
}

template <int BITS>
__device__ __forceinline__ void store_words(uint32_t *p, const uint32_t (&w)[BITS]) {
    if constexpr (BITS == 1) {
        asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
    } else if constexpr (BITS == 2) {
        asm volatile("st.global.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(w[0]), "r"(w[1]) : "memory");
    } else if constexpr (BITS == 3) {
        asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
        asm volatile("st.global.u32 [%0+4], %1;" :: "l"(p), "r"(w[1]) : "memory");
        asm volatile("st.global.u32 [%0+8], %1;" :: "l"(p), "r"(w[2]) : "memory");
    } else {
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    }
}

template <int BITS>
__device__ __forceinline__ void load_words(const uint32_t *p, uint32_t (&w)[BITS]) {
    if constexpr (BITS == 1) {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
    } else if constexpr (BITS == 2) {
        asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(p) : "memory");
    } else if constexpr (BITS == 3) {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+4];" : "=r"(w[1]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+8];" : "=r"(w[2]) : "l"(p) : "memory");
    } else {
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p) : "memory");
    }
}

// ---------------------------------------------------------------------------
// Forward: y = f(x), code = position of x among s, packed = bit stream of codes
// ---------------------------------------------------------------------------
template <int ACT, int BITS, typename T>
__global__ void __launch_bounds__(kThreads)
fwd_kernel(const __grid_constant__ Boundaries tb, const T *x, T *y, uint32_t *packed, size_t n) {
    const int lane = threadIdx.x & 31;
    const size_t wb = static_cast<size_t>(blockIdx.x) * kWarpsPerCta + (threadIdx.x >> 5);
    const size_t full = n / kWarpElems;
    if (wb < full) {
        const size_t base = wb * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
        float v[kTilesPerWarp][8];
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) load8(x + base + t * kTileElems, v[t]);
        uint32_t grp[4];
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) {
            float o[8];
            uint32_t g = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                o[e] = activation<ACT, T>(v[t][e]);
                g |= bucketize<BITS>(tb, v[t][e]) << (BITS * e);
            }
            grp[t] = g;
            store8(y + base + t * kTileElems, o);
        }
        quad_transpose(grp, lane);
        uint32_t w[BITS];
        groups_to_words<BITS>(grp, w);
        store_words<BITS>(packed + wb * (32 * BITS) + (lane & 3) * (8 * BITS) + (lane >> 2) * BITS, w);
    } else if (wb == full && (n % kWarpElems) != 0) {
        // ragged tail: lane owns 32 consecutive elements = BITS words
        const size_t base = full * kWarpElems + static_cast<size_t>(lane) * 32;
        uint32_t w[BITS + 1];
#pragma unroll
        for (int j = 0; j <= BITS; ++j) w[j] = 0;
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            if (base + e < n) {
                const float xv = load1(x + base + e);
                store1(y + base + e, activation<ACT, T>(xv));
                const uint32_t c = bucketize<BITS>(tb, xv);
                const int pos = e * BITS;
                w[pos >> 5] |= c << (pos & 31);
                if ((pos & 31) + BITS > 32) w[(pos >> 5) + 1] |= c >> (32 - (pos & 31));
            }
        }
        const size_t total_words = (n * BITS + 31) / 32;
        const size_t first = full * (32 * BITS) + static_cast<size_t>(lane) * BITS;
#pragma unroll
        for (int j = 0; j < BITS; ++j)
            if (first + j < total_words) packed[first + j] = w[j];
    }
}

// ---------------------------------------------------------------------------
// Backward: grad_in = grad_out * lev[code]   (binary32 multiply, one rounding)
// ---------------------------------------------------------------------------
template <int BITS, typename T>
__global__ void __launch_bounds__(kThreads)
bwd_kernel(const __grid_constant__ Levels tl, const uint32_t *packed, const T *grad_out, T *grad_in, size_t n) {
    __shared__ float lev[kMaxLevels];
    if (threadIdx.x < kMaxLevels) lev[threadIdx.x] = tl.lev[threadIdx.x];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const size_t wb = static_cast<size_t>(blockIdx.x) * kWarpsPerCta + (threadIdx.x >> 5);
    const size_t full = n / kWarpElems;
    constexpr uint32_t kMask = (1u << BITS) - 1u;
    if (wb < full) {
        const size_t base = wb * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
        uint32_t w[BITS];
        load_words<BITS>(packed + wb * (32 * BITS) + (lane & 3) * (8 * BITS) + (lane >> 2) * BITS, w);
        float v[kTilesPerWarp][8];
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) load8(grad_out + base + t * kTileElems, v[t]);
        uint32_t grp[4];
        words_to_groups<BITS>(w, grp);
        quad_transpose(grp, lane);
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) {
            float o[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = __fmul_rn(v[t][e], lev[(grp[t] >> (BITS * e)) & kMask]);
            store8(grad_in + base + t * kTileElems, o);
        }
    } else if (wb == full && (n % kWarpElems) != 0) {
        const size_t base = full * kWarpElems + static_cast<size_t>(lane) * 32;
        const size_t total_words = (n * BITS + 31) / 32;
        const size_t first = full * (32 * BITS) + static_cast<size_t>(lane) * BITS;
        uint32_t w[BITS + 1];
#pragma unroll
        for (int j = 0; j < BITS; ++j) w[j] = (first + j < total_words) ? packed[first + j] : 0u;
        w[BITS] = 0;
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            if (base + e < n) {
                const int pos = e * BITS;
                uint32_t c = w[pos >> 5] >> (pos & 31);
                if ((pos & 31) + BITS > 32) c |= w[(pos >> 5) + 1] << (32 - (pos & 31));
                store1(grad_in + base + e, __fmul_rn(load1(grad_out + base + e), lev[c & kMask]));
            }
        }
    }
}

// ---------------------------------------------------------------------------
// dispatch
// ---------------------------------------------------------------------------
using FwdLaunch = cudaError_t (*)(const Boundaries &, const void *, void *, uint32_t *, size_t, cudaStream_t);
using BwdLaunch = cudaError_t (*)(const Levels &, const uint32_t *, const void *, void *, size_t, cudaStream_t);

inline unsigned grid_for(size_t n) {
    const size_t warps = n / kWarpElems + ((n % kWarpElems) ? 1 : 0);
    return static_cast<unsigned>((warps + kWarpsPerCta - 1) / kWarpsPerCta);
}

template <int ACT, int BITS, typename T>
cudaError_t launch_fwd(const Boundaries &tb, const void *x, void *y, uint32_t *packed, size_t n, cudaStream_t st) {
    fwd_kernel<ACT, BITS, T><<<grid_for(n), kThreads, 0, st>>>(tb, static_cast<const T *>(x), static_cast<T *>(y), packed, n);
    return cudaGetLastError();
}

template <int BITS, typename T>
cudaError_t launch_bwd(const Levels &tl, const uint32_t *packed, const void *g, void *gi, size_t n, cudaStream_t st) {
    bwd_kernel<BITS, T><<<grid_for(n), kThreads, 0, st>>>(tl, packed, static_cast<const T *>(g), static_cast<T *>(gi), n);
    return cudaGetLastError();
}

#define FEWBIT_FWD_ROW(A) \
    { { launch_fwd<A, 1, float>, launch_fwd<A, 1, __nv_bfloat16> }, { launch_fwd<A, 2, float>, launch_fwd<A, 2, __nv_bfloat16> }, \
      { launch_fwd<A, 3, float>, launch_fwd<A, 3, __nv_bfloat16> }, { launch_fwd<A, 4, float>, launch_fwd<A, 4, __nv_bfloat16> } }

const FwdLaunch kFwd[FEWBIT_NUM_ACTS][kMaxBits][2] = {
    FEWBIT_FWD_ROW(FEWBIT_GELU), FEWBIT_FWD_ROW(FEWBIT_SILU), FEWBIT_FWD_ROW(FEWBIT_SIGMOID), FEWBIT_FWD_ROW(FEWBIT_TANH),
    FEWBIT_FWD_ROW(FEWBIT_ELU), FEWBIT_FWD_ROW(FEWBIT_SOFTPLUS), FEWBIT_FWD_ROW(FEWBIT_LEAKY_RELU),
};

const BwdLaunch kBwd[kMaxBits][2] = {
    { launch_bwd<1, float>, launch_bwd<1, __nv_bfloat16> }, { launch_bwd<2, float>, launch_bwd<2, __nv_bfloat16> },
    { launch_bwd<3, float>, launch_bwd<3, __nv_bfloat16> }, { launch_bwd<4, float>, launch_bwd<4, __nv_bfloat16> },
};

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

}  // namespace fewbit

extern "C" {

fewbit_status fewbit_fwd(const fewbit_table *table, const void *x, void *y, uint32_t *packed, size_t n,
                         fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || (dtype != FEWBIT_F32 && dtype != FEWBIT_BF16)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (x == nullptr || y == nullptr || packed == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (!aligned(x, 32) || !aligned(y, 32) || !aligned(packed, 16)) return FEWBIT_ERR_ALIGNMENT;
    Boundaries tb;
    for (int m = 0; m < kMaxLevels; ++m) tb.s[m] = table->s[m];
    const cudaError_t err = kFwd[table->act][table->bits - 1][dtype == FEWBIT_BF16](
        tb, x, y, packed, n, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FEWBIT_OK;
}

fewbit_status fewbit_bwd(const fewbit_table *table, const uint32_t *packed, const void *grad_out, void *grad_in,
                         size_t n, fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || (dtype != FEWBIT_F32 && dtype != FEWBIT_BF16)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (packed == nullptr || grad_out == nullptr || grad_in == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (!aligned(grad_out, 32) || !aligned(grad_in, 32) || !aligned(packed, 16)) return FEWBIT_ERR_ALIGNMENT;
    Levels tl;
    for (int m = 0; m < kMaxLevels; ++m) tl.lev[m] = table->lev[m];
    const cudaError_t err = kBwd[table->bits - 1][dtype == FEWBIT_BF16](
        tl, packed, grad_out, grad_in, n, static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FEWBIT_OK;
}

int fewbit_last_cuda_error(void) { return fewbit::t_last_cuda_error; }

uint64_t fewbit_launch_count(void) { return fewbit::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
