// Device helpers shared by the forward and backward kernels of Listing 1.
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
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "fewbit_internal.h"

namespace fewbit {

struct Boundaries { float s[kMaxLevels]; };
struct Levels { float lev[kMaxLevels]; };

constexpr int kLaneElems = 8;
constexpr int kTileElems = 32 * kLaneElems;               // 256
constexpr int kTilesPerWarp = 4;
constexpr int kWarpElems = kTilesPerWarp * kTileElems;    // 1024
constexpr int kThreads = 256;
constexpr int kWarpsPerCta = kThreads / 32;

// ---------------------------------------------------------------------------
// programmatic dependent launch: the next kernel of the stream may be scheduled once every CTA of
// this grid has started; a kernel launched that way must not touch global memory before pdl_wait(),
// which returns when the grids it depends on have completed and their writes are visible.  Both
// are no-ops for a kernel launched the ordinary way.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... Params, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem, cudaStream_t st, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}

// ---------------------------------------------------------------------------
// global memory access: 8 elements per lane, widened to binary32
// ---------------------------------------------------------------------------
// `wide` (warp-uniform): the address is 32-byte aligned, so the lane-chunk of eight binary32 values
// moves as one 256-bit access; otherwise (16-byte alignment only) as two 128-bit ones.  The 16-bit
// types always move 128 bits and ignore the flag.
__device__ __forceinline__ void load8(const float *p, float (&v)[8], bool wide = true) {
    if (wide) {
        asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7])
                     : "l"(p) : "memory");
    } else {
        asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                     : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4+16];"
                     : "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(p) : "memory");
    }
}

__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8], bool = true) {
    uint32_t r[4];
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p) : "memory");
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(r[i] << 16);                // exact widening
        v[2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
    }
}

__device__ __forceinline__ void store8(float *p, const float (&v)[8], bool wide = true) {
    if (wide) {
        asm volatile("st.global.v8.f32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                     :: "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "l"(p)
                     : "memory");
    } else {
        asm volatile("st.global.v4.f32 [%4], {%0,%1,%2,%3};" :: "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "l"(p) : "memory");
        asm volatile("st.global.v4.f32 [%4+16], {%0,%1,%2,%3};" :: "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]), "l"(p) : "memory");
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));   // round-to-nearest-even
    return d;
}

__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float (&v)[8], bool = true) {
    const uint32_t a = pack_bf16x2(v[0], v[1]), b = pack_bf16x2(v[2], v[3]);
    const uint32_t c = pack_bf16x2(v[4], v[5]), d = pack_bf16x2(v[6], v[7]);
    asm volatile("st.global.v4.u32 [%4], {%0,%1,%2,%3};" :: "r"(a), "r"(b), "r"(c), "r"(d), "l"(p) : "memory");
}

__device__ __forceinline__ void load8(const __half *p, float (&v)[8], bool = true) {
    uint32_t r[4];
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "l"(p) : "memory");
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&r[i]));   // exact widening
        v[2 * i] = f.x;
        v[2 * i + 1] = f.y;
    }
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));   // round-to-nearest-even
    return d;
}

__device__ __forceinline__ void store8(__half *p, const float (&v)[8], bool = true) {
    const uint32_t a = pack_f16x2(v[0], v[1]), b = pack_f16x2(v[2], v[3]);
    const uint32_t c = pack_f16x2(v[4], v[5]), d = pack_f16x2(v[6], v[7]);
    asm volatile("st.global.v4.u32 [%4], {%0,%1,%2,%3};" :: "r"(a), "r"(b), "r"(c), "r"(d), "l"(p) : "memory");
}

__device__ __forceinline__ float load1(const __half *p) { return __half2float(*p); }
__device__ __forceinline__ void store1(__half *p, float v) { *p = __float2half_rn(v); }
__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ __forceinline__ void store1(float *p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------
// Eq. 2 / the sorted search of Listing 1: code = #{ j : s[j] < x }, a branch-free binary
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

// `vec` (warp-uniform): the packed buffer is aligned for the vector access of this bit width (8 bytes
// at 2 bits, 16 at 4); otherwise (4-byte alignment only) the words move one by one.
template <int BITS>
__device__ __forceinline__ void store_words(uint32_t *p, const uint32_t (&w)[BITS], bool vec = true) {
    if constexpr (BITS == 1) {
        asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
    } else if constexpr (BITS == 2) {
        if (vec) {
            asm volatile("st.global.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(w[0]), "r"(w[1]) : "memory");
        } else {
            asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
            asm volatile("st.global.u32 [%0+4], %1;" :: "l"(p), "r"(w[1]) : "memory");
        }
    } else if constexpr (BITS == 3) {
        asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
        asm volatile("st.global.u32 [%0+4], %1;" :: "l"(p), "r"(w[1]) : "memory");
        asm volatile("st.global.u32 [%0+8], %1;" :: "l"(p), "r"(w[2]) : "memory");
    } else if (vec) {
        asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]) : "memory");
    } else {
        asm volatile("st.global.u32 [%0], %1;" :: "l"(p), "r"(w[0]) : "memory");
        asm volatile("st.global.u32 [%0+4], %1;" :: "l"(p), "r"(w[1]) : "memory");
        asm volatile("st.global.u32 [%0+8], %1;" :: "l"(p), "r"(w[2]) : "memory");
        asm volatile("st.global.u32 [%0+12], %1;" :: "l"(p), "r"(w[3]) : "memory");
    }
}

template <int BITS>
__device__ __forceinline__ void load_words(const uint32_t *p, uint32_t (&w)[BITS], bool vec = true) {
    if constexpr (BITS == 1) {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
    } else if constexpr (BITS == 2) {
        if (vec) {
            asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(p) : "memory");
        } else {
            asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
            asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+4];" : "=r"(w[1]) : "l"(p) : "memory");
        }
    } else if constexpr (BITS == 3) {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+4];" : "=r"(w[1]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+8];" : "=r"(w[2]) : "l"(p) : "memory");
    } else if (vec) {
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p) : "memory");
    } else {
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1];" : "=r"(w[0]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+4];" : "=r"(w[1]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+8];" : "=r"(w[2]) : "l"(p) : "memory");
        asm volatile("ld.global.L1::no_allocate.u32 %0, [%1+12];" : "=r"(w[3]) : "l"(p) : "memory");
    }
}


}  // namespace fewbit
