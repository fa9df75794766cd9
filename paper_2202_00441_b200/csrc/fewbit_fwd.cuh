// Forward half of Listing 1 for sm_100a: y = f(x), code = position of x among
// the boundaries (Eq. 2), codes bit-packed into whole 32-bit words.
//
// A warp works on warp-blocks of 1024 elements (see fewbit_device.cuh for the
// lane / tile / warp-block decomposition and the quad transpose that turns
// per-lane code groups into whole words).  Which warp-blocks a warp gets:
//   * variants without a code table: a CTA owns a contiguous stretch of
//     warps * iters warp-blocks, warp w takes w, w + warps, ... of it; the CTA
//     size is chosen at launch (16-bit types: 4 warps) and the hardware block
//     scheduler balances the CTAs over the SMs;
//   * code-table variants: one wave of long-lived CTAs (the table is expanded
//     once per CTA); the warp-blocks are handed out dynamically through leased
//     work counters when a lease is available (fewbit_queue.cu), else statically
//     as above.
//
// Bucketize (code = #{ j : s[j] < x }, Eq. 2) has three implementations:
//   search   : branch-free binary search on one binary32 element (ALU pipe);
//   packed   : 16-bit types -- the same search on TWO elements per
//              instruction with bf16x2 / f16x2 compares against boundaries
//              rounded down to the storage type (exact: s < x <=> floor(s) < x
//              for an x of that type), threshold selection by bitwise masks
//              (at 4 bits the last pair of boundaries comes from a 64-word
//              shared-memory table indexed by both 3-bit prefixes);
//   look-up  : the code is a step function of x, so it is read from a byte
//              table in shared memory indexed by the top bits of the pattern:
//                16-bit   : 65 536 entries, one per pattern, the exact code;
//                binary32 : 8 192 entries (sign, exponent, 4 mantissa bits);
//                           an entry m is the smallest code in its cell and
//                           code = m + (s[m] < x), one binary32 comparison; a
//                           cell with two or more boundaries (or infinity next
//                           to NaNs) is marked dense and the warp redoes that
//                           tile by search.
//              The table arrives run-length encoded as a kernel parameter (a
//              few dozen runs) and is expanded by the CTA before streaming.
//              Random indices cost ~3.3 shared-memory wavefronts per warp
//              look-up.
// LUT = false: no table (16-bit types: packed search; binary32: search).  Which
// variant runs is decided per call from bits, dtype, activation and n
// (fewbit_fwd in fewbit_kernels.cu); all give identical codes.
#pragma once

#include <atomic>
#include <cstdlib>

#include "fewbit_device.cuh"
#include "fewbit_math.cuh"

namespace fewbit {

// threads per CTA the kernels are compiled for: binary32 keeps 32 registers of input in flight per
// thread, so it runs fewer, fatter threads (register cap 80) than the 16-bit types (cap 64); two
// CTAs of that size are resident per SM.  Variants without a table may be launched with fewer warps.
#ifndef FEWBIT_LUT_STAGES_BF16
#define FEWBIT_LUT_STAGES_BF16 1            // cp.async ring stages of the 16-bit table variant (the table takes 64 KB)
#endif
#ifndef FEWBIT_ASYNC_STAGES
#define FEWBIT_ASYNC_STAGES 2               // cp.async ring stages of the 16-bit variants without a code table
#endif
// binary32 without a code table: some (activation, bits) pairs run faster as more, thinner warps --
// compiled for 512 threads (64 registers) with a one-stage ring (4 KB of shared memory per warp), so
// that 32 warps are resident per SM instead of 24.  (The second ring stage is never filled: these
// variants take one warp-block per warp.)  Measured L2-cold at 2^24 and 2^28 elements, search variants:
// 3 bits, every activation with an exponential or tanh: 5-7 % faster (sigmoid 27.1 -> 25.9 us and
// 366 -> 346 us, softplus 28.4 -> 26.4 and 389 -> 365); 4 bits: sigmoid 33.3 -> 30.7 / 463 -> 408,
// SiLU 33.6 -> 31.8 / 467 -> 425, softplus equal / 471 -> 454, but ELU, SELU, tanh and the ReLUs
// 3-8 % slower (they keep 384 threads); 2 bits: SiLU only (334 -> 323 us).  GELU is bound by the FMA
// pipe and does not change with occupancy (445 us at 1 bit with 24 or 32 warps).
template <int ACT, int BITS>
constexpr bool kThinWarps = (BITS == 3 && ACT != FEWBIT_LEAKY_RELU && ACT != FEWBIT_RELU) ||
                            (BITS == 4 && (ACT == FEWBIT_SIGMOID || ACT == FEWBIT_SILU || ACT == FEWBIT_SOFTPLUS)) ||
                            (BITS == 2 && ACT == FEWBIT_SILU);
// (The 16-bit variants measured 1-5 % slower when compiled for 640 or 768 threads -- 40 or 48 resident warps at 48 / 40 registers.)
template <typename T, bool LUT = false, bool THIN = false> struct FwdThreads { static constexpr int value = sizeof(T) == 2 ? 512 : ((!LUT && THIN) ? 512 : 384); };
template <typename T, bool LUT> struct FwdCtas { static constexpr int value = 2; };
// cp.async ring stages of the variants without a code table
template <typename T, bool THIN> constexpr int kAsyncStages = sizeof(T) == 2 ? FEWBIT_ASYNC_STAGES : (THIN ? 1 : 2);

template <typename T> constexpr bool kIsHalf = false;
template <> constexpr bool kIsHalf<__half> = true;

template <typename T> struct Raw;                 // the 8 elements of a lane-chunk as loaded
template <> struct Raw<float> { float v[8]; };
template <> struct Raw<__nv_bfloat16> { uint32_t v[4]; };
template <> struct Raw<__half> { uint32_t v[4]; };

__device__ __forceinline__ void load_raw(const float *p, Raw<float> &r, bool wide) { load8(p, r.v, wide); }
__device__ __forceinline__ void load_raw(const __nv_bfloat16 *p, Raw<__nv_bfloat16> &r, bool) {
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]) : "l"(p) : "memory");
}
__device__ __forceinline__ void load_raw(const __half *p, Raw<__half> &r, bool) {
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]) : "l"(p) : "memory");
}
__device__ __forceinline__ float elem(const Raw<__half> &r, int e) {
    const __half2 h = *reinterpret_cast<const __half2 *>(&r.v[e >> 1]);
    return (e & 1) ? __high2float(h) : __low2float(h);
}
__device__ __forceinline__ uint32_t pair_bits(const Raw<__half> &r, int e) { return r.v[e >> 1]; }
__device__ __forceinline__ uint32_t cell(const Raw<__half> &r, int e) {
    return (e & 1) ? (r.v[e >> 1] >> 16) : (r.v[e >> 1] & 0xffffu);
}
__device__ __forceinline__ float elem(const Raw<float> &r, int e) { return r.v[e]; }
__device__ __forceinline__ float elem(const Raw<__nv_bfloat16> &r, int e) {
    return __uint_as_float((e & 1) ? (r.v[e >> 1] & 0xffff0000u) : (r.v[e >> 1] << 16));
}
__device__ __forceinline__ uint32_t pair_bits(const Raw<float> &, int) { return 0; }
__device__ __forceinline__ uint32_t pair_bits(const Raw<__nv_bfloat16> &r, int e) { return r.v[e >> 1]; }   // elements e, e+1 (e even)
__device__ __forceinline__ uint32_t cell(const Raw<float> &r, int e) { return __float_as_uint(r.v[e]) >> (32 - kCellBitsF32); }
__device__ __forceinline__ uint32_t cell(const Raw<__nv_bfloat16> &r, int e) {
    return (e & 1) ? (r.v[e >> 1] >> 16) : (r.v[e >> 1] & 0xffffu);
}

// ---------------------------------------------------------------------------
// optional bias in front of the activation: the lane-chunk becomes x + bias,
// the exact sum rounded once to the storage type (one IEEE addition in that
// type: add.rn.f32, add.rn.bf16x2, add.rn.f16x2).
// ---------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float round_to(float v) {     // v rounded to T (nearest even), widened back
    if constexpr (std::is_same<T, __nv_bfloat16>::value) return __bfloat162float(__float2bfloat16_rn(v));
    else if constexpr (std::is_same<T, __half>::value) return __half2float(__float2half_rn(v));
    else return v;
}
__device__ __forceinline__ void add_bias(Raw<float> &r, const float *b, bool wide) {
    float v[8];
    if (wide) {
        asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(b));
    } else {
        asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "l"(b));
        asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4+16];" : "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "l"(b));
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) r.v[e] = __fadd_rn(r.v[e], v[e]);
}
__device__ __forceinline__ void add_bias(Raw<__nv_bfloat16> &r, const __nv_bfloat16 *b, bool) {
    uint32_t v[4];
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "l"(b));
#pragma unroll
    for (int i = 0; i < 4; ++i) asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r.v[i]) : "r"(r.v[i]), "r"(v[i]));   // one rounding per half
}
__device__ __forceinline__ void add_bias(Raw<__half> &r, const __half *b, bool) {
    uint32_t v[4];
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "l"(b));
#pragma unroll
    for (int i = 0; i < 4; ++i) asm("add.rn.f16x2 %0, %1, %2;" : "=r"(r.v[i]) : "r"(r.v[i]), "r"(v[i]));
}

// ---------------------------------------------------------------------------
// asynchronous prefetch ring (variants without a code table): every lane copies
// its own lane-chunks of the next kStages warp-blocks global -> shared with
// cp.async and reads the same bytes back just before use.  No lane reads what
// another lane copied, so no barrier is involved; cp.async.wait_group is a
// blocking instruction, not a spin loop.
// ---------------------------------------------------------------------------
#ifndef FEWBIT_INDEXED_SEARCH
#define FEWBIT_INDEXED_SEARCH 1             // binary32 search variant at 4 bits: boundaries indexed in shared memory (0: select tree)
#endif

__device__ __forceinline__ void cp_async_chunk(uint32_t saddr, const __nv_bfloat16 *g) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(saddr), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_chunk(uint32_t saddr, const __half *g) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(saddr), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_chunk(uint32_t saddr, const float *g) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(saddr), "l"(g) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(saddr + 16), "l"(g + 4) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

__device__ __forceinline__ void load_raw_shared(uint32_t saddr, Raw<__nv_bfloat16> &r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ void load_raw_shared(uint32_t saddr, Raw<__half> &r) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]) : "r"(saddr) : "memory");
}
__device__ __forceinline__ void load_raw_shared(uint32_t saddr, Raw<float> &r) {
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]) : "r"(saddr) : "memory");
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7]) : "r"(saddr + 16) : "memory");
}

struct FwdSmem {
    uint32_t runs[kMaxRuns + 1];     // start | value << 24, plus a sentinel run starting one past the last cell
    float thr[kMaxLevels];           // the boundaries, for the binary32 one-comparison step
};

// Largest r with start(runs[r]) <= c.
__device__ __forceinline__ uint32_t find_run(const uint32_t *runs, uint32_t count, uint32_t c) {
    uint32_t lo = 0, hi = count;                    // invariant: start[lo] <= c < start[hi]
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if ((runs[mid] & 0xffffffu) <= c) lo = mid; else hi = mid;
    }
    return lo;
}

// Expands the run-length table into `lut` (CELLS bytes of shared memory).
template <int CELLS, int THREADS>
__device__ __forceinline__ void expand_runs(const CodeRuns &enc, uint8_t *lut, FwdSmem &sm) {
    const uint32_t count = enc.count;
    for (uint32_t i = threadIdx.x; i <= count; i += THREADS) sm.runs[i] = (i < count) ? enc.run[i] : static_cast<uint32_t>(CELLS);
    __syncthreads();
    // A warp owns a contiguous stretch of 16-cell groups; lane l takes groups l, l + 32, ... of it,
    // so that the 128-bit stores of one instruction fall on consecutive addresses (no bank conflict).
    // A group inside one run is one splat store; the few groups that straddle a run boundary (at
    // most one per run) are assembled byte by byte in registers by the same thread.
    constexpr int kGroups = CELLS / 16;             // 16 cells = one 128-bit shared store
    constexpr int kWarps = THREADS / 32;
    constexpr int kPerWarp = (kGroups + kWarps - 1) / kWarps;
    constexpr int kPerLane = (kPerWarp + 31) / 32;
    const uint32_t first = (threadIdx.x >> 5) * kPerWarp + (threadIdx.x & 31);
    if (first < kGroups) {
        uint32_t r = find_run(sm.runs, count, first * 16);
#pragma unroll 1
        for (int i = 0; i < kPerLane; ++i) {
            const uint32_t g = first + 32 * i;
            if (g >= kGroups || g >= ((threadIdx.x >> 5) + 1) * kPerWarp) break;
            const uint32_t a = g * 16;
            uint32_t next = sm.runs[r + 1] & 0xffffffu;
            while (next <= a) { ++r; next = sm.runs[r + 1] & 0xffffffu; }
            uint32_t w[4];
            if (next >= a + 16) {
                w[0] = w[1] = w[2] = w[3] = (sm.runs[r] >> 24) * 0x01010101u;
            } else {
                uint32_t rr = r, nn = next, v = sm.runs[r] >> 24;
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    while (nn <= a + c) { ++rr; nn = sm.runs[rr + 1] & 0xffffffu; v = sm.runs[rr] >> 24; }
                    if ((c & 3) == 0) w[c >> 2] = 0;
                    w[c >> 2] |= v << (8 * (c & 3));
                }
            }
            *reinterpret_cast<uint4 *>(lut + a) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    __syncthreads();
}

struct FwdParams {
    Boundaries tb;
    uint32_t sb2[kMaxLevels];        // boundaries rounded down to bfloat16, replicated in both halves
    CodeRuns runs;
    uint32_t *queue;                 // table variants: a leased set of zeroed work counters (dynamic distribution), or NULL (static)
    const void *bias;                // one value of the storage type per column, added to x before everything else, or NULL
    uint32_t cols;                   // with a bias: the row length, a multiple of kLaneElems (a lane-chunk never straddles a row end)
    uint64_t chunks_magic;           // floor(2^64 / (cols / kLaneElems)) + 1: exact division of 32-bit chunk numbers by a multiply-high
    uint32_t long_iters;             // warp-blocks per warp of the long CTAs of a static partition
    uint32_t flags;                  // kWideData | kVecPacked: what the alignment of the caller's buffers allows
    unsigned int *tail_counter;      // diagnostic (FEWBIT_OPT_COUNT_TAILS): counts the warps that run the ragged-tail path, or NULL
};
constexpr uint32_t kWideData = 1;    // x, y (and bias) are 32-byte aligned: binary32 lane-chunks move as one 256-bit access
constexpr uint32_t kVecPacked = 2;   // packed is aligned for the vector store of this bit width (8 bytes at 2 bits, 16 at 4)

// ---------------------------------------------------------------------------
// packed search: codes of the two bfloat16 elements of `x2`, low element in
// bits 0..3, high element in bits 16..19
// ---------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ uint32_t gt2(uint32_t a, uint32_t b) {          // per half: 0xffff if a > b (false for NaN)
    uint32_t r;
    if constexpr (sizeof(T) == 2 && !kIsHalf<T>) asm("set.gt.u32.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    else asm("set.gt.u32.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t sel2(uint32_t m, uint32_t a, uint32_t b) { return (m & a) | (~m & b); }

template <int BITS, typename T>
__device__ __forceinline__ uint32_t bucketize_bf16x2(const uint32_t (&S)[kMaxLevels], uint32_t x2, uint32_t pair_table = 0) {
    if constexpr (BITS == 1) {
        return gt2<T>(x2, S[0]) & 0x00010001u;
    } else if constexpr (BITS == 2) {
        const uint32_t m1 = gt2<T>(x2, S[1]);
        const uint32_t m0 = gt2<T>(x2, sel2(m1, S[2], S[0]));
        return (m1 & 0x00020002u) | (m0 & 0x00010001u);
    } else if constexpr (BITS == 3) {
        const uint32_t m2 = gt2<T>(x2, S[3]);
        const uint32_t m1 = gt2<T>(x2, sel2(m2, S[5], S[1]));
        const uint32_t m0 = gt2<T>(x2, sel2(m1, sel2(m2, S[6], S[2]), sel2(m2, S[4], S[0])));
        uint32_t c = m2 & 0x00040004u;
        c |= m1 & 0x00020002u;
        return c | (m0 & 0x00010001u);
    } else {
        const uint32_t m3 = gt2<T>(x2, S[7]);
        const uint32_t m2 = gt2<T>(x2, sel2(m3, S[11], S[3]));
        const uint32_t m1 = gt2<T>(x2, sel2(m2, sel2(m3, S[13], S[5]), sel2(m3, S[9], S[1])));
        uint32_t c = m3 & 0x00080008u;
        c |= m2 & 0x00040004u;
        c |= m1 & 0x00020002u;
        uint32_t last;                                              // the boundaries S[c_lo], S[c_hi] of the last step
        if (pair_table != 0) {
            // one shared-memory word indexed by both 3-bit prefixes instead of seven selects
            // word index 8 * (low prefix) + (high prefix): the prefixes sit doubled in bytes 0 and 2 of c, so
            // one byte-wise dot product with the weights (16, 0, 2, 0) is the byte offset
            asm("ld.shared.u32 %0, [%1];" : "=r"(last) : "r"(__dp4a(c, 0x00020010u, pair_table)));
        } else {
            const uint32_t e0 = sel2(m3, S[8], S[0]), e1 = sel2(m3, S[10], S[2]);
            const uint32_t e2 = sel2(m3, S[12], S[4]), e3 = sel2(m3, S[14], S[6]);
            last = sel2(m1, sel2(m2, e3, e1), sel2(m2, e2, e0));
        }
        const uint32_t m0 = gt2<T>(x2, last);
        return c | (m0 & 0x00010001u);
    }
}

// ---------------------------------------------------------------------------
// indexed search (binary32, 4 bits): the same binary search as bucketize<BITS>, but the boundary
// of each step is read from a 16-word shared-memory copy of the table at the index the previous
// steps produced, instead of being picked by a tree of selects: per element and level one load,
// one comparison and one predicated add (11 instructions at 4 bits against ~19).  The 16 words
// lie in 16 different banks, so a warp's load is one wavefront whatever the indices.  Measured
// against the select tree (L2-cold, 2^22 .. 2^28 elements): 4 bits, tanh 30.7 -> 28.0 us and leaky
// ReLU 27.9 -> 25.2 us at 2^24, 420 -> 394 and 384 -> 350 us at 2^28, SiLU equal; slower at 3 bits
// (the tree is 4 selects there) and for GELU, whose arithmetic leaves the ALU pipe that runs the
// selects idle anyway (39.9 -> 42.8 us): used at 4 bits for every activation but GELU.  Each warp
// keeps its own copy of the 16 words, written by the warp itself: a CTA-wide barrier in front of a
// CTA that lives for one warp-block per warp cost 6-10 % (tanh at 2^24: 28.0 -> 26.1 us, leaky ReLU
// 25.0 -> 23.6, sigmoid at 2^23: 18.2 -> 16.4).
// Returns 4 * code (the running byte offset); `first` is the middle boundary.
// ---------------------------------------------------------------------------
template <int BITS>
__device__ __forceinline__ uint32_t bucketize_indexed(uint32_t thr, float first, float x) {
    uint32_t c4 = first < x ? (4u << (BITS - 1)) : 0u;
#pragma unroll
    for (int h = BITS - 2; h >= 0; --h) {
        float sj;
        asm("ld.shared.f32 %0, [%1];" : "=f"(sj) : "r"(thr + c4 + 4u * ((1u << h) - 1u)));
        c4 += sj < x ? (4u << h) : 0u;
    }
    return c4;
}

// y values (o) and the 8 * BITS-bit code group of one lane-chunk: activation, interval search (whichever
// variant the instantiation uses) and the merge of the eight codes.
template <int ACT, int BITS, typename T, bool LUT, bool FOLD, bool kIndexed>
__device__ __forceinline__ uint32_t chunk_codes(const Raw<T> &c, float (&o)[8], const FwdParams &prm, const uint8_t *lut, const float *thr,
                                                uint32_t pair_table, uint32_t thr_idx) {
    constexpr bool kIsBf16 = sizeof(T) == 2;
    uint32_t g = 0;
    [[maybe_unused]] uint32_t dense = 0;
    [[maybe_unused]] uint32_t pc[4];                        // bfloat16: codes of element pair i, low @0, high @16
#pragma unroll
    for (int e = 6; e >= 0; e -= 2) {                       // two neighbouring elements at a time
        const float2 xv = make_float2(elem(c, e), elem(c, e + 1));
        const float2 yv = activation2<ACT, T>(xv);
        o[e] = yv.x;
        o[e + 1] = yv.y;
        if constexpr (kIsBf16) {
            if constexpr (LUT) {
                pc[e / 2] = lut[cell(c, e)] + (static_cast<uint32_t>(lut[cell(c, e + 1)]) << 16);
            } else {
                pc[e / 2] = bucketize_bf16x2<BITS, T>(prm.sb2, FOLD ? (pair_bits(c, e) & 0x7fff7fffu) : pair_bits(c, e), pair_table);
            }
        } else {
            uint32_t c0, c1;
            const float k0 = FOLD ? fabsf(xv.x) : xv.x, k1 = FOLD ? fabsf(xv.y) : xv.y;   // what is searched for
            if constexpr (kIndexed) {
                const float mid = prm.tb.s[(1 << (BITS - 1)) - 1];
                c0 = bucketize_indexed<BITS>(thr_idx, mid, k0);
                c1 = bucketize_indexed<BITS>(thr_idx, mid, k1);
                c0 = ((c1 << BITS) + c0) >> 2;              // both codes at once: (c1 << BITS) + c0
                c1 = 0;
            } else if constexpr (!LUT) {
                c0 = bucketize<BITS>(prm.tb, k0);
                c1 = bucketize<BITS>(prm.tb, k1);
            } else {
                const uint32_t m0 = lut[cell(c, e)], m1 = lut[cell(c, e + 1)];
                dense |= m0 | m1;
                c0 = (m0 & 15u) + (thr[m0 & 15u] < k0 ? 1u : 0u);
                c1 = (m1 & 15u) + (thr[m1 & 15u] < k1 ? 1u : 0u);
            }
            g = kIndexed ? (g << (2 * BITS)) + c0 : (((g << BITS) + c1) << BITS) + c0;
        }
    }
    if constexpr (kIsBf16) {
        // eight codes -> one 8*BITS-bit group: merge pairs two by two while the low and the
        // high elements still sit in separate halves, then fold the high half next to the low
        const uint32_t a01 = pc[0] + (pc[1] << (2 * BITS)), a23 = pc[2] + (pc[3] << (2 * BITS));
        constexpr uint32_t kFold = (1u << BITS) - (1u << 16);               // hi * 2^16 -> hi * 2^BITS
        const uint32_t b01 = a01 + (a01 >> 16) * kFold, b23 = a23 + (a23 >> 16) * kFold;
        g = b01 + (b23 << (4 * BITS));
    }
    if constexpr (LUT && !kIsBf16) {
        if (__any_sync(0xffffffffu, dense & 0x80u)) {        // a dense cell: redo this tile's codes by search
            g = 0;
#pragma unroll
            for (int e = 7; e >= 0; --e)
                g = (g << BITS) + bucketize<BITS>(prm.tb, FOLD ? fabsf(elem(c, e)) : elem(c, e));
        }
    }
    return g;
}

// FOLD: the code is the position of |x| (even f', table on [0, B]); the code tables arrive already
// built that way, the searches strip the sign first.
template <int ACT, int BITS, typename T, bool LUT, bool FOLD, bool BIAS = false, bool TILE = false>
__global__ void __launch_bounds__((FwdThreads<T, LUT, kThinWarps<ACT, BITS>>::value), (FwdCtas<T, LUT>::value))
fwd_kernel(const __grid_constant__ FwdParams prm, const T *x, T *y, uint32_t *packed, size_t n, int iters, unsigned long_ctas) {
    pdl_launch_dependents();
    constexpr bool kIsBf16 = sizeof(T) == 2;
    constexpr int kFwdThreads = FwdThreads<T, LUT, kThinWarps<ACT, BITS>>::value;
    constexpr int kCells = kIsBf16 ? (1 << kCellBitsBf16) : (1 << kCellBitsF32);
    extern __shared__ __align__(16) uint8_t smem_raw[];
    uint8_t *lut = smem_raw;
    const float *thr = reinterpret_cast<const FwdSmem *>(smem_raw + kCells)->thr;

    const int lane = threadIdx.x & 31;
    const bool wide = prm.flags & kWideData, vec = prm.flags & kVecPacked;
    const size_t warps = blockDim.x >> 5;                                        // stride between a warp's warp-blocks (<= kFwdThreads / 32)
    // Static partition: the first long_ctas CTAs own warps * iters warp-blocks each, the rest of the
    // grid warps * 1 (short CTAs at the end of the launch order fill the tail that the long ones
    // leave when they finish at different times).
    if (blockIdx.x >= long_ctas) iters = 1;
    const size_t cta_begin = blockIdx.x < long_ctas
        ? static_cast<size_t>(blockIdx.x) * warps * iters
        : static_cast<size_t>(long_ctas) * warps * prm.long_iters + static_cast<size_t>(blockIdx.x - long_ctas) * warps;
    const size_t warp0 = cta_begin + (threadIdx.x >> 5);
    const size_t all_full = n / kWarpElems;
    const size_t cta_end = cta_begin + warps * iters;
    // Table variants may hand out warp-blocks dynamically.  Their grid is one wave of long-lived CTAs
    // (the table is expanded once per CTA), and with a static partition the SMs that get less
    // bandwidth finish late: 10-14 % of the kernel time at 2^28 elements.  A warp starts with the
    // warp-block of its global warp number and takes the next unclaimed one from a counter in global
    // memory, two iterations ahead of use, so the atomic's latency hides behind a warp-block of work.
    // The claims go through kQueues counters, 256 bytes apart: counter q serves the warps whose
    // global number is congruent to q and hands out the warp-blocks congruent to q (one address
    // alone sustains only ~0.4 G atomics per second; every SM has warps in every group, so the
    // groups finish together).
    const bool dynamic = LUT && prm.queue != nullptr && gridDim.x * warps >= kQueues;   // every counter needs a warp that draws from it
    const size_t full = dynamic ? all_full : (all_full < cta_end ? all_full : cta_end);   // static: this CTA's warp-blocks are [cta_begin, full)
    const uint32_t global_warp = blockIdx.x * static_cast<uint32_t>(warps) + (threadIdx.x >> 5);
    const size_t first_wb = dynamic ? global_warp : warp0;
    auto next_after = [&](size_t wb) -> size_t {
        if constexpr (LUT) {
            if (dynamic) {
                uint32_t v = 0;
                if (lane == 0) v = atomicAdd(prm.queue + (global_warp % kQueues) * kQueueStride, 1u);
                v = __shfl_sync(0xffffffffu, v, 0);
                return static_cast<size_t>(gridDim.x) * warps + static_cast<size_t>(v) * kQueues + global_warp % kQueues;
            }
        }
        return wb + warps;
    };
    constexpr int kStages = LUT ? (kIsBf16 ? FEWBIT_LUT_STAGES_BF16 : 0) : kAsyncStages<T, kThinWarps<ACT, BITS>>;   // 0: prefetch into registers
    static_assert(kStages >= 0 && kStages <= 2, "the loop tracks two warp-blocks ahead");
    constexpr uint32_t kRingOffset = LUT ? (kCells + static_cast<uint32_t>(sizeof(FwdSmem)) + 127u) / 128u * 128u : 0u;
    constexpr uint32_t kChunkBytes = kLaneElems * sizeof(T);
    constexpr uint32_t kStageBytes = kTilesPerWarp * 32 * kChunkBytes;          // one warp-block
    [[maybe_unused]] uint32_t ring = 0, stage = 0;                  // this lane's slot base in the ring; stage in use
    // Software pipeline.  Without a code table: the cp.async ring above, kStages warp-blocks ahead.
    // With one (shared memory is taken): as soon as a tile of the current warp-block has been
    // consumed, the same registers are reloaded with that tile of the warp's next warp-block, so
    // four loads per lane stay in flight while the warp computes.
    // The 64 KB table of the 16-bit types is expanded before the wait on the previous kernel of the
    // stream (it touches shared memory and kernel parameters only), so under programmatic dependent
    // launch it overlaps that kernel's tail; the 8 KB binary32 table is expanded behind the first
    // loads instead (its CTAs may be short, and each would pay the serialisation).
    constexpr bool kExpandFirst = LUT && kIsBf16;
    if constexpr (kExpandFirst) {
        FwdSmem &sm = *reinterpret_cast<FwdSmem *>(smem_raw + kCells);
        if (threadIdx.x < kMaxLevels) sm.thr[threadIdx.x] = prm.tb.s[threadIdx.x];
        expand_runs<kCells, kFwdThreads>(prm.runs, lut, sm);
    }
    // 4 bits, packed search: the boundary pair of the last comparison, for every pair of 3-bit
    // prefixes (low element * 8 + high element), 64 words
    [[maybe_unused]] uint32_t pair_table = 0;
    if constexpr (kIsBf16 && !LUT && BITS == 4) {
        // one copy per warp, filled by the warp itself: no CTA-wide barrier at the start of these short-lived CTAs
        __shared__ uint32_t last_pair[kFwdThreads / 32][64];
        uint32_t *mine = last_pair[threadIdx.x >> 5];
#pragma unroll
        for (uint32_t i = lane; i < 64; i += 32)
            mine[i] = (prm.sb2[2 * (i >> 3)] & 0x0000ffffu) | (prm.sb2[2 * (i & 7)] & 0xffff0000u);
        __syncwarp();
        pair_table = static_cast<uint32_t>(__cvta_generic_to_shared(mine));
    }
    // binary32 without a code table, 4 bits: the boundaries in shared memory for the indexed search
    constexpr bool kIndexed = FEWBIT_INDEXED_SEARCH && !kIsBf16 && !LUT && BITS == 4 && ACT != FEWBIT_GELU;
    [[maybe_unused]] uint32_t thr_idx = 0;
    if constexpr (kIndexed) {
        __shared__ float thr_s[kFwdThreads / 32][kMaxLevels];       // one copy per warp: no CTA-wide barrier
        float *mine = thr_s[threadIdx.x >> 5];
        if (lane < kMaxLevels) mine[lane] = prm.tb.s[lane];
        __syncwarp();
        thr_idx = static_cast<uint32_t>(__cvta_generic_to_shared(mine));
    }
    pdl_wait();                                                     // nothing above touches global memory
    // Tile mode (small tensors, variants without a code table): one 256-element tile per warp instead
    // of a 1024-element warp-block, so that a tensor of a few hundred thousand elements still puts
    // several warps on every scheduler.  The four lanes of a quad hold 32 consecutive codes between
    // them: each lane fetches the other three groups by shuffle, assembles the BITS words and lane r
    // of the quad stores word r.  Same bit stream as the warp-block path.
    // A separate instantiation (TILE), so that the warp-block path compiles exactly as without it.
    [[maybe_unused]] size_t tile_tail_begin = 0;                    // tile mode: first element of the ragged tail
    [[maybe_unused]] bool tile_tail_owner = false;
    if constexpr (TILE) {
        static_assert(!LUT, "tile mode has no code table");
        {
            const size_t tile = static_cast<size_t>(blockIdx.x) * warps + (threadIdx.x >> 5);
            const size_t full_tiles = n / kTileElems;
            if (tile < full_tiles) {
                const size_t base = tile * kTileElems + static_cast<size_t>(lane) * kLaneElems;
                Raw<T> c;
                load_raw(x + base, c, wide);
                if constexpr (BIAS) {
                    const uint64_t chunk = tile * 32;                        // number of the tile's first lane-chunk
                    const uint32_t row_chunks = prm.cols / kLaneElems;
                    const uint64_t rem = chunk < (1ull << 32) ? chunk - __umul64hi(chunk, prm.chunks_magic) * row_chunks : chunk % row_chunks;
                    uint64_t col = (rem + lane) * kLaneElems;
                    if (col >= prm.cols) col = prm.cols >= kTileElems ? col - prm.cols : col % prm.cols;
                    add_bias(c, static_cast<const T *>(prm.bias) + col, wide);
                }
                float o[8];
                const uint32_t g = chunk_codes<ACT, BITS, T, LUT, FOLD, kIndexed>(c, o, prm, lut, thr, pair_table, thr_idx);
                store8(y + base, o, wide);
                uint32_t grp[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) grp[j] = __shfl_sync(0xffffffffu, g, (lane & ~3) + j);
                uint32_t w[BITS];
                groups_to_words<BITS>(grp, w);
                const int r = lane & 3;
                if (r < BITS) {
                    uint32_t word = w[0];
#pragma unroll
                    for (int j = 1; j < BITS; ++j) word = r == j ? w[j] : word;
                    packed[tile * (8 * BITS) + (lane >> 2) * BITS + r] = word;
                }
                return;
            }
            tile_tail_begin = full_tiles * kTileElems;
            tile_tail_owner = tile == full_tiles;
            if (!tile_tail_owner) return;
        }
    }
    if constexpr (!TILE) {                                          // (in tile mode only the tail's owner gets here, and skips to the tail)
    Raw<T> cur[kTilesPerWarp];
    size_t wb = first_wb;                                           // the warp-block in hand, the one after it,
    size_t nxt = wb < full ? next_after(wb) : full;                 // and (inside the loop) the one after that
    if constexpr (kStages > 0) {
        ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw)) + kRingOffset + (threadIdx.x >> 5) * (kStages * kStageBytes) +
               lane * kChunkBytes;
#pragma unroll
        for (int s = 0; s < kStages; ++s) {
            const size_t wbs = s == 0 ? wb : nxt;
            if (wbs < full) {
                const T *px = x + wbs * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
#pragma unroll
                for (int t = 0; t < kTilesPerWarp; ++t)
                    cp_async_chunk(ring + s * kStageBytes + t * (32 * kChunkBytes), px + t * kTileElems);
            }
            cp_async_commit();
        }
    } else if (wb < full) {
        const T *px = x + wb * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) load_raw(px + t * kTileElems, cur[t], wide);
    }
    if constexpr (LUT && !kExpandFirst) {                           // expanded while the first loads are in flight
        FwdSmem &sm = *reinterpret_cast<FwdSmem *>(smem_raw + kCells);
        if (threadIdx.x < kMaxLevels) sm.thr[threadIdx.x] = prm.tb.s[threadIdx.x];
        expand_runs<kCells, kFwdThreads>(prm.runs, lut, sm);
    }
    while (wb < full) {
        const size_t base = wb * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
        T *py = y + base;
        const bool more = nxt < full;
        const size_t nxt2 = more ? next_after(nxt) : full;
        const T *px_next = x + nxt * kWarpElems + static_cast<size_t>(lane) * kLaneElems;   // read only if `more`
        uint32_t grp[4];
        // with a bias: this lane's bias values for tile 0 of the warp-block (a row is a whole number of warp-blocks)
        // with a bias: the column of this lane's chunk in tile 0 of the warp-block (one 64-bit remainder
        // per warp-block; the tiles that follow add 256 and wrap around the row end)
        [[maybe_unused]] uint64_t col0 = 0;
        [[maybe_unused]] bool one_row = false;                      // the whole warp-block lies in one row (warp-uniform)
        if constexpr (BIAS) {
            const uint64_t chunk = wb * (kWarpElems / kLaneElems);          // number of the warp-block's first lane-chunk
            const uint32_t row_chunks = prm.cols / kLaneElems;
            const uint64_t rem = chunk < (1ull << 32) ? chunk - __umul64hi(chunk, prm.chunks_magic) * row_chunks : chunk % row_chunks;
            one_row = (rem + kWarpElems / kLaneElems) * kLaneElems <= prm.cols;
            col0 = (rem + lane) * kLaneElems;
        }
        if constexpr (kStages > 0) cp_async_wait<(kStages > 0 ? kStages - 1 : 0)>();   // the oldest stage has landed
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) {
            if constexpr (kStages > 0) load_raw_shared(ring + stage * kStageBytes + t * (32 * kChunkBytes), cur[t]);
            if constexpr (BIAS) {
                if (one_row) {
                    add_bias(cur[t], static_cast<const T *>(prm.bias) + col0 + t * kTileElems, wide);
                } else {
                    uint64_t col = col0 + static_cast<uint64_t>(t) * kTileElems;
                    if (col >= prm.cols) col = prm.cols >= kWarpElems ? col - prm.cols : col % prm.cols;
                    add_bias(cur[t], static_cast<const T *>(prm.bias) + col, wide);
                }
            }
            float o[8];
            const uint32_t g = chunk_codes<ACT, BITS, T, LUT, FOLD, kIndexed>(cur[t], o, prm, lut, thr, pair_table, thr_idx);
            grp[t] = g;
            store8(py + t * kTileElems, o, wide);
            if constexpr (kStages == 0) {
                if (more) load_raw(px_next + t * kTileElems, cur[t], wide);
            }
        }
        if constexpr (kStages > 0) {                               // refill the stage just consumed
            const size_t wbn = kStages == 2 ? nxt2 : nxt;
            if (wbn < full) {
                const T *px = x + wbn * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
#pragma unroll
                for (int t = 0; t < kTilesPerWarp; ++t)
                    cp_async_chunk(ring + stage * kStageBytes + t * (32 * kChunkBytes), px + t * kTileElems);
            }
            cp_async_commit();
            stage = (stage + 1 == kStages) ? 0 : stage + 1;
        }
        quad_transpose(grp, lane);
        uint32_t w[BITS];
        groups_to_words<BITS>(grp, w);
        store_words<BITS>(packed + wb * (32 * BITS) + (lane & 3) * (8 * BITS) + (lane >> 2) * BITS, w, vec);
        wb = nxt;
        nxt = nxt2;
    }
    }

    // ragged tail: the one warp whose sequence warp0, warp0 + warps, ... reaches the index of the last,
    // partial warp-block (all_full >= warp0 keeps the unsigned difference from wrapping: 2^64 is not a
    // multiple of every CTA width); a lane owns 32 consecutive elements = BITS words
    const bool owns_tail = TILE ? true : dynamic ? (blockIdx.x == 0 && threadIdx.x < 32)
                                   : (all_full >= warp0 && all_full < cta_end && (all_full - warp0) % warps == 0);
    const size_t tail_begin = TILE ? tile_tail_begin : all_full * kWarpElems;   // first element of the ragged tail
    if ((TILE ? tail_begin != n : (n % kWarpElems) != 0) && owns_tail) {
        if (prm.tail_counter != nullptr && lane == 0) atomicAdd(prm.tail_counter, 1u);
        const size_t base = tail_begin + static_cast<size_t>(lane) * 32;
        uint32_t w[BITS + 1];
#pragma unroll
        for (int j = 0; j <= BITS; ++j) w[j] = 0;
        // eight loads at a time ahead of their stores: y may alias x, so the compiler cannot move a load
        // above a store, and 32 load-use-store rounds in a row would each pay the full memory latency
#pragma unroll
        for (int e0 = 0; e0 < 32; e0 += 8) {
            float xs[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = e0 + i;
                xs[i] = 0.0f;
                if (base + e < n) {
                    xs[i] = load1(x + base + e);
                    if constexpr (BIAS)                              // the sum rounded once to the storage type
                        xs[i] = round_to<T>(__fadd_rn(xs[i], load1(static_cast<const T *>(prm.bias) + (base + e) % prm.cols)));
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int e = e0 + i;
                if (base + e < n) {
                    const float xv = xs[i];
                    store1(y + base + e, activation<ACT, T>(xv));
                    const uint32_t c = bucketize<BITS>(prm.tb, FOLD ? fabsf(xv) : xv);
                    const int pos = e * BITS;
                    w[pos >> 5] |= c << (pos & 31);
                    if ((pos & 31) + BITS > 32) w[(pos >> 5) + 1] |= c >> (32 - (pos & 31));
                }
            }
        }
        const size_t total_words = (n * BITS + 31) / 32;
        const size_t first = (TILE ? tail_begin / 32 * BITS : all_full * (32 * BITS)) + static_cast<size_t>(lane) * BITS;
#pragma unroll
        for (int j = 0; j < BITS; ++j)
            if (first + j < total_words) packed[first + j] = w[j];
    }

    // Dynamic distribution: the last CTA of the grid to get here puts the work counters back to
    // zero for the next launch that leases them (every warp has made its last claim by then).
    if constexpr (LUT) {
        if (dynamic) {                                              // uniform over the grid
            __syncthreads();
            if (threadIdx.x == 0) {
                __threadfence();
                if (atomicAdd(prm.queue + kQueueDoneWord, 1u) == gridDim.x - 1) {
#pragma unroll
                    for (uint32_t q = 0; q < kQueues; ++q) prm.queue[q * kQueueStride] = 0;
                    prm.queue[kQueueDoneWord] = 0;
                    __threadfence();
                }
            }
        }
    }
}

template <typename T, bool LUT, bool THIN>
constexpr size_t fwd_smem_bytes() {
    return LUT ? ((sizeof(T) == 2 ? (1u << kCellBitsBf16) : (1u << kCellBitsF32)) + sizeof(FwdSmem) + 127u) / 128u * 128u +
                     (sizeof(T) == 2 ? static_cast<size_t>(FEWBIT_LUT_STAGES_BF16) * (FwdThreads<T, true>::value / 32) * kWarpElems * sizeof(T) : 0)
               : static_cast<size_t>(kAsyncStages<T, THIN>) * (FwdThreads<T, false, THIN>::value / 32) * kWarpElems * sizeof(T);
}

int device_sm_count(cudaError_t *err);   // of the current device, cached

// How much arithmetic an activation costs in binary32: 0 = a few instructions (ReLU, leaky ReLU),
// 1 = one exponential or tanh, 2 = enough to make the forward kernel issue-bound (GELU, SiLU).
constexpr int act_weight(int act) {
    return (act == FEWBIT_RELU || act == FEWBIT_LEAKY_RELU) ? 0
         : (act == FEWBIT_GELU || act == FEWBIT_SILU) ? 2 : 1;
}
// Tile mode below this many warp-blocks per resident warp (numerator / denominator), measured L2-cold
// in batches of 8 launches, tile mode against warp-blocks: binary32 at 2^20 elements GELU 3 bits
// 6.4 -> 5.1 us, SiLU 4 bits 6.1 -> 4.4; at 2^21 10.0 -> 7.4 and 9.2 -> 6.4; 2^14 .. 2^19: 3.6-4.9 ->
// 2.3-4.1; from 2^22 (one wave) on equal or slower.  16-bit types: 2^20 4.0-4.4 -> 3.3-3.6 us, 2^21
// 5.6-6.1 -> 4.9-5.1 (the cheapest, 1-bit leaky ReLU: 3.8 -> 4.4), 2^22 (0.86 waves) 6.1-7.7 -> 6.7-8.7:
// hence one half.
template <typename T> constexpr size_t kTileModeNum = 1;
template <typename T> constexpr size_t kTileModeDen = sizeof(T) == 2 ? 2 : 1;
constexpr size_t kLutMinIters = 8;      // below this many warp-blocks per warp the table does not pay for its expansion
int fwd_iters_override();                // FEWBIT_OPT_FWD_ITERS: 0 = the size-based choice
bool pdl_enabled();                      // FEWBIT_OPT_PDL
int fwd_warps_override();                // FEWBIT_OPT_FWD_WARPS (variants without a table): 0 = the default
int fwd_tile_mode();                     // FEWBIT_OPT_FWD_TILE: 0 = by size, 1 = tile mode whenever there is no table, 2 = never

template <int ACT, int BITS, typename T, bool LUT, bool FOLD, bool BIAS = false>
cudaError_t launch_fwd(const FwdParams &prm, const void *x, void *y, uint32_t *packed, size_t n, cudaStream_t st) {
    cudaError_t err = cudaSuccess;
    const int sms = device_sm_count(&err);
    if (err != cudaSuccess) return err;
    constexpr bool kThin = kThinWarps<ACT, BITS>;
    constexpr size_t smem = fwd_smem_bytes<T, LUT, kThin>();
    auto kernel = fwd_kernel<ACT, BITS, T, LUT, FOLD, BIAS>;
    if constexpr (smem > 48 * 1024) {           // opt in to the large dynamic shared memory once per device
        static std::atomic<uint64_t> opted_in{0};
        int dev = 0;
        err = cudaGetDevice(&dev);
        if (err != cudaSuccess) return err;
        const uint64_t bit = 1ull << (dev & 63);
        if (!(opted_in.load(std::memory_order_relaxed) & bit)) {
            err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
            if (err != cudaSuccess) return err;
            opted_in.fetch_or(bit, std::memory_order_relaxed);
        }
    }
    constexpr int kFwdThreads = FwdThreads<T, LUT, kThin>::value;
    // Without a table the CTA size is free (a warp's work does not depend on it): 4-warp CTAs fill
    // and drain the SMs more evenly than the 12 or 16 warps the kernel is compiled for (binary32
    // sigmoid, 51 M elements: 74.7 -> 70.6 us; bfloat16 SiLU, 12.6 M: 15.0 -> 12.9 us).
    size_t warps_per_cta = kFwdThreads / 32;
    if constexpr (!LUT) {
        warps_per_cta = 4;
        const int v = fwd_warps_override();
        if (v >= 1 && v <= kFwdThreads / 32) warps_per_cta = static_cast<size_t>(v);
    }
    const size_t warp_blocks = n / kWarpElems + ((n % kWarpElems) ? 1 : 0);
    // Iterations per warp.  Without a table: two from about 1.5 waves of resident warps on (the
    // prefetch ring then overlaps a warp's loads with its arithmetic), at most 4 (short CTAs let
    // the block scheduler even out SMs that run slow); binary32 measured fastest with one at every
    // size (its loads are twice as wide, and more, shorter CTAs balance better).  With the 64 KB
    // table of the 16-bit types the expansion has to be amortised: exactly one wave, every CTA
    // resident from the start (the caller only picks that variant when this gives each warp at
    // least kLutMinIters iterations).
    const size_t slots = static_cast<size_t>(sms) * FwdCtas<T, LUT>::value * (kFwdThreads / 32) / warps_per_cta;
    size_t iters;
    if constexpr (LUT) {
        const size_t waves = (warp_blocks + warps_per_cta * slots - 1) / (warps_per_cta * slots);
        iters = waves;
        if constexpr (sizeof(T) == 4) {
            // The binary32 table is 8 KB: cheap to expand, so the CTAs may be short.  Measured at
            // 2^22 .. 2^27 elements: kernels that stay memory-bound want short CTAs (the one-wave
            // grid loses ~15 % to imbalance), issue-bound ones want the long-lived CTAs of one wave
            // (every CTA start is a bubble in which its SM partner cannot fill the issue slots alone).
            constexpr int kWeight = act_weight(ACT);
            if (prm.queue != nullptr) {
                // dynamic distribution: one wave, balanced by the work counters (measured against the
                // short static CTAs at 2^27: sigmoid 194 -> 177 us, SiLU 190 -> 183 us, tanh equal)
            } else if (kWeight < 2 || waves < kLutMinIters) {
                iters = waves / 2;
                const size_t cap = kWeight == 0 ? 1 : 4;
                iters = iters < 1 ? 1 : (iters > cap ? cap : iters);
            }
        }
    } else {
        iters = sizeof(T) == 2 ? warp_blocks * 2 / (warps_per_cta * slots * 3) : 1;
        iters = iters < 1 ? 1 : (iters > 4 ? 4 : iters);
    }
    if (const int forced = fwd_iters_override(); forced >= 1) iters = static_cast<size_t>(forced);
    // When the CTAs take several warp-blocks per warp, the last wave's worth of warp-blocks goes to
    // short CTAs (one warp-block per warp) at the end of the launch order: they fill the tail that
    // the long CTAs leave when they finish at different times (2^26 elements: 50.2 -> 48.1 us,
    // 2^28: 171 -> 169 us).  Without a table only (a table variant is one wave).
    const size_t per_cta = warps_per_cta * iters;
    size_t short_blocks = 0;
    if (!LUT && iters > 1) {
        short_blocks = warps_per_cta * slots;
        if (short_blocks > warp_blocks) short_blocks = warp_blocks;
    }
    const size_t long_ctas = (warp_blocks - short_blocks) / per_cta;
    const size_t rest = warp_blocks - long_ctas * per_cta;               // done by short CTAs (or, if none are wanted, one more long one)
    const size_t short_ctas = short_blocks ? (rest + warps_per_cta - 1) / warps_per_cta : (rest + per_cta - 1) / per_cta;
    const unsigned grid = static_cast<unsigned>(long_ctas + short_ctas);
    FwdParams p2 = prm;
    p2.long_iters = static_cast<uint32_t>(iters);
    const unsigned n_long = short_blocks ? static_cast<unsigned>(long_ctas) : grid;
    // Programmatic dependent launch lets this grid's CTAs take their places while the previous kernel
    // of the stream drains (they wait there for it to complete): back-to-back launches of small
    // tensors go from 4.2 us to ~2 us apiece, and no size or activation measured slower with it
    // (batches of 8 launches, 2^16 .. 2^28 elements).
    const bool pdl = pdl_enabled();
    if constexpr (!LUT) {
        // Tile mode for small tensors: with fewer warp-blocks than a fraction of the resident warps, a
        // 256-element tile per warp puts four times as many warps to work (measurements at kTileModeNum).
        const int mode = fwd_tile_mode();
        const size_t resident_warps = slots * warps_per_cta;
        if (mode == 1 || (mode == 0 && warp_blocks * kTileModeDen<T> < resident_warps * kTileModeNum<T>)) {
            const size_t tiles = n / kTileElems + ((n % kTileElems) ? 1 : 0);
            const unsigned tgrid = static_cast<unsigned>((tiles + warps_per_cta - 1) / warps_per_cta);
            return launch_pdl(fwd_kernel<ACT, BITS, T, false, FOLD, BIAS, true>, tgrid, static_cast<unsigned>(warps_per_cta * 32), 0, st, pdl,
                              p2, static_cast<const T *>(x), static_cast<T *>(y), packed, n, 1, tgrid);
        }
    }
    return launch_pdl(kernel, grid, static_cast<unsigned>(warps_per_cta * 32), smem * warps_per_cta / (kFwdThreads / 32), st, pdl,
                      p2, static_cast<const T *>(x), static_cast<T *>(y), packed, n, static_cast<int>(iters), n_long);
}

using FwdLaunch = cudaError_t (*)(const FwdParams &, const void *, void *, uint32_t *, size_t, cudaStream_t);

// Launchers of one activation: [bits - 1][dtype: f32, bf16, f16][use look-up table][folded table]
// and, for f(x + bias) (no folded tables): [bits - 1][dtype][use look-up table]
struct FwdLaunchers { FwdLaunch fn[kMaxBits][3][2][2]; FwdLaunch with_bias[kMaxBits][3][2]; };

template <int ACT, int BITS, bool FOLD>
constexpr void fill_fwd_launchers(FwdLaunchers &l) {
    // 1-2 bit binary32 tables: the search is 1-3 comparisons, cheaper than the table;
    // 16-bit types: the packed search is 1-3 comparisons per element pair
    constexpr bool kLutF32 = BITS >= 3, kLutBf16 = BITS >= 3;
    l.fn[BITS - 1][0][0][FOLD] = launch_fwd<ACT, BITS, float, false, FOLD>;
    l.fn[BITS - 1][0][1][FOLD] = launch_fwd<ACT, BITS, float, kLutF32, FOLD>;
    l.fn[BITS - 1][1][0][FOLD] = launch_fwd<ACT, BITS, __nv_bfloat16, false, FOLD>;
    l.fn[BITS - 1][1][1][FOLD] = launch_fwd<ACT, BITS, __nv_bfloat16, kLutBf16, FOLD>;
    l.fn[BITS - 1][2][0][FOLD] = launch_fwd<ACT, BITS, __half, false, FOLD>;
    l.fn[BITS - 1][2][1][FOLD] = launch_fwd<ACT, BITS, __half, kLutBf16, FOLD>;
    if constexpr (!FOLD) {
        l.with_bias[BITS - 1][0][0] = launch_fwd<ACT, BITS, float, false, false, true>;
        l.with_bias[BITS - 1][0][1] = launch_fwd<ACT, BITS, float, kLutF32, false, true>;
        l.with_bias[BITS - 1][1][0] = launch_fwd<ACT, BITS, __nv_bfloat16, false, false, true>;
        l.with_bias[BITS - 1][1][1] = launch_fwd<ACT, BITS, __nv_bfloat16, kLutBf16, false, true>;
        l.with_bias[BITS - 1][2][0] = launch_fwd<ACT, BITS, __half, false, false, true>;
        l.with_bias[BITS - 1][2][1] = launch_fwd<ACT, BITS, __half, kLutBf16, false, true>;
    }
}

template <int ACT>
FwdLaunchers make_fwd_launchers() {
    FwdLaunchers l{};
    fill_fwd_launchers<ACT, 1, false>(l);
    fill_fwd_launchers<ACT, 2, false>(l);
    fill_fwd_launchers<ACT, 3, false>(l);
    fill_fwd_launchers<ACT, 4, false>(l);
    if constexpr (ACT == FEWBIT_SIGMOID || ACT == FEWBIT_TANH) {       // even f': folded tables exist
        fill_fwd_launchers<ACT, 1, true>(l);
        fill_fwd_launchers<ACT, 2, true>(l);
        fill_fwd_launchers<ACT, 3, true>(l);
        fill_fwd_launchers<ACT, 4, true>(l);
    }
    return l;
}

const FwdLaunchers &fwd_launchers(int act);   // defined by the per-activation translation units

}  // namespace fewbit
