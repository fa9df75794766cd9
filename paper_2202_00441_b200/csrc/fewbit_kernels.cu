// Backward half of Listing 1 for sm_100a, the dispatch tables and the two
// DEVICE-pointer entry points of the C ABI.
#include <atomic>

#include "fewbit_fwd.cuh"

namespace fewbit {

std::atomic<uint64_t> g_launches{0};
thread_local int t_last_cuda_error = 0;

// ---------------------------------------------------------------------------
// Backward: grad_in = grad_out * lev[code]   (binary32 multiply, one rounding)
// ---------------------------------------------------------------------------
template <int BITS, typename T>
__global__ void __launch_bounds__(kThreads)
bwd_kernel(const __grid_constant__ Levels tl, const uint32_t *packed, const T *grad_out, T *grad_in, size_t n, uint32_t flags) {
    pdl_launch_dependents();
    __shared__ float lev[kMaxLevels];
    if (threadIdx.x < kMaxLevels) lev[threadIdx.x] = tl.lev[threadIdx.x];
    __syncthreads();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const bool wide = flags & kWideData, vec = flags & kVecPacked;
    const size_t wb = static_cast<size_t>(blockIdx.x) * kWarpsPerCta + (threadIdx.x >> 5);
    const size_t full = n / kWarpElems;
    constexpr uint32_t kMask = (1u << BITS) - 1u;
    if (wb < full) {
        const size_t base = wb * kWarpElems + static_cast<size_t>(lane) * kLaneElems;
        uint32_t w[BITS];
        load_words<BITS>(packed + wb * (32 * BITS) + (lane & 3) * (8 * BITS) + (lane >> 2) * BITS, w, vec);
        float v[kTilesPerWarp][8];
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) load8(grad_out + base + t * kTileElems, v[t], wide);
        uint32_t grp[4];
        words_to_groups<BITS>(w, grp);
        quad_transpose(grp, lane);
#pragma unroll
        for (int t = 0; t < kTilesPerWarp; ++t) {
            float o[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) o[e] = __fmul_rn(v[t][e], lev[(grp[t] >> (BITS * e)) & kMask]);
            store8(grad_in + base + t * kTileElems, o, wide);
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
using BwdLaunch = cudaError_t (*)(const Levels &, const uint32_t *, const void *, void *, size_t, uint32_t, cudaStream_t);

inline unsigned bwd_grid_for(size_t n) {
    const size_t warps = n / kWarpElems + ((n % kWarpElems) ? 1 : 0);
    return static_cast<unsigned>((warps + kWarpsPerCta - 1) / kWarpsPerCta);
}

template <int BITS, typename T>
cudaError_t launch_bwd(const Levels &tl, const uint32_t *packed, const void *g, void *gi, size_t n, uint32_t flags, cudaStream_t st) {
    return launch_pdl(bwd_kernel<BITS, T>, bwd_grid_for(n), kThreads, 0, st, pdl_enabled(), tl, packed, static_cast<const T *>(g), static_cast<T *>(gi), n, flags);
}

const BwdLaunch kBwd[kMaxBits][3] = {      // [bits - 1][dtype: f32, bf16, f16]
    { launch_bwd<1, float>, launch_bwd<1, __nv_bfloat16>, launch_bwd<1, __half> },
    { launch_bwd<2, float>, launch_bwd<2, __nv_bfloat16>, launch_bwd<2, __half> },
    { launch_bwd<3, float>, launch_bwd<3, __nv_bfloat16>, launch_bwd<3, __half> },
    { launch_bwd<4, float>, launch_bwd<4, __nv_bfloat16>, launch_bwd<4, __half> },
};

const FwdLaunchers &fwd_launchers_act0();
const FwdLaunchers &fwd_launchers_act1();
const FwdLaunchers &fwd_launchers_act2();
const FwdLaunchers &fwd_launchers_act3();
const FwdLaunchers &fwd_launchers_act4();
const FwdLaunchers &fwd_launchers_act5();
const FwdLaunchers &fwd_launchers_act6();
const FwdLaunchers &fwd_launchers_act7();
const FwdLaunchers &fwd_launchers_act8();

const FwdLaunchers &fwd_launchers(int act) {
    switch (act) {
    case 0: return fwd_launchers_act0();
    case 1: return fwd_launchers_act1();
    case 2: return fwd_launchers_act2();
    case 3: return fwd_launchers_act3();
    case 4: return fwd_launchers_act4();
    case 5: return fwd_launchers_act5();
    case 6: return fwd_launchers_act6();
    case 7: return fwd_launchers_act7();
    default: return fwd_launchers_act8();
    }
}

// Number of SMs of the current device (the persistent forward grid is sized from it).
int device_sm_count(cudaError_t *err) {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return 0;
    if (dev >= 0 && dev < kMaxDevices) {
        const int c = cache[dev].load(std::memory_order_relaxed);
        if (c > 0) return c;
    }
    int sms = 0;
    *err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (*err != cudaSuccess) return 0;
    if (dev >= 0 && dev < kMaxDevices) cache[dev].store(sms, std::memory_order_relaxed);
    return sms;
}

// Process-wide options (fewbit_set_option): plain atomics, read with relaxed loads on every launch.
// No environment variable is read anywhere in the library.
constexpr int kNumOptions = 7;
std::atomic<int> g_option[kNumOptions] = {{0}, {0}, {0}, {0}, {1}, {0}, {0}};   // defaults; FEWBIT_OPT_PDL is on
inline int option(fewbit_option o) { return g_option[o].load(std::memory_order_relaxed); }

int fwd_iters_override() { return option(FEWBIT_OPT_FWD_ITERS); }
bool pdl_enabled() { return option(FEWBIT_OPT_PDL) != 0; }
int fwd_warps_override() { return option(FEWBIT_OPT_FWD_WARPS); }
int fwd_tile_mode() { return option(FEWBIT_OPT_FWD_TILE); }

inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// What the alignment of the caller's buffers allows (the rule itself -- 16 bytes for element
// buffers, 4 for the packed words -- is checked by the entry points).  a, b, c: the element buffers
// of the call (c may be NULL).
inline uint32_t access_flags(const void *a, const void *b, const void *c, const void *packed, int bits) {
    uint32_t f = 0;
    if (aligned(a, 32) && aligned(b, 32) && (c == nullptr || aligned(c, 32))) f |= kWideData;
    if (aligned(packed, bits == 2 ? 8 : 16)) f |= kVecPacked;
    return f;
}

}  // namespace fewbit

namespace fewbit {
namespace {

// The forward launch behind fewbit_fwd and fewbit_fwd_bias (bias == nullptr: none; else rows of
// `cols` elements, a multiple of the lane-chunk).
fewbit_status forward(const fewbit_table *table, const void *x, const void *bias, uint32_t cols, void *y,
                      uint32_t *packed, size_t n, fewbit_dtype dtype, void *stream) {
    FwdParams prm;
    prm.bias = bias;
    prm.cols = cols;
    prm.chunks_magic = cols > static_cast<uint32_t>(kLaneElems) ? ~0ull / (cols / kLaneElems) + 1 : 0;   // one chunk per row: remainder 0
    const bool bf16 = dtype != FEWBIT_F32;                              // a 16-bit storage type (same kernel geometry)
    for (int m = 0; m < kMaxLevels; ++m) {
        prm.tb.s[m] = table->s[m];
        prm.sb2[m] = dtype == FEWBIT_F16 ? table->s_f16x2[m] : table->s_bf16x2[m];
    }
    prm.runs = dtype == FEWBIT_F16 ? table->runs_f16 : (bf16 ? table->runs_bf16 : table->runs_f32);
    prm.queue = nullptr;
    prm.flags = access_flags(x, y, bias, packed, table->bits);
    prm.tail_counter = nullptr;
    if (option(FEWBIT_OPT_COUNT_TAILS) != 0) {
        const cudaError_t terr = tail_counter_address(&prm.tail_counter);
        if (terr != cudaSuccess) { t_last_cuda_error = static_cast<int>(terr); return FEWBIT_ERR_CUDA; }
    }
    // the shared-memory code table pays off only when every warp of a one-wave grid gets enough work
    cudaError_t sm_err = cudaSuccess;
    const size_t slots = static_cast<size_t>(device_sm_count(&sm_err)) * (bf16 ? FwdCtas<__nv_bfloat16, true>::value : FwdCtas<float, true>::value);
    if (sm_err != cudaSuccess) { t_last_cuda_error = static_cast<int>(sm_err); return FEWBIT_ERR_CUDA; }
    const size_t warps_per_cta = static_cast<size_t>(bf16 ? FwdThreads<__nv_bfloat16, true>::value : FwdThreads<float, true>::value) / 32;
    const size_t waves = n / kWarpElems / (warps_per_cta * slots);
    // 16-bit types: from how many waves on the 64 KB pattern table beats the packed search, measured
    // L2-cold at 2^24 .. 2^28 elements (3 .. 55 waves) for every activation, with dynamic distribution;
    // 0 = never.  The heavier the arithmetic of f, the earlier the table's shorter instruction stream
    // pays for its expansion and its bank conflicts; for the cheapest ones the search is faster at any size.
    //                                             gelu silu sigm tanh elu  sopl leak relu selu
    static const unsigned char kMinWavesBf16[2][FEWBIT_NUM_ACTS] = {{20,  0,   0,   0,   0,  20,  0,   0,   0},     // 3 bits
                                                                    { 3,  6,  24,   0,   6,   6, 24,   0,   6}};    // 4 bits
    static const unsigned char kMinWavesF16[2][FEWBIT_NUM_ACTS] = {{ 0,  0,   0,   0,  24,  48,  0,   0,   6},
                                                                   { 6, 24,   0,   6,   6,   6,  0,   0,   3}};
    bool use_lut = false;
    if (bf16 && prm.runs.count != 0 && table->bits >= 3) {
        const unsigned min_waves = (dtype == FEWBIT_F16 ? kMinWavesF16 : kMinWavesBf16)[table->bits - 3][table->act];
        use_lut = min_waves != 0 && waves >= min_waves;
    }
    if (!bf16 && prm.runs.count != 0) {
        // binary32 (measured L2-cold at 2^20 .. 2^28 elements against the search variants): at 4 bits the
        // 8 KB table wins from 8 waves for GELU, SiLU, sigmoid and softplus (SiLU at 2^28: 361 against 415
        // us; at 2^24, 4.6 waves, 32.2 against 30.0), from 16 for tanh (2^26: 94 against 96 us), never for
        // ELU, SELU and the ReLU-like activations, where the indexed search is faster at every size (ELU at
        // 2^28: 337 against 349 us); at 3 bits only for GELU (from 16 waves), SiLU and sigmoid (from 24: 354
        // against 367 us at 2^28) -- for the others the search in thin warps is as fast or faster at every
        // size (softplus at 2^28: 364 against 377 us)
        const int a = table->act;
        const size_t min_waves4 = (a == FEWBIT_GELU || a == FEWBIT_SILU || a == FEWBIT_SIGMOID || a == FEWBIT_SOFTPLUS) ? 8
                                : (a == FEWBIT_TANH ? 16 : 0);
        const size_t min_waves3 = a == FEWBIT_GELU ? 16 : ((a == FEWBIT_SILU || a == FEWBIT_SIGMOID) ? 24 : 0);
        use_lut = (table->bits == 4 && min_waves4 != 0 && waves >= min_waves4) || (table->bits == 3 && min_waves3 != 0 && waves >= min_waves3);
    }
    bool forced_table = false;
    if (const int force = option(FEWBIT_OPT_FWD_TABLE); force == 1) { use_lut = prm.runs.count != 0; forced_table = true; }
    else if (force == 2) use_lut = false;
    // The table variants distribute their warp-blocks dynamically when a set of work counters can
    // be leased (not during stream capture); the 16-bit types at 3 bits only beat the packed search
    // that way.  binary32 ReLU / leaky ReLU measured faster with short CTAs and a static partition,
    // and below two waves there is nothing to balance.
    const FwdLaunchers &all = fwd_launchers(table->act);
    auto launcher = [&](bool lut) {
        return bias != nullptr ? all.with_bias[table->bits - 1][static_cast<int>(dtype)][lut]
                               : all.fn[table->bits - 1][static_cast<int>(dtype)][lut][table->folded ? 1 : 0];
    };
    if (launcher(use_lut) == nullptr || launcher(false) == nullptr) return FEWBIT_ERR_UNSUPPORTED;   // before any lease is taken
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    QueueLease lease;
    if (use_lut && (bf16 || (act_weight(table->act) >= 1 && waves >= 2)) && option(FEWBIT_OPT_FWD_QUEUE) == 0) {
        const cudaError_t qerr = queue_acquire(st, &lease);
        if (qerr != cudaSuccess) { t_last_cuda_error = static_cast<int>(qerr); return FEWBIT_ERR_CUDA; }
        prm.queue = lease.counters;
    }
    if (use_lut && bf16 && table->bits == 3 && prm.queue == nullptr && !forced_table) use_lut = false;
    const cudaError_t err = launcher(use_lut)(prm, x, y, packed, n, st);
    const cudaError_t rerr = queue_release(lease, st);
    if (err != cudaSuccess || rerr != cudaSuccess) {
        t_last_cuda_error = static_cast<int>(err != cudaSuccess ? err : rerr);
        return FEWBIT_ERR_CUDA;
    }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FEWBIT_OK;
}

}  // namespace
}  // namespace fewbit

extern "C" {

fewbit_status fewbit_fwd(const fewbit_table *table, const void *x, void *y, uint32_t *packed, size_t n,
                         fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (x == nullptr || y == nullptr || packed == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(y, 16) || !aligned(packed, 4)) return FEWBIT_ERR_ALIGNMENT;
    return forward(table, x, nullptr, 0, y, packed, n, dtype, stream);
}

fewbit_status fewbit_fwd_bias(const fewbit_table *table, const void *x, const void *bias, void *y, uint32_t *packed,
                              size_t rows, size_t cols, fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return FEWBIT_OK;
    if (x == nullptr || bias == nullptr || y == nullptr || packed == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (cols % kLaneElems != 0 || cols > 0xffffffffull || table->folded) return FEWBIT_ERR_UNSUPPORTED;
    if (rows > SIZE_MAX / cols) return FEWBIT_ERR_INVALID_ARG;
    if (!aligned(x, 16) || !aligned(bias, 16) || !aligned(y, 16) || !aligned(packed, 4)) return FEWBIT_ERR_ALIGNMENT;
    return forward(table, x, bias, static_cast<uint32_t>(cols), y, packed, rows * cols, dtype, stream);
}

fewbit_status fewbit_bwd(const fewbit_table *table, const uint32_t *packed, const void *grad_out, void *grad_in,
                         size_t n, fewbit_dtype dtype, void *stream) {
    using namespace fewbit;
    if (table == nullptr || !valid_dtype(dtype)) return FEWBIT_ERR_INVALID_ARG;
    if (n == 0) return FEWBIT_OK;
    if (packed == nullptr || grad_out == nullptr || grad_in == nullptr) return FEWBIT_ERR_INVALID_ARG;
    if (!aligned(grad_out, 16) || !aligned(grad_in, 16) || !aligned(packed, 4)) return FEWBIT_ERR_ALIGNMENT;
    Levels tl;
    for (int m = 0; m < kMaxLevels; ++m) tl.lev[m] = table->lev[m];
    const cudaError_t err = kBwd[table->bits - 1][static_cast<int>(dtype)](
        tl, packed, grad_out, grad_in, n, access_flags(grad_out, grad_in, nullptr, packed, table->bits), static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return FEWBIT_OK;
}

fewbit_status fewbit_set_option(fewbit_option opt, int value) {
    using namespace fewbit;
    bool ok = false;
    switch (opt) {
    case FEWBIT_OPT_FWD_TABLE: ok = value >= 0 && value <= 2; break;
    case FEWBIT_OPT_FWD_QUEUE: ok = value == 0 || value == 1; break;
    case FEWBIT_OPT_FWD_ITERS: ok = value >= 0 && value <= 64; break;
    case FEWBIT_OPT_FWD_WARPS: ok = value >= 0 && value <= 16; break;
    case FEWBIT_OPT_PDL: ok = value == 0 || value == 1; break;
    case FEWBIT_OPT_COUNT_TAILS: ok = value == 0 || value == 1; break;
    case FEWBIT_OPT_FWD_TILE: ok = value >= 0 && value <= 2; break;
    default: break;
    }
    if (!ok) return FEWBIT_ERR_INVALID_ARG;
    g_option[opt].store(value, std::memory_order_relaxed);
    return FEWBIT_OK;
}

int fewbit_get_option(fewbit_option opt) {
    return (static_cast<int>(opt) >= 0 && static_cast<int>(opt) < fewbit::kNumOptions) ? fewbit::option(opt) : -1;
}

fewbit_status fewbit_tail_warp_count(uint64_t *count, int reset) {
    using namespace fewbit;
    if (count == nullptr) return FEWBIT_ERR_INVALID_ARG;
    const cudaError_t err = tail_counter_read(count, reset != 0);
    if (err != cudaSuccess) { t_last_cuda_error = static_cast<int>(err); return FEWBIT_ERR_CUDA; }
    return FEWBIT_OK;
}

int fewbit_last_cuda_error(void) { return fewbit::t_last_cuda_error; }

uint64_t fewbit_launch_count(void) { return fewbit::g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
