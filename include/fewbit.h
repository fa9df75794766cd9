/*
 * fewbit.h -- C ABI of the Few-Bit Backward hot path for NVIDIA B200 (sm_100a).
 *
 * The method (arXiv 2202.00441): a pointwise activation f keeps, for its
 * backward pass, not the input x but only the index of the interval of a
 * piecewise-constant approximation q of f' that x falls into (Eq. 2), i.e.
 * `bits` = log2(K) bits per element.  Backward multiplies grad_out by the
 * level of that interval instead of f'(x) (Listing 1).  The intervals and
 * levels minimise the L2 error of Eq. 3 and are found once, offline, by the
 * dynamic programme of Eq. 7-9.
 *
 * Conventions that hold for every call
 *   - plain C types only; every pointer is commented HOST or DEVICE;
 *   - the library never throws, never calls exit(), never synchronises the
 *     device in the DEVICE-pointer calls and never allocates device memory;
 *     the only allocation is the host-side table object;
 *   - the caller owns every buffer; a table is immutable after creation and
 *     may be used from many threads and streams at once;
 *   - every function that can fail returns a fewbit_status.
 *
 * Table layout: K = 2^bits levels lev[0..K-1] and K-1 interior boundaries
 * s[0..K-2] (non-decreasing), both binary32.  The code of x is
 *     code(x) = #{ j : s[j] < x }        (strict, compared in binary32)
 * so interval i is (s[i-1], s[i]], anything below s[0] has code 0, anything
 * above s[K-2] has code K-1, and NaN has code 0.
 *
 * Saved-tensor layout ("packed"): one flat bit stream, element e occupies
 * bits [e*bits, e*bits + bits), least significant bit first, stored in
 * little-endian 32-bit words.  32 consecutive elements always fill exactly
 * `bits` words.  Unused high bits of the last word are written as zero.
 */
#ifndef FEWBIT_H_
#define FEWBIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(_WIN32)
#define FEWBIT_API
#else
#define FEWBIT_API __attribute__((visibility("default")))
#endif

typedef struct fewbit_table fewbit_table;

/* Activations f (Sec. 2; the rows of Table 1 plus ELU and LeakyReLU). */
typedef enum fewbit_act {
    FEWBIT_GELU = 0,       /* x * Phi(x), the erf form                       */
    FEWBIT_SILU = 1,       /* x * sigmoid(x)  (Swish)                        */
    FEWBIT_SIGMOID = 2,    /* 1 / (1 + exp(-x))                              */
    FEWBIT_TANH = 3,
    FEWBIT_ELU = 4,        /* x > 0 ? x : exp(x) - 1        (alpha = 1)      */
    FEWBIT_SOFTPLUS = 5,   /* log(1 + exp(x))               (beta = 1)       */
    FEWBIT_LEAKY_RELU = 6, /* x > 0 ? x : 0.01 x                             */
    FEWBIT_RELU = 7,       /* max(x, 0); exact with 1 bit (Sec. 2)           */
    FEWBIT_SELU = 8        /* 1.0507 (x > 0 ? x : 1.6733 (exp(x) - 1))       */
} fewbit_act;
#define FEWBIT_NUM_ACTS 9

typedef enum fewbit_dtype {
    FEWBIT_F32 = 0,        /* IEEE binary32                                  */
    FEWBIT_BF16 = 1,       /* bfloat16                                       */
    FEWBIT_F16 = 2         /* IEEE binary16                                  */
} fewbit_dtype;

typedef enum fewbit_status {
    FEWBIT_OK = 0,
    FEWBIT_ERR_INVALID_ARG = 1,   /* NULL pointer, bits outside 1..4, bad enum, unsorted table */
    FEWBIT_ERR_UNSUPPORTED = 2,   /* valid request this build cannot serve                      */
    FEWBIT_ERR_ALIGNMENT = 3,     /* a buffer breaks the alignment rule of the call             */
    FEWBIT_ERR_CUDA = 4,          /* a CUDA call failed; see fewbit_last_cuda_error()           */
    FEWBIT_ERR_ALLOC = 5,         /* host allocation failed / workspace too small               */
    FEWBIT_ERR_TOO_LARGE = 6      /* n exceeds the fixed capacity of an allocation-free call    */
} fewbit_status;

/* ------------------------------------------------------------------------- */
/* Tables (Eq. 2: parameters s and y; solved by Eq. 7-9, levels by Eq. 4)     */
/* ------------------------------------------------------------------------- */

/*
 * Optimal `bits`-bit table for `act`: the dynamic programme of Eq. 7 over a
 * uniform grid of 4096 cells on [-8, 8] with the uniform weight of Eq. 10
 * (A = -8, B = 8), prefix integrals as in Eq. 8-9, levels by Eq. 4.  Runs on
 * the CPU (a fraction of a second; results are cached per activation).
 * Returns a HOST handle, or NULL when act/bits are invalid or memory is
 * exhausted.  Release with fewbit_table_destroy().
 */
FEWBIT_API fewbit_table *fewbit_table_create(fewbit_act act, int bits);

/*
 * Same solver with explicit range [A, B] and number of grid cells
 * (2^bits <= n_cells <= 65536).  *out (HOST) receives the handle.
 */
FEWBIT_API fewbit_status fewbit_table_create_ex(fewbit_act act, int bits, double A, double B,
                                                int n_cells, fewbit_table **out);

/*
 * Table from caller-supplied parameters (Listing 1's globally stored s, y):
 * s = 2^bits - 1 boundaries, lev = 2^bits levels, both HOST binary32 arrays,
 * copied.  s must be non-decreasing and free of NaN, else
 * FEWBIT_ERR_INVALID_ARG.
 */
FEWBIT_API fewbit_status fewbit_table_from_arrays(fewbit_act act, int bits, const float *s,
                                                  const float *lev, fewbit_table **out);

/*
 * Folded table for an activation whose derivative is even (caption of Fig. 3:
 * for such an f only the non-negative half-axis needs intervals, which is
 * worth one more bit):
 * 2^bits pieces on [0, B], found by the same dynamic programme on a grid of
 * n_cells cells; the code of x is then #{ j : s[j] < |x| }.  Defined for
 * FEWBIT_SIGMOID and FEWBIT_TANH, otherwise FEWBIT_ERR_UNSUPPORTED.  The
 * objective reported by fewbit_table_get is the error over [-B, B] (twice the
 * half-axis value).  fewbit_fwd / fewbit_bwd take such a table like any other.
 * Suggested: B = 8, n_cells = 2048 (the grid step of the default tables).
 */
FEWBIT_API fewbit_status fewbit_table_create_folded(fewbit_act act, int bits, double B, int n_cells,
                                                    fewbit_table **out);

/*
 * The solver with every choice the paper leaves open (Sec. 3):
 *   A, B           support of the weight w of Eq. 3 (folded: A must be 0);
 *   n_cells        grid of the dynamic programme (Eq. 7);
 *   weight         FEWBIT_WEIGHT_UNIFORM: w = 1 on [A,B] (Eq. 10);
 *                  FEWBIT_WEIGHT_NORMAL: w = standard normal density on [A,B];
 *   finetune_iters 0: boundaries stay on the grid; > 0: at most that many
 *                  gradient steps on the boundaries by Eq. 5, started from the
 *                  DP result (boundaries then leave the grid; a few dozen
 *                  steps reach 2 f'(s_i) = y_i + y_{i-1} to ~1e-7);
 *   folded         as fewbit_table_create_folded.
 * The struct is read during the call only.
 */
#define FEWBIT_WEIGHT_UNIFORM 0
#define FEWBIT_WEIGHT_NORMAL 1
typedef struct fewbit_solver_options {
    double A, B;
    int n_cells;
    int weight;
    int finetune_iters;
    int folded;
} fewbit_solver_options;
FEWBIT_API fewbit_status fewbit_table_create_opt(fewbit_act act, int bits, const fewbit_solver_options *opt,
                                                 fewbit_table **out);

/* fewbit_table_from_arrays with the folded flag (folded != 0: s are boundaries of |x|). */
FEWBIT_API fewbit_status fewbit_table_from_arrays_ex(fewbit_act act, int bits, const float *s,
                                                     const float *lev, int folded, fewbit_table **out);

/* 1 if the table is folded, else 0 (also for NULL). */
FEWBIT_API int fewbit_table_is_folded(const fewbit_table *table);

/* Frees a table; NULL is accepted. */
FEWBIT_API void fewbit_table_destroy(fewbit_table *table);

/*
 * Reads a table back.  Any output pointer (all HOST) may be NULL.
 * s_out needs room for 2^bits - 1 floats, lev_out for 2^bits floats.
 * *objective is the value of Eq. 3 reached by the solver (NaN for a table
 * made by fewbit_table_from_arrays).
 */
FEWBIT_API fewbit_status fewbit_table_get(const fewbit_table *table, int *act, int *bits,
                                          float *s_out, float *lev_out, double *objective);

/* Bytes of the saved tensor for n elements: 4 * ceil(n * bits / 32); 0 if bits is invalid. */
FEWBIT_API size_t fewbit_packed_bytes(size_t n, int bits);

/* ------------------------------------------------------------------------- */
/* Hot path on DEVICE buffers (Listing 1)                                     */
/* ------------------------------------------------------------------------- */

/*
 * Forward half, one kernel launch on `stream` (a cudaStream_t passed as
 * void*; NULL = the legacy default stream), asynchronous:
 *     y[e]      = f(x[e])                 exact activation, rounded to dtype
 *     code[e]   = #{ j : s[j] < x[e] }    Eq. 2 / the sorted search of Listing 1
 *     packed    = the codes as a `bits`-bit stream (layout above)
 * x, y: DEVICE, n elements of `dtype`, 16-byte aligned; y == x (exact alias)
 * is allowed, any other overlap is undefined.  packed: DEVICE,
 * fewbit_packed_bytes(n, bits) bytes, 4-byte aligned; nothing beyond those
 * bytes is written.  n == 0 returns FEWBIT_OK without a launch.
 * (Alignment beyond the rule only widens the accesses: binary32 buffers that
 * are all 32-byte aligned move 256 bits per lane instead of 2 x 128, packed
 * words that are 8-byte (2 bits) or 16-byte (4 bits) aligned are stored as one
 * vector.  Any view of a tensor that starts on a multiple of 32 elements
 * therefore satisfies the rule for x, y and packed at once.)
 * Errors: FEWBIT_ERR_INVALID_ARG (NULL table or buffer, bad dtype),
 * FEWBIT_ERR_ALIGNMENT, FEWBIT_ERR_CUDA (launch failed).
 * The interval search has several equivalent kernel variants (binary search,
 * two-at-a-time bfloat16 search, shared-memory code table) chosen from the
 * activation, bits, dtype and n by measured thresholds; all give identical
 * codes.  The code-table variants (3-4 bits, from a few waves of resident warps
 * on, earlier the costlier f is) distribute their work through a set of
 * counters in a
 * file-scope device array (16 sets per device; nothing is allocated, but the
 * first such call on a device creates up to 16 CUDA events, and each call
 * records one after its kernel).  While `stream` is being captured,
 * or when all sets are in use by other streams, the kernel falls back to a
 * static partition: same results, ~10 % slower.  Small tensors (fewer 1024-
 * element blocks than resident warps) are processed a 256-element tile per
 * warp, which puts four times as many warps to work.  The choices can be overridden
 * for testing and tuning with fewbit_set_option (below); the library reads no
 * environment variable.
 * Both device kernels are launched with programmatic stream serialization:
 * their CTAs may be scheduled while the previous kernel of `stream` drains,
 * and wait there for its completion before they touch memory, so stream order
 * holds as usual (FEWBIT_OPT_PDL = 0 launches them the ordinary way).
 */
FEWBIT_API fewbit_status fewbit_fwd(const fewbit_table *table, const void *x, void *y,
                                    uint32_t *packed, size_t n, fewbit_dtype dtype, void *stream);

/*
 * Forward half with a bias in front of the activation (an extension; Listing 1
 * starts at the activation's input): for x of shape rows x cols, row-major,
 *   z[r][c] = x[r][c] + bias[c]     the exact sum, rounded once to `dtype`,
 *   y = f(z),  code = #{ j : s_j < z }   exactly as fewbit_fwd would on z.
 * The backward half needs nothing new: grad_in = fewbit_bwd(packed, grad_out)
 * is the gradient with respect to x, and its column sums are the gradient with
 * respect to the bias.
 *
 * x, y: DEVICE, rows * cols elements; bias: DEVICE, cols elements of `dtype`,
 * 16-byte aligned like x and y; packed: DEVICE, fewbit_packed_bytes(rows * cols,
 * bits) bytes, 4-byte aligned.  y may alias x exactly.  cols must be a multiple
 * of 8 below 2^32 (a lane's 8 consecutive elements then never straddle a row
 * end) and the table must not be a folded one, else FEWBIT_ERR_UNSUPPORTED;
 * rows * cols == 0 is a no-op.  Asynchronous on `stream`, allocates nothing; same kernel
 * variants and launch rules as fewbit_fwd.
 * Errors: INVALID_ARG (NULL, bad dtype, rows * cols overflows), UNSUPPORTED,
 * ALIGNMENT, CUDA.
 */
FEWBIT_API fewbit_status fewbit_fwd_bias(const fewbit_table *table, const void *x, const void *bias,
                                         void *y, uint32_t *packed, size_t rows, size_t cols,
                                         fewbit_dtype dtype, void *stream);

/*
 * Backward half, one kernel launch on `stream`, asynchronous:
 *     grad_in[e] = round_dtype( (float)grad_out[e] * lev[code[e]] )
 * (Eq. 1 with f' replaced by q of Eq. 2; one binary32 multiply, one rounding).
 * packed: DEVICE, as written by fewbit_fwd with a table of the same `bits`,
 * 4-byte aligned.  grad_out, grad_in: DEVICE, n elements of `dtype`,
 * 16-byte aligned; grad_in == grad_out allowed.  Errors as fewbit_fwd.
 */
FEWBIT_API fewbit_status fewbit_bwd(const fewbit_table *table, const uint32_t *packed,
                                    const void *grad_out, void *grad_in, size_t n,
                                    fewbit_dtype dtype, void *stream);

/* ------------------------------------------------------------------------- */
/* Hot path on HOST buffers                                                   */
/* ------------------------------------------------------------------------- */

/*
 * Device bytes fewbit_fwd_host / fewbit_bwd_host need in `workspace` to
 * stream `chunk_elems` elements per pipeline stage (rounded up to a multiple
 * of 1024 elements; the pipeline has 3 stages).
 */
FEWBIT_API size_t fewbit_host_workspace_bytes(size_t chunk_elems, fewbit_dtype dtype, int bits);

/*
 * Forward half on HOST buffers: x_host -> (y_host, packed_host), same
 * results as fewbit_fwd.  The tensor is cut into chunks; each chunk is copied
 * to `workspace` (DEVICE, caller-owned, 256-byte aligned, `workspace_bytes`
 * long), run through the forward kernel and copied back, with the copies of
 * neighbouring chunks overlapping the kernel on three internal streams (created
 * by the first call on a device and kept for later calls; concurrent calls get
 * triples of their own).  Blocks until the results are in host memory.  Page-locked host buffers are
 * needed for the copies to overlap; pageable ones work, slower.
 * FEWBIT_ERR_ALLOC if the workspace cannot hold one 1024-element chunk.
 * Calls on the same device that overlap in time must use disjoint workspaces.
 */
FEWBIT_API fewbit_status fewbit_fwd_host(const fewbit_table *table, const void *x_host,
                                         void *y_host, uint32_t *packed_host, size_t n,
                                         fewbit_dtype dtype, void *workspace,
                                         size_t workspace_bytes);

/* Backward half on HOST buffers: (packed_host, grad_out_host) -> grad_in_host; see fewbit_fwd_host. */
FEWBIT_API fewbit_status fewbit_bwd_host(const fewbit_table *table, const uint32_t *packed_host,
                                         const void *grad_out_host, void *grad_in_host, size_t n,
                                         fewbit_dtype dtype, void *workspace,
                                         size_t workspace_bytes);

/*
 * Forward half on HOST buffers WITHOUT any device allocation -- not even one
 * made by the caller.  (The paper has no counterpart: this is a packaging
 * variant of fewbit_fwd_host, same kernel, same results.)
 *
 * Who needs it: code that must not, or cannot, call cudaMalloc at the point
 * where it wants the forward pass -- a plug-in running inside a host
 * application whose memory pool already owns the whole device, a process held
 * to a fixed device-memory budget, or a latency-sensitive loop that cannot
 * afford the device-wide synchronisation an allocation may imply.  For them
 * the staging area that fewbit_fwd_host expects as `workspace` is a fixed
 * array inside the library image: FEWBIT_STATIC_MAX_ELEMS elements of room
 * (about 2.1 MiB of device memory), held by every GPU on which the library is
 * loaded until the process exits.
 *
 * x_host, y_host, packed_host: HOST buffers as in fewbit_fwd_host.  `stream`:
 * the copies and the kernel are enqueued on it and it is synchronised before
 * the call returns.  n > fewbit_static_max_elements() is rejected with
 * FEWBIT_ERR_TOO_LARGE (split the tensor on a multiple of 1024 elements and
 * call once per piece, or use fewbit_fwd_host).  The call makes no
 * cudaMalloc / cudaFree and, with the default options, creates no stream or
 * event (at this capacity the kernel variants that lease work counters are
 * never the size-based choice).
 *
 * The first call on each device looks up the device address of the array
 * (cudaGetSymbolAddress, with that device current); make that first call
 * outside of any stream capture.  Under CUDA's lazy module loading that same
 * first call is what loads the part of the library holding the array, i.e. it
 * is the moment the ~2.1 MiB are taken from the device: a caller whose pool
 * later claims all device memory should make one (small) call at start-up,
 * before the pool does, or run with CUDA_MODULE_LOADING=EAGER.  The address is
 * cached per device for the life of the process; it does not survive a
 * cudaDeviceReset.  All calls on a device share the one array:
 * it still holds the previous call's data (harmless -- every byte that is
 * read is written first, so nothing needs clearing), and two calls whose GPU
 * work overlaps in time, from different threads or streams, race on it.
 * Serialise them.
 */
#define FEWBIT_STATIC_MAX_ELEMS 262144
FEWBIT_API size_t fewbit_static_max_elements(void);
FEWBIT_API fewbit_status fewbit_fwd_host_static(const fewbit_table *table, const void *x_host,
                                                void *y_host, uint32_t *packed_host, size_t n,
                                                fewbit_dtype dtype, void *stream);

/* ------------------------------------------------------------------------- */
/* Options and diagnostics                                                    */
/* ------------------------------------------------------------------------- */

/*
 * Process-wide switches for testing and tuning (the paper has no counterpart;
 * every setting gives the same results, only the kernel variant or the launch
 * geometry changes).  Stored in atomics: may be set from any thread at any
 * time and apply to the launches that follow.
 *   FEWBIT_OPT_FWD_TABLE    0 size-based choice (default), 1 the shared-memory
 *                           code-table variant whenever the table has one,
 *                           2 never;
 *   FEWBIT_OPT_FWD_QUEUE    0 lease work counters when possible (default),
 *                           1 always the static partition;
 *   FEWBIT_OPT_FWD_ITERS    0 size-based (default), 1..64 warp-blocks per warp;
 *   FEWBIT_OPT_FWD_WARPS    0 default, 1..16 warps per CTA of the variants
 *                           without a code table (values beyond what the kernel
 *                           is compiled for are ignored);
 *   FEWBIT_OPT_PDL          1 programmatic dependent launch (default), 0 off;
 *   FEWBIT_OPT_COUNT_TAILS  1: every warp that runs the forward kernel's
 *                           ragged-tail path adds one to a device counter read
 *                           by fewbit_tail_warp_count (default 0: no counting);
 *   FEWBIT_OPT_FWD_TILE     0 by size (default): small tensors are processed a
 *                           256-element tile per warp instead of a 1024-element
 *                           block, 1 always (variants without a code table),
 *                           2 never.
 * fewbit_set_option returns FEWBIT_ERR_INVALID_ARG for an unknown option or a
 * value outside its range; fewbit_get_option returns -1 for an unknown option.
 */
typedef enum fewbit_option {
    FEWBIT_OPT_FWD_TABLE = 0,
    FEWBIT_OPT_FWD_QUEUE = 1,
    FEWBIT_OPT_FWD_ITERS = 2,
    FEWBIT_OPT_FWD_WARPS = 3,
    FEWBIT_OPT_PDL = 4,
    FEWBIT_OPT_COUNT_TAILS = 5,
    FEWBIT_OPT_FWD_TILE = 6
} fewbit_option;
FEWBIT_API fewbit_status fewbit_set_option(fewbit_option option, int value);
FEWBIT_API int fewbit_get_option(fewbit_option option);

/*
 * Diagnostic: *count (HOST) receives how many warps have run the ragged-tail
 * path of the forward kernel on the current device while FEWBIT_OPT_COUNT_TAILS
 * was 1 (exactly one per launch whose n is not a multiple of 1024 -- of 256 for
 * a launch in tile mode); reset != 0
 * clears the counter afterwards.  Synchronises the device.
 */
FEWBIT_API fewbit_status fewbit_tail_warp_count(uint64_t *count, int reset);

/* Static, never NULL. */
FEWBIT_API const char *fewbit_status_string(fewbit_status status);

/* The cudaError_t (as int) behind the calling thread's last FEWBIT_ERR_CUDA; 0 if none. */
FEWBIT_API int fewbit_last_cuda_error(void);

/* Kernels launched by this library in this process so far (all threads). */
FEWBIT_API uint64_t fewbit_launch_count(void);

/*
 * Accuracy scan of the binary32 evaluation of an activation (the arithmetic fewbit_fwd uses for
 * FEWBIT_F32) against the same function evaluated in binary64 and rounded once, for the `count`
 * input bit patterns first_pattern, first_pattern + 1, ... (first_pattern + count <= 2^32; the
 * whole range takes a few seconds).  Non-finite inputs are skipped.  The paper has no counterpart:
 * this is a self-check of the library's arithmetic (Sec. 2 only names the functions).
 *
 * result_device: DEVICE pointer to 5 uint64 words, 8-byte aligned, owned by the caller; the call
 * clears them on `stream`, then the kernel fills them:
 *   [0], [1], [2]  inputs whose result is 0, 1, 2 ulp from the rounded binary64 value;
 *   [3]            inputs further away (a NaN on one side only counts here);
 *   [4]            (largest distance, capped at 2^31 - 1) << 32 | an input pattern that has it.
 * Asynchronous on `stream`; read the words after synchronising.
 * Errors: INVALID_ARG (bad enum, NULL, range beyond 2^32), ALIGNMENT, CUDA.
 */
FEWBIT_API fewbit_status fewbit_f32_activation_scan(fewbit_act act, uint64_t first_pattern,
                                                    uint64_t count, uint64_t *result_device,
                                                    void *stream);

#ifdef __cplusplus
}
#endif
#endif /* FEWBIT_H_ */
