/* zipml.h -- C ABI of the B200 (sm_100a) library for double-sampled low-precision SGD on linear
 * models (ZipML, arxiv 1611.05402).
 *
 * Conventions
 *   - C linkage, plain pointers and sizes.  Every function returns an int status: ZIPML_OK (0) or
 *     a negative ZIPML_ERR_* value; zipml_strerror() names it.  No exceptions, no abort, no device
 *     trap.
 *   - Unless a parameter says HOST, data pointers are DEVICE pointers owned by the caller and must
 *     stay valid until the work is complete.  The library allocates only its own workspace, inside
 *     the context (it may grow on a call that needs more).
 *   - Work is enqueued on the context's CUDA stream and the call returns without waiting.
 *     Argument errors are reported by the call itself; errors found on the device (non-finite
 *     input, a grid barrier that ran out of patience) are reported by zipml_sync().
 *   - Matrices are row-major with 64-bit sizes and an explicit leading dimension in elements.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with
 *     ZIPML_ERR_CUDA.
 *
 * Packed sample layout ("plane"): row-major, `row_bytes` bytes per row, row_bytes a multiple of 16
 * and >= zipml_row_bytes(n, bits).  Feature j occupies cb bits at bit position j*cb of its row,
 * low bits first, where the container width cb is 2 for bits = 1, 2; 4 for bits = 3, 4; 8 for bits = 5 .. 8.  Padding bits
 * are zero.  A double-sampled dataset is two such planes (two independent quantizations of every
 * sample, Eq. (double) of the paper) plus what turns a code back into a value: per-feature
 * (lo_j, step_j) for a uniform grid, value = lo_j + code * step_j, or an n x 2^bits table of
 * ascending levels.
 */
#ifndef ZIPML_H_
#define ZIPML_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    ZIPML_OK = 0,
    ZIPML_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, bad stride or alignment        */
    ZIPML_ERR_UNSUPPORTED = -2, /* bits not in 1..8, a level table with more than 4 bits, ...   */
    ZIPML_ERR_NONFINITE = -3,   /* the sample matrix holds a NaN or an infinity (seen on device)   */
    ZIPML_ERR_CUDA = -4,        /* a CUDA runtime call failed (no device, out of memory, ...)       */
    ZIPML_ERR_TIMEOUT = -5,     /* a device-side wait gave up; the context stays usable            */
    ZIPML_ERR_WORKSPACE = -6    /* the problem does not fit the kernels' on-chip or scratch limits */
};

enum { ZIPML_LEVELS_UNIFORM = 0, ZIPML_LEVELS_TABLE = 1 };
/* How a plane lies in memory.  ROWS is the layout described above and the one every call produces and
 * accepts.  COLUMN_BLOCKS is a rearrangement for zipml_sgd_epoch's column engine (made and undone by
 * zipml_convert_layout, bit for bit): the plane is cut into blocks of 128 bytes of the row, block j
 * (bytes 128 j .. 128 j + 127 of every row, zero where the row has ended) stored as m consecutive
 * pieces of 128 bytes: piece (j, k) of row k at byte (j * m + k) * 128.  A plane then takes
 * zipml_column_blocks_bytes(m, row_bytes) bytes; row_bytes still names the row-major stride it came from. */
enum { ZIPML_LAYOUT_ROWS = 0, ZIPML_LAYOUT_COLUMN_BLOCKS = 1 };
enum { ZIPML_LOSS_DENSE = 0, ZIPML_LOSS_CODES = 1 };
/* Regulariser of zipml_sgd_epoch (paper Eq. (proxupdate): x <- prox_{lr R}(x - lr g), the proximal
 * operator taken coordinate by coordinate on y = x - lr g; and the Supplement's least-squares SVM,
 * whose gradient gains the term c x).  reg_param is c or lambda; constants are rounded to fp32 once
 * per call: shrink = 1 / (1 + lr c), thr = lr lambda, lr c. */
enum {
    ZIPML_REG_NONE = 0,     /* R = 0                                  x = y                          */
    ZIPML_REG_L2 = 1,       /* R = c/2 ||x||^2                        x = y * shrink                 */
    ZIPML_REG_L1 = 2,       /* R = lambda ||x||_1                     x = sign(y) max(|y| - thr, 0)  */
    ZIPML_REG_NONNEG = 3,   /* R = indicator of x >= 0                x = max(y, 0)                  */
    ZIPML_REG_LSSVM = 4     /* least-squares SVM term c x in the gradient:  x = y - (lr c) x_old     */
};
/* How zipml_sgd_epoch runs its minibatch chain.  Results do not depend on the choice. */
enum {
    ZIPML_ENGINE_AUTO = 0,      /* cluster, else lean, for steps of at most 2 MiB of codes; else column,
                                   else stream, where they apply (wide rows, uniform grid, fp32 model
                                   and gradient), else ring                                           */
    ZIPML_ENGINE_STEPWISE = 1,  /* a few kernel launches per minibatch                               */
    ZIPML_ENGINE_PERSISTENT = 2, /* one cooperative launch per call, grid barriers between the phases */
    ZIPML_ENGINE_RING = 3,       /* one cooperative launch; producer warp streams code chunks through a
                                    shared-memory ring, gradients meet by reduce-scatter / all-gather  */
    ZIPML_ENGINE_LEAN = 4,       /* one cooperative launch for small minibatch tiles: row parts only,
                                    two barriers and two packet exchanges per step                    */
    ZIPML_ENGINE_CLUSTER = 5,    /* one thread-block cluster (at most 16 row parts) for small tiles:
                                    gradients and model travel between the CTAs' shared memories.
                                    Uniform grids contract in fp32 or, on taller tiles, on the int8
                                    tensor cores; zipml_sgd_params.cluster_contraction overrides that
                                    choice                                                            */
    ZIPML_ENGINE_STREAM = 6,     /* one cooperative launch for large tiles on uniform grids with an fp32
                                    model and gradient: both passes of a step read the codes straight
                                    from global memory into int8 tensor-core fragments (the second pass
                                    from L2), a CTA owns whole column blocks of the gradient, one grid
                                    barrier per step.  ZIPML_ERR_WORKSPACE for level tables, quantized
                                    model or gradient, batches above 8192 rows.
                                    zipml_sgd_params.stream_prefetch overrides how many eighths of the
                                    next step's tile are requested into L2 ahead of time               */
    ZIPML_ENGINE_COLUMN = 7      /* one cooperative launch for large tiles on uniform grids with an fp32
                                    model and gradient, rows of 128 bytes .. 128 bytes x the number of
                                    SMs: a CTA owns a 128-byte column block of the packed rows for the
                                    whole launch; chunks of rows visit shared memory once for the dots
                                    and once more, out of L2, for the gradient, so the codes are read
                                    from HBM once per step; CTAs exchange only the rows' dots (integer
                                    atomics that count their own completion), there is no grid-wide
                                    barrier.  The only engine that takes ZIPML_LAYOUT_COLUMN_BLOCKS
                                    (where its copies are contiguous; AUTO picks it for such data).
                                    ZIPML_ERR_WORKSPACE for what it does not cover (as for STREAM)     */
};

typedef struct zipml_ctx zipml_ctx;

/* A double-sampled, bit-packed dataset in device memory. */
typedef struct zipml_dataset {
    uint32_t struct_size;   /* sizeof(zipml_dataset), for ABI evolution                              */
    int32_t bits;           /* 1 .. 8 (level tables: 1 .. 4)                                         */
    int32_t level_mode;     /* ZIPML_LEVELS_UNIFORM or ZIPML_LEVELS_TABLE                            */
    int32_t layout;         /* ZIPML_LAYOUT_ROWS, or ZIPML_LAYOUT_COLUMN_BLOCKS (zipml_sgd_epoch only)         */
    int64_t m, n;           /* samples, features                                                     */
    int64_t row_bytes;      /* stride of both planes                                                 */
    const uint8_t* plane1;  /* m * row_bytes bytes, 16-byte aligned                                  */
    const uint8_t* plane2;
    const float* feat_lo;   /* n; UNIFORM                                                            */
    const float* feat_step; /* n; UNIFORM                                                            */
    const float* levels;    /* n * 2^bits ascending; TABLE                                           */
} zipml_dataset;

/* The same double-sampled data in the shared-base storage of the paper's Section 2.2 ("Overhead of Storing
 * Samples"): the two quantizations of a value are the lower or the upper end of one interval of levels, so the
 * smaller code is stored once and each sample keeps one bit saying whether it lies one level higher --
 * bits + 2 instead of 2 * bits per value (container widths: 4 / 6 / 6 / 10 instead of 4 / 8 / 8 / 16).
 *   base      an ordinary plane (layout ZIPML_LAYOUT_ROWS, stride row_bytes) of the smaller codes
 *   up1, up2  one bit per feature: feature j at bit j of its row, low bits first, stride up_row_bytes
 *             (a multiple of 16, >= zipml_up_row_bytes(n)); code of sample c = base + up_c
 * Uniform grids only (value = lo_j + code * step_j). */
typedef struct zipml_shared_base {
    uint32_t struct_size;   /* sizeof(zipml_shared_base)                                             */
    int32_t bits;           /* 1 .. 8                                                                */
    int64_t m, n;
    int64_t row_bytes;      /* stride of the base plane                                              */
    int64_t up_row_bytes;   /* stride of the two up planes                                           */
    const uint8_t* base;    /* m * row_bytes bytes, 16-byte aligned                                  */
    const uint8_t* up1;     /* m * up_row_bytes bytes, 16-byte aligned                               */
    const uint8_t* up2;
    const float* feat_lo;   /* n (not needed by the conversions)                                     */
    const float* feat_step; /* n                                                                     */
} zipml_shared_base;

/* Parameters of one zipml_sgd_epoch call. */
enum { ZIPML_NORM_L2 = 0, ZIPML_NORM_LINF = 1 };

typedef struct zipml_sgd_params {
    uint32_t struct_size;       /* sizeof(zipml_sgd_params)                                          */
    int32_t model_bits;         /* 0: gradients see the fp32 model; 2..8: see Q3(x), redrawn per step */
    int32_t grad_bits;          /* 0: fp32 gradient; 2..8: the update uses Q4(g)                     */
    int32_t engine;             /* ZIPML_ENGINE_*                                                    */
    int64_t batch;              /* minibatch size B; batch t holds rows [t*B, min(m, (t+1)*B))       */
    int64_t epoch;              /* keys the Q3/Q4 random draws together with the step index          */
    int64_t first_step;         /* the call executes positions first_step .. first_step+num_steps-1  */
    int64_t num_steps;          /* of the batch order; num_steps < 0 means "to the end"              */
    uint64_t seed;              /* keys the Q3/Q4 random draws                                       */
    const int32_t* batch_order; /* HOST pointer or NULL: T = ceil(m/B) batch indices; NULL = 0..T-1  */
    float lr;                   /* step length gamma, constant within the call                       */
    int32_t grid_feature_parts; /* tuning, 0 = automatic: CTAs along the features                    */
    int32_t grid_row_parts;     /* tuning, 0 = automatic: CTAs along the rows of a minibatch (stream
                                   engine: an upper limit on its CTAs, ignored where too few)        */
    int32_t trace_steps;        /* profiling: number of steps to trace (0 = none)                    */
    uint64_t* trace;            /* profiling, DEVICE pointer or NULL: 8 uint64 per traced step; CTA 0
                                   stores its SM's cycle counter at the step's phase boundaries
                                   Ring engine: 0 step start, 1 residuals ready, 2 gradient parts
                                   published, 3 own sub-slice collected, 4 model updated, 5 model
                                   published, 6 all owners' packets seen, 7 step end.  Lean and
                                   cluster engines:
                                   0 step start, 1 tile arrived, 2 residuals ready, 3 gradient
                                   parts sent, 4 own features summed, 5 model published, 6 model
                                   collected, 7 step end.  The last step of a call stops after
                                   mark 4.  Stream engine: 0 step start, 1 own dots added, 2 barrier
                                   passed, 3 residual digits ready, 4 own gradient blocks summed,
                                   5 model updated and digits published, 6 dots and labels read,
                                   7 residual scale known.  Column engine (the buffer must be zeroed):
                                   0 clock at the step's first dots, 7 clock when the next w is out;
                                   cycles that warp 0 of a role spent waiting in the step: 1 A warp
                                   for first-visit copies, 2 R warp for complete dots (of its chunks),
                                   3 R warp for its digit buffer, 4 B warp for digits, 5 B warp for
                                   second-visit copies; 6 cycles of the step-end update.  Other engines
                                   ignore the request.                                               */
    int32_t reg;                /* ZIPML_REG_*                                                       */
    float reg_param;            /* c or lambda (>= 0); ignored by ZIPML_REG_NONE and _NONNEG          */
    float* model_out;           /* debug, DEVICE pointer or NULL: n floats, the model that the last
                                   executed step's gradient saw -- Q3(x) of that step when model_bits > 0
                                   (Supplement "Quantizing the Model"), else x as it stood before the step.
                                   ZIPML_ERR_WORKSPACE from the stream and column engines, which keep
                                   no such copy                                                      */
    int32_t cluster_contraction; /* tuning, cluster engine on uniform grids: 0 = automatic, 1 = fp32,
                                   2 = int8 tensor cores                                             */
    int32_t stream_prefetch;    /* tuning, stream engine: 0 = automatic, 1..9 = request (value - 1)
                                   eighths of the next step's tile into L2 ahead of time             */
    int32_t column_chunk_rows;  /* tuning, column engine: 0 = automatic, else rows of a minibatch that
                                   travel through shared memory together (a multiple of 32; values
                                   above 128 count as 128)                                            */
    int32_t vector_norm;        /* scale M(v) of Q3 and Q4 (Supplement Eq. (quant2) leaves it general):
                                   ZIPML_NORM_L2 = ||v||_2, the paper's choice and the default;
                                   ZIPML_NORM_LINF = max |v_i| (lower variance; the largest entry is exact).
                                   With LINF and model_bits or grad_bits set only the first-generation
                                   engine runs (AUTO picks it; the others answer ZIPML_ERR_UNSUPPORTED) */
} zipml_sgd_params;

/* Context: binds a device, a stream (a cudaStream_t passed as void*, NULL = the legacy default
 * stream) and a workspace.  One context must not be used from two threads at once. */
int zipml_create(zipml_ctx** ctx_out, int device, void* cuda_stream);
int zipml_destroy(zipml_ctx* ctx);
/* Waits for the stream and returns the first device-side error since the previous zipml_sync
 * (ZIPML_OK if none), clearing it. */
int zipml_sync(zipml_ctx* ctx);
const char* zipml_strerror(int status);
/* Diagnostics: how many of the library's kernels this context has launched since zipml_create. */
int64_t zipml_kernel_launches(const zipml_ctx* ctx);
/* Diagnostics: the ZIPML_ENGINE_* value that the context's latest zipml_sgd_epoch call ran (what
 * AUTO resolved to), or ZIPML_ENGINE_AUTO before the first call. */
int32_t zipml_last_engine(const zipml_ctx* ctx);
/* Diagnostics for the latency model of zipml_sgd_epoch: runs `iterations` steps of the per-step
 * communication skeleton on `ctas` co-resident CTAs (each publishes floats_per_cta floats through
 * L2, a bounded-spin grid barrier, each reads 16 bytes of every other CTA) and writes the elapsed
 * nanoseconds (device timer) to ns_out (one uint64, DEVICE pointer).  floats_per_cta % 4 == 0.
 * ZIPML_ERR_WORKSPACE if `ctas` CTAs cannot be resident at once. */
int zipml_barrier_latency(zipml_ctx* ctx, int32_t ctas, int32_t floats_per_cta, int32_t iterations, uint64_t* ns_out);
/* Diagnostics for the error path of the device-side waits: one thread polls a flag that nothing sets, with
 * the engines' bounded-wait pattern and a limit of spin_limit polls (1 .. 2^24), gives up and records
 * ZIPML_ERR_TIMEOUT, which the next zipml_sync returns (and clears); the context stays usable.  The paper
 * has no counterpart; it exists so that the time-out route can be exercised without a hung kernel. */
int zipml_wait_probe(zipml_ctx* ctx, int64_t spin_limit);
/* Smallest legal row stride for n features: ceil(n*cb/8) rounded up to 16; 0 if bits is unsupported. */
int64_t zipml_row_bytes(int64_t n, int32_t bits);
/* Bytes of one plane of m rows with row stride row_bytes in the ZIPML_LAYOUT_COLUMN_BLOCKS layout. */
int64_t zipml_column_blocks_bytes(int64_t m, int64_t row_bytes);

/* Rearranges both planes of `data` into the other layout (the packed layout is not fixed by the paper: the
 * Supplement's FPGA section only says that the pipeline consumes 64-byte lines; a column engine wants each
 * CTA's share of a minibatch contiguous in memory).  `data` is in the layout its `layout` field names; out1
 * and out2 (16-byte aligned, m * row_bytes bytes for ROWS, zipml_column_blocks_bytes for COLUMN_BLOCKS, not
 * overlapping the inputs) receive planes 1 and 2 in `to_layout`.  Converting there and back gives the
 * original bytes. */
int zipml_convert_layout(zipml_ctx* ctx, const zipml_dataset* data, int32_t to_layout, uint8_t* out1, uint8_t* out2);

/* Stochastic quantization with double sampling (paper Section 2.1, Eq. (double); Supplement
 * "Randomized Quantization", "Column Scaling").
 *   A          m x n fp32, leading dimension lda >= n.
 *   bits       1 .. 8: L = 2^bits levels, s = L-1 intervals (the paper's operating points are 5-6 bits and below;
 *              codes of 1, 3, 5, 6, 7 bits live in the next wider container).
 *   level_mode UNIFORM: levels lo_j + i*(hi_j-lo_j)/s on the feature's own range [lo_j, hi_j]
 *              (found by this call).  TABLE: `levels` (n x L ascending, levels[j][0] <= every value
 *              of feature j <= levels[j][L-1], e.g. from zipml_optimal_levels); more than 4 bits unsupported.
 *   seed       each element (row k, feature j) is rounded twice, to the lower or upper neighbouring
 *              level with the probabilities that make the expectation equal to the value, using
 *              two 24-bit uniforms from Philox4x32-10 keyed by (seed, k, j, copy).
 * Out: plane1, plane2 (m * row_bytes bytes each, fully written including zero padding),
 *      feat_lo (n; the per-feature minimum), feat_step (n; UNIFORM only, may be NULL for TABLE).
 * A NaN or infinity in A makes the next zipml_sync() return ZIPML_ERR_NONFINITE (outputs undefined). */
int zipml_quantize(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int32_t bits,
                   int32_t level_mode, const float* levels, uint64_t seed, uint8_t* plane1,
                   uint8_t* plane2, int64_t row_bytes, float* feat_lo, float* feat_step);

/* Variance-optimal level placement (paper Section 3: the problem statement, the recursion
 * T(k,m) = min_j T(k-1,j) + V(j,m), and "Dynamic Programming with Candidate Points").
 * Per feature: normalise to [0,1] by its range, count the values in `hist_bins` equal bins (one
 * pass over A), and choose the s-1 interior endpoints among the bin edges that minimise the total
 * quantization variance of the bin centres; exact integer arithmetic, ties to the smaller edge.
 *   bits 2, 3 or 4; s = 2^bits - 1 <= hist_bins <= 1024; m <= 10^9.
 * Out: levels_out n x 2^bits fp32 ascending with first = lo_j and last = hi_j;
 *      objective_out (n uint64, may be NULL): 4 * hist_bins^2 * (sum of variances), normalised units. */
int zipml_optimal_levels(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda,
                         int32_t bits, int32_t hist_bins, float* levels_out, uint64_t* objective_out);

/* Mini-batch SGD over the stored double samples (Supplement "Double Sampling", the averaged form of
 * its footnote; "End-to-end Quantization" for the optional model and gradient quantizers):
 *   g = 1/(2 B_t) sum_{k in batch} [ Q1(a_k)(Q2(a_k)^T x~ - b_k) + Q2(a_k)(Q1(a_k)^T x~ - b_k) ],
 *   x~ = Q3(x) or x,  g^ = Q4(g) or g,  x <- x - lr * g^   (update in fp32).
 * Q3 and Q4 are l2-scaled sign-magnitude stochastic quantizers with 2^(bits-1)-1 magnitude levels,
 * keyed by (seed, epoch, step position, coordinate).
 *   b        m labels;  x  n, read and updated in place.
 *   grad_out NULL or 2n floats: the last executed step's gradient before and after Q4.
 * ZIPML_ERR_WORKSPACE if n is too large for the kernels' shared memory plan. */
int zipml_sgd_epoch(zipml_ctx* ctx, const zipml_dataset* data, const float* b, float* x,
                    const zipml_sgd_params* params, float* grad_out);

/* Training loss (paper Eq. (leastsquares) with l = a^T x - b): 1/(2m) sum_k (a_k^T x - b_k)^2.
 *   ZIPML_LOSS_DENSE  on the fp32 samples A (m x n, lda); `data` ignored.
 *   ZIPML_LOSS_CODES  the unbiased estimate 1/(2m) sum (Q1(a_k)^T x - b_k)(Q2(a_k)^T x - b_k) from
 *                     `data`; A, m, n, lda ignored (sizes come from `data`).
 * Out: loss_out, one double in device memory.  Deterministic for a given device and shape. */
int zipml_loss(zipml_ctx* ctx, int32_t mode, const float* A, int64_t m, int64_t n, int64_t lda,
               const zipml_dataset* data, const float* b, const float* x, double* loss_out);

/* Shared-base storage (paper Section 2.2, "Overhead of Storing Samples"; see zipml_shared_base).
 * zipml_up_row_bytes: smallest legal stride of an up plane, ceil(n / 8) rounded up to 16.
 * zipml_shared_base_encode: the two planes of `data` (ZIPML_LAYOUT_ROWS) -> out->base, out->up1, out->up2 (the
 *   caller's buffers behind the const pointers of `out`, fully written; bits, m, n, row_bytes as in `data`).
 *   A value whose two codes lie more than one level apart makes the next zipml_sync() return
 *   ZIPML_ERR_INVALID_ARG (such planes are not two samples of the same values).
 * zipml_shared_base_decode: back to two planes of stride data->row_bytes, bit for bit.
 * zipml_loss_shared_base: the estimate of zipml_loss(ZIPML_LOSS_CODES) computed from the three planes as they lie,
 *   Q_c(a)^T x = lo^T x + base^T w + up_c^T w with w = step * x (fp32 products in short runs, combined in double).
 * zipml_sgd_epoch_shared_base: zipml_sgd_epoch on such data.  The epoch engines read two planes: they are rebuilt in
 *   the context's staging buffer first (shared with zipml_train_host, kept until the next such call), so the saving
 *   is in what is stored, not in what an epoch reads. */
int64_t zipml_up_row_bytes(int64_t n);
int zipml_shared_base_encode(zipml_ctx* ctx, const zipml_dataset* data, const zipml_shared_base* out);
int zipml_shared_base_decode(zipml_ctx* ctx, const zipml_shared_base* data, uint8_t* plane1, uint8_t* plane2);
int zipml_loss_shared_base(zipml_ctx* ctx, const zipml_shared_base* data, const float* b, const float* x, double* loss_out);
int zipml_sgd_epoch_shared_base(zipml_ctx* ctx, const zipml_shared_base* data, const float* b, float* x,
                                const zipml_sgd_params* params, float* grad_out);

/* Polynomials of a^T x over several independent quantizations (paper Section 4.1 "Quantizing Polynomials"; Section 4.2
 * uses them for smooth classification losses).  ZIPML_POLY_MAX_DEGREE bounds the degree d.
 * zipml_quantize_draw: zipml_quantize with a draw index and a choice of grid.  Draw q gives the quantizations Q_{2q+1},
 *   Q_{2q+2} of the same samples on the same grid, independent of every other draw (the Philox counter's last word is
 *   q; draw 0 with ZIPML_GRID_RANGE is zipml_quantize itself); d quantizations take ceil(d / 2) calls with the same
 *   seed.  grid: ZIPML_GRID_RANGE, the feature's own range [min_j, max_j]; ZIPML_GRID_SYMMETRIC (uniform levels
 *   only), the paper's [-M_j, M_j] with M_j = max |value| of the feature (Supplement "Column Scaling"): feat_lo is
 *   then -M_j and feat_step 2 M_j / s.
 * zipml_poly_rows: rows_out[k] (m doubles, device memory) = Q(P)_k = sum_{i=0..d} coef[i] * prod_{j<=i} Q_j(a_k)^T x,
 *   times scale[k] where scale (m floats, device memory, e.g. the labels) is not NULL.  `grid` gives bits, level mode,
 *   m, n, row_bytes and feat_lo / feat_step / levels (its plane pointers are checked like any data set's but not
 *   read); planes is a HOST array of d
 *   device pointers (16-byte aligned, stride grid->row_bytes, ZIPML_LAYOUT_ROWS), coef a HOST array of d + 1 doubles.
 *   Dots as in zipml_loss's code path (fp32 products in short runs, combined in double); product and sum in double.
 * zipml_weighted_plane_mean: g_out (n floats, device memory) = (1/m) sum_k c[k] * Q(a_k) for the plane Q and the m
 *   doubles c (device memory): with c = b_k Q(P)_k and Q = Q_{d+1} the gradient of Section 4.2's protocol.  Sums
 *   in double in a fixed order.
 * Errors: ZIPML_ERR_INVALID_ARG (null or misaligned pointers, degree out of range, a bad `grid`), ZIPML_ERR_UNSUPPORTED
 * (layout other than ZIPML_LAYOUT_ROWS); nothing is launched then. */
#define ZIPML_POLY_MAX_DEGREE 8
enum { ZIPML_GRID_RANGE = 0, ZIPML_GRID_SYMMETRIC = 1 };
int zipml_quantize_draw(zipml_ctx* ctx, const float* A, int64_t m, int64_t n, int64_t lda, int32_t bits,
                        int32_t level_mode, const float* levels, uint64_t seed, uint32_t draw, int32_t grid, uint8_t* plane1,
                        uint8_t* plane2, int64_t row_bytes, float* feat_lo, float* feat_step);
int zipml_poly_rows(zipml_ctx* ctx, const zipml_dataset* grid, const uint8_t* const* planes, int32_t degree,
                    const double* coef, const float* x, const float* scale, double* rows_out);
int zipml_weighted_plane_mean(zipml_ctx* ctx, const zipml_dataset* grid, const uint8_t* plane, const double* c, float* g_out);

/* The end of a step on its own: x <- R(x - lr * Q4(g)) for a gradient g (n floats, device memory) that the caller has
 * formed, e.g. the sum of several devices' shares of a minibatch (paper "End-to-end Quantization" for Q4, the
 * l2-scaled sign-magnitude quantizer of the Supplement; Eq. (proxupdate) and the LS-SVM term for R).  Read from
 * `params`: lr, grad_bits (0: g as it is), seed and epoch (with `step`, the step's position in the batch order, they
 * key Q4's draws exactly as zipml_sgd_epoch does, so a gradient equal to the one that call forms gives the same
 * update), reg, reg_param.  x (n floats, device memory) is updated in place; applied_out (DEVICE pointer or NULL)
 * receives the n floats of Q4(g).  The pre-Q4 gradient of one step comes from zipml_sgd_epoch with num_steps = 1,
 * lr = 0, grad_bits = 0, reg = ZIPML_REG_NONE and grad_out set (its first n floats; x is left as it was).
 * Errors: ZIPML_ERR_INVALID_ARG / ZIPML_ERR_UNSUPPORTED as for zipml_sgd_epoch; nothing is launched then. */
int zipml_sgd_apply_gradient(zipml_ctx* ctx, float* x, const float* g, int64_t n, const zipml_sgd_params* params,
                             int64_t step, float* applied_out);

/* Whole path from HOST buffers, for callers that hold their data in host memory: copies A and b to
 * the device, quantizes (UNIFORM, or TABLE with levels from zipml_optimal_levels when
 * optimal_levels != 0), runs `epochs` epochs of zipml_sgd_epoch (epoch index e = 0..epochs-1, step
 * length lr, or lr/(e+1) when lr_decay != 0: the paper's alpha/epoch schedule), evaluates the dense
 * loss, copies x and the loss back and waits.  Everything in `params` except epoch, first_step and
 * num_steps is honoured.
 *   A_host m x n fp32 (lda), b_host m, x_host n in/out, loss_out_host one double: all HOST. */
int zipml_train_host(zipml_ctx* ctx, const float* A_host, int64_t m, int64_t n, int64_t lda,
                     const float* b_host, float* x_host, int32_t bits, int32_t optimal_levels,
                     int32_t hist_bins, uint64_t quantize_seed, const zipml_sgd_params* params,
                     int32_t epochs, int32_t lr_decay, double* loss_out_host);

/* The code-plane loss of zipml_loss (ZIPML_LOSS_CODES) for callers that may not allocate device
 * memory.  (The paper has no counterpart: this is a packaging variant of the same computation.)
 * Who needs it: code that runs where cudaMalloc is forbidden or harmful -- between the kernels of a
 * latency-critical loop (an allocation may synchronise the whole device), under a framework whose
 * memory pool already owns the GPU's memory, or on a system with a fixed memory budget.  Such a
 * caller cannot create a zipml_ctx either, so this call takes the device and the stream directly.
 *   - Its scratch (the table step*x or level*x and one partial sum per block) is a fixed array
 *     inside the library image, about 1 MiB, which every GPU that loads the library holds until the
 *     process exits.  Limit: n <= 262144 features for a uniform grid, 2^bits * n <= 262144 with a
 *     level table; larger problems are refused with ZIPML_ERR_WORKSPACE.  The dataset is checked as
 *     by every other call (planes 16-byte aligned, stride a multiple of 16).
 *   - It calls no cudaMalloc/cudaFree and no allocating library routine.  The first call on a
 *     device looks up the array's device address (once per device); make that first call outside
 *     any stream capture.
 *   - All calls on one device share the array and the array keeps the previous call's contents.
 *     Every slot a call reads it has written itself, so nothing needs clearing, but two calls that
 *     overlap on the GPU (different streams, or two host threads) race on it: serialise them.
 *   device       ordinal of the GPU that holds the data
 *   cuda_stream  cudaStream_t as void* (NULL: the legacy default stream); the work is enqueued there
 *   data, b, x   as for zipml_loss; DEVICE pointers.   loss_out  one double, DEVICE pointer.
 * Returns like the other calls.  It is the same estimator as zipml_loss(CODES) in other arithmetic: fp32
 * products summed in short runs and combined in double here, where zipml_loss on a uniform grid
 * rounds step*x once to fixed point and sums integers; the two agree to about 1e-6 relative.  The
 * one-time address lookup is guarded by a lock, so two host threads may make a device's first call
 * together (their kernels still must not overlap, see above). */
int zipml_loss_codes_static(int device, void* cuda_stream, const zipml_dataset* data, const float* b,
                            const float* x, double* loss_out);

#ifdef __cplusplus
}
#endif
#endif /* ZIPML_H_ */
