/*
 * lapsum.h - C ABI of the B200 (sm_100a) LapSum exact-budget soft top-k solver.
 *
 * Operator (paper Eq. 1-3): for scores r (rows x n, fp32, row-major), budget k
 * and temperature alpha < 0 (t = |alpha|), each row gets the unique scalar
 * threshold b with  sum_i sigma((r_i - b)/t) = k,  sigma the Laplace CDF, and
 * the soft mask p_i = sigma((r_i - b)/t).  The backward (Eq. 5) is the
 * analytical vector-Jacobian product grad = f .* (v - sum(v f)/sum(f)),
 * f_i = exp(-|b - r_i|/t) / (2t).
 * alpha > 0 is accepted too and means Eq. 1 as printed with that sign:
 * p_i = sigma((b - r_i)/alpha), sum_i p_i = k, a mask that falls as the score
 * rises (the k smallest scores).  Its threshold is that of the alpha' = -alpha
 * problem with budget n - k (sigma(-u) = 1 - sigma(u)), which is what the
 * solver runs; p is the complement, grad_r changes sign, and the formulas
 * for grad_k and grad_alpha stay as they are.  Bracket statistics reported
 * by lapsum_status, lapsum_debug_bracket and lapsum_describe are then those
 * of that complementary problem.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless the comment says "host".
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *    stream).  lapsum_forward / lapsum_backward only enqueue work: they never
 *    synchronise the host and never allocate or free device memory.
 *  - The caller owns every buffer.  Inputs are const; outputs must not alias
 *    inputs.  One workspace serves one stream at a time.
 *  - Scores must be finite.  NaN/Inf give an unspecified result but never a
 *    hang: every device-side wait is bounded and reports through the status
 *    word (lapsum_status).
 *  - Return value: LAPSUM_OK (0) or a negative lapsum_error.  Argument errors
 *    are detected on the host before anything is enqueued.
 */
#ifndef LAPSUM_H
#define LAPSUM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lapsum_error {
    LAPSUM_OK = 0,
    LAPSUM_ERR_NULL = -1,        /* a required pointer is NULL                     */
    LAPSUM_ERR_SHAPE = -2,       /* rows < 1, n < 1 or n beyond LAPSUM_MAX_N       */
    LAPSUM_ERR_BUDGET = -3,      /* not 0 < k < n, or k not finite                 */
    LAPSUM_ERR_ALPHA = -4,       /* alpha zero or not finite, or |alpha| outside
                                    fp32's normal range [1.18e-38, 3e38]           */
    LAPSUM_ERR_WORKSPACE = -5,   /* workspace unknown, too small or built for other dims */
    LAPSUM_ERR_CUDA = -6,        /* a CUDA runtime call failed (see lapsum_last_cuda_error) */
    LAPSUM_ERR_PARAM = -7,       /* a field of lapsum_params is out of range       */
    LAPSUM_ERR_UNSUPPORTED = -8  /* entry point not available for this configuration */
} lapsum_error;

/* Largest row length accepted (tile look-back words carry 30-bit counts). */
#define LAPSUM_MAX_N (((int64_t)1 << 30) - 1)

/* Which pipeline computes the threshold (paper Sec. 1 and Table "Large-N
 * summary": the operator dispatches between the full sort and the bracket). */
typedef enum lapsum_path {
    LAPSUM_PATH_AUTO = 0,
    LAPSUM_PATH_BLOCK = 1,     /* one thread block per row, shared-memory bitonic sort     */
    LAPSUM_PATH_FULLSORT = 2,  /* global radix sort of the whole row, tile scan            */
    LAPSUM_PATH_BRACKET = 3    /* sampled bracket, one stream pass, sort of the middle band */
} lapsum_path;

/* Storage type of scores, upstream gradients, masks and gradients (lapsum_params.io_dtype).  The arithmetic is
 * fp32 (fp64 where sums are combined) whatever the storage type; thresholds b are always fp32. */
typedef enum lapsum_io_dtype {
    LAPSUM_IO_F32 = 0,
    LAPSUM_IO_F16 = 1,   /* IEEE binary16 */
    LAPSUM_IO_BF16 = 2   /* bfloat16 */
} lapsum_io_dtype;

typedef struct lapsum_params {
    double z;               /* bracket half-width in binomial standard deviations (Eq. 8); default 5.16 */
    int64_t bracket_min_n;  /* AUTO uses the bracket path for n >= this; default 16,385 = every row longer than
                               the block path (measured on B200: a forward of 16,385 ... 262,144 scores takes
                               35-50 us on the bracket path and 69-79 us on the full sort).  A single row
                               (rows = 1) takes it from bracket_min_n / 2 on: one thread block is slower than
                               the bracket path there, while a batch keeps the block path, which runs all rows
                               at once.  The bracket path itself accepts n >= 4096. */
    int64_t band_capacity;  /* middle-band buffer (elements); 0 = max(8192, ceil(8 z n / sqrt(K))), capped at n:
                               four times the widest band Eq. 8 predicts (budget k = n/2).  The bracket is taken
                               on the noised sample, so a temperature above the spread of the scores widens the
                               band in the scores by the ratio of the two densities at b; beyond the factor 4
                               the band overflows and the call pays the stream pass plus the full sort
                               (LAPSUM_ST_BAND_OVERFLOW, counted in lapsum_stats.fallbacks; results stay exact) */
    int32_t force_path;     /* lapsum_path; AUTO picks by n */
    int32_t sort_payload;   /* 1: sorts carry the original index as payload (needed by
                               lapsum_debug_sort_pairs on rows longer than the block path) */
    int32_t block_max_n;    /* AUTO uses the block path for n <= this; default and maximum 16384 */
    int32_t full_sorts;     /* bracket path: 0 (default) finds the two sample order statistics by radix
                               selection and sorts only the bucket of the band that holds the root;
                               1 sorts the whole sample and the whole band, as Alg. 1 words it.
                               Both give the same bracket and the same threshold. */
    int32_t max_widenings;  /* bracket path: how often a failed certificate may widen the bracket on the
                               failing side (App. C: a_L <- a_R, a_R <- a_R + 2(a_R - a_L), and its mirror)
                               and stream again before the full sort takes over; default 2, 0 = never.
                               Ignored (0) with full_sorts = 1. */
    int32_t io_dtype;       /* lapsum_io_dtype of r, v, p, grad_r; default LAPSUM_IO_F32.  The entry points with float
                               pointers serve fp32 workspaces only (LAPSUM_ERR_WORKSPACE otherwise); lapsum_forward_io /
                               lapsum_backward_io serve every type.  Half the bytes per score: 16 instead of 32 for a
                               forward + backward on the bracket path. */
} lapsum_params;

/* Status bits accumulated in the workspace by the kernels (lapsum_stats.status_bits). */
#define LAPSUM_ST_FALLBACK 0x1u          /* bracket certificate failed or band overflowed: full sort ran */
#define LAPSUM_ST_BAND_OVERFLOW 0x2u     /* |M| exceeded band_capacity                                   */
#define LAPSUM_ST_ROOT_LEFT 0x4u         /* Lap(a_L) < k : root was left of the bracket                  */
#define LAPSUM_ST_ROOT_RIGHT 0x8u        /* Lap(a_R) > k : root was right of the bracket                 */
#define LAPSUM_ST_LOOKBACK_TIMEOUT 0x10u /* a bounded look-back wait gave up: results invalid            */
#define LAPSUM_ST_NO_CROSSING 0x20u      /* no interval held the root (non-finite input)                 */
#define LAPSUM_ST_WIDENED 0x40u          /* a failed certificate was answered by widening the bracket    */
#define LAPSUM_ST_BAD_BUDGET 0x80u       /* a row's own budget (k_rows) was not in (0, n): that row is void      */
#define LAPSUM_ST_BOUNDS 0x200u          /* check build only (-DLAPSUM_CHECK_BOUNDS): a computed store index was beyond its
                                            limit; the access was skipped, the results are invalid                 */
#define LAPSUM_ST_BAD_ALPHA 0x100u       /* a row's own temperature (alpha_rows) was zero, not finite or outside
                                            fp32's normal range: that row is void                                */

typedef struct lapsum_stats {
    uint32_t status_bits;   /* OR of LAPSUM_ST_* since workspace_init                       */
    int32_t path;           /* lapsum_path taken by the last forward                          */
    int64_t forwards;       /* forward calls since workspace_init                             */
    int64_t fallbacks;      /* bracket attempts that fell back to the full sort               */
    int64_t widenings;      /* bracket widenings (each costs one more stream pass)            */
    int64_t lookback_timeouts;
    int64_t K, j, l;        /* last bracket: sample size and order-statistic ranks (Eq. 8)    */
    float a_L, a_R;         /* last bracket ends (-inf / +inf when open)                      */
    int64_t n_L, n_M, n_R;  /* last bracket: |L|, |M|, |R| (App. B)                            */
    double S_L, S_R;        /* last bracket: tail sums (Eq. 7)                                */
    double S_f, S_vf;       /* last backward: sum f and sum v f of the last row               */
} lapsum_stats;

/* Fill *prm (host) with the defaults listed above. */
void lapsum_default_params(lapsum_params *prm);

/*
 * Size of the scratch workspace for rows x n problems (host out).  prm may be
 * NULL (defaults).  Covers the worst case of the chosen path, including the
 * full-sort fallback of the bracket path (Alg. 1, "fall back").  A batch of rows
 * longer than the block path gets up to sixteen copies of the per-call buffers
 * (fewer when they would exceed 8 GB): the bracket path serves that many rows
 * with one launch per kernel, on the caller's stream; the full-sort path works
 * on the rows one by one, on up to three side streams of the caller's stream
 * that the library creates on first use and destroys in lapsum_workspace_release.
 */
int lapsum_workspace_bytes(int64_t rows, int64_t n, const lapsum_params *prm, size_t *bytes);

/*
 * What a workspace for rows x n problems would do, without a GPU (host only; prm may be NULL): the path the
 * dispatch picks (Sec. 4; Table "Large-N summary"), and for the bracket path the sample size
 * K (Alg. 1 line 1), the sampling stride floor(n / K) and the capacity of the middle-band buffer.
 * k may be 0 (then j and l are left 0); otherwise 0 < k < n and j, l are the two ranks of Eq. 8
 * (j < 1 or l > K mean that end of the bracket is open).
 */
typedef struct lapsum_plan {
    int32_t path;           /* lapsum_path */
    int32_t reserved;
    int64_t K, stride, band_capacity;
    int64_t j, l;
    size_t workspace_bytes;
} lapsum_plan;
int lapsum_describe(int64_t rows, int64_t n, double k, const lapsum_params *prm, lapsum_plan *out);

/*
 * Prepare a caller-allocated workspace (256-byte aligned, `bytes` as returned
 * above): zeroes the control region and look-back words, and uploads the
 * kernel-noise table of the systematic sampler (Sec. 4, App. D), e_s = unit-Laplace by inverse CDF of a hashed
 * counter, evaluated on the host in fp64 and rounded to fp32.  Registers the
 * workspace (host side) so that forward/backward know its layout.  The call
 * enqueues copies on `stream` and synchronises that stream before returning.
 */
int lapsum_workspace_init(void *ws, size_t bytes, int64_t rows, int64_t n, const lapsum_params *prm,
                          uint64_t seed, void *stream);

/* Forget a workspace registered by lapsum_workspace_init (does not free it). */
int lapsum_workspace_release(void *ws);

/*
 * Forward (Eq. 1-3; full-sort solver of App. A; bracketed solver of Sec. 4,
 * App. B and Alg. 1).  r: rows*n scores; p: rows*n mask out; b: rows
 * thresholds out.  k and alpha are shared by all rows; k may be fractional.
 */
int lapsum_forward(const float *r, int64_t rows, int64_t n, double k, double alpha, float *p, float *b,
                   void *ws, void *stream);

/*
 * Forward with one budget and / or one temperature per row (Eq. 1-3 per row; the paper's applications learn
 * both k and alpha, Sec. 6, and a batch may then carry different values for each sample).
 * k_rows, alpha_rows: rows DEVICE doubles each; either may be NULL, the call's scalar k or alpha then serves
 * every row (and is checked on the host as in lapsum_forward; the scalar that a vector replaces is ignored).
 * The vectors are read by the kernels, so nothing about them is checked on the host.  On the device every
 * row gets the checks lapsum_forward applies to its scalars: 0 < k < n, alpha finite, non-zero, |alpha| a
 * normal fp32 number.  A row that fails is void: b = NaN, a NaN mask, LAPSUM_ST_BAD_BUDGET and / or
 * LAPSUM_ST_BAD_ALPHA raised in the status word; the other rows are unaffected.  Rows may mix both signs of
 * alpha.  Served on every path (lapsum_describe tells which one a shape takes): short rows by the same
 * kernels with one parameter set per row; longer rows one after the other as in lapsum_forward, Eq. 8's
 * ranks being formed on the device from the row's own budget.  The parameter sets live in the workspace
 * (72 bytes per row).
 */
int lapsum_forward_rows(const float *r, int64_t rows, int64_t n, const double *k_rows, const double *alpha_rows, double k,
                        double alpha, float *p, float *b, void *ws, void *stream);

/*
 * Forward for any storage type (Eq. 1-3): r and p hold rows*n elements of the workspace's io_dtype (fp32, fp16
 * or bf16), b rows floats.  A 16-bit score is the fp32 of the same value to the solver: sort order, sample,
 * bracket ends, band counts and threshold are exactly those of lapsum_forward on the up-converted scores, and
 * the mask is that call's mask rounded to nearest even in the storage type.  k_rows, alpha_rows, k, alpha as in
 * lapsum_forward_rows (both vectors NULL: one budget and temperature for all rows).
 */
int lapsum_forward_io(const void *r, int64_t rows, int64_t n, const double *k_rows, const double *alpha_rows, double k,
                      double alpha, void *p, float *b, void *ws, void *stream);

/*
 * Backward for any storage type (Eq. 5): v, r and grad_r hold rows*n elements of the workspace's io_dtype, b rows
 * floats; alpha_rows, grad_k, grad_alpha as in lapsum_backward_rows.  The gradient is computed in fp32 and
 * rounded to nearest even on store; a magnitude beyond the storage type's range (fp16: 65504) becomes infinity.
 */
int lapsum_backward_io(const void *v, const void *r, const float *b, const double *alpha_rows, double alpha, void *grad_r,
                       float *grad_k, float *grad_alpha, void *ws, void *stream);

/* lapsum_forward_rows with a budget vector only (k_rows must not be NULL): kept for callers of the earlier name. */
int lapsum_forward_row_budgets(const float *r, int64_t rows, int64_t n, const double *k_rows, double alpha,
                               float *p, float *b, void *ws, void *stream);

/*
 * Backward (Eq. 5).  v: upstream gradient (rows*n); r: the forward's scores;
 * b: the forward's thresholds (rows); grad_r: rows*n out.  rows and n are
 * those the workspace was initialised with.  k is accepted for symmetry with
 * the forward and does not enter Eq. 5.  If sum f underflows to 0 the row's
 * gradient is 0.
 */
int lapsum_backward(const float *v, const float *r, const float *b, double k, double alpha, float *grad_r,
                    void *ws, void *stream);

/*
 * One forward + backward step from HOST buffers (Eq. 1-3 and Eq. 5; the paper has no counterpart: it is the
 * two calls above with the copies a caller with host data would otherwise issue one after the other).
 * r_host, v_host: rows*n floats each, read; p_host, grad_host: rows*n floats each, b_host: rows floats, written.
 * staging: DEVICE memory of at least (4*rows*n + rows) floats, owned by the caller, used as r, v, p, grad, b.
 * All work is enqueued; the results are complete when `stream` has finished.  The mask travels to the host on
 * a second stream while v still arrives on a third (a PCIe link carries both directions at once), so a step
 * costs three transfers' time instead of four.  The two side streams and five events are created on the first
 * call with this workspace and destroyed by lapsum_workspace_release.  Host buffers should be page-locked;
 * with pageable memory the copies still work but do not overlap.  Not for use inside a stream capture.
 * Errors as lapsum_forward / lapsum_backward; a failing CUDA call returns LAPSUM_ERR_CUDA.
 */
int lapsum_forward_backward_host(const float *r_host, const float *v_host, int64_t rows, int64_t n, double k,
                                 double alpha, float *p_host, float *grad_host, float *b_host, float *staging,
                                 void *ws, void *stream);

/*
 * Backward that also returns the gradients of the two scalars (the paper's applications learn k and
 * alpha, Sec. 6; it prints no formula - implicit differentiation of sum_i p_i = k gives, per row,
 *   grad_k     = sum(v f) / sum(f)
 *   grad_alpha = (1/t) [ sum v f (r - b) - (sum v f / sum f) sum f (r - b) ],   t = |alpha|,
 * both 0 when sum f underflows).  grad_k, grad_alpha: rows device floats each, either may be NULL.
 * Everything else as lapsum_backward; the extra sums ride on the same reduction pass.
 */
int lapsum_backward_scalars(const float *v, const float *r, const float *b, double k, double alpha, float *grad_r,
                            float *grad_k, float *grad_alpha, void *ws, void *stream);

/*
 * lapsum_backward_scalars for a forward that ran with one temperature per row (Eq. 5 per row; Sec. 6).
 * alpha_rows: rows DEVICE doubles, or NULL (then `alpha` serves every row and this is lapsum_backward_scalars).
 * A row whose temperature fails the device-side check of lapsum_forward_rows gets a NaN gradient and raises
 * LAPSUM_ST_BAD_ALPHA.  The budget does not enter Eq. 5, so budgets per row need nothing here.
 * grad_k, grad_alpha: rows device floats each, either may be NULL.
 */
int lapsum_backward_rows(const float *v, const float *r, const float *b, const double *alpha_rows, double alpha,
                         float *grad_r, float *grad_k, float *grad_alpha, void *ws, void *stream);

/*
 * Backward without a workspace and without any allocation (the paper has no counterpart: this entry
 * point exists for integration reasons only).
 *
 * Who needs it: hosts that may not allocate device memory once they are running - a serving process
 * whose memory budget is pinned at start-up, a plugin inside another engine that owns the allocator,
 * a real-time loop in which cudaMalloc's implicit device synchronisation is not acceptable - and that
 * cannot or do not want to carry a lapsum workspace around just to differentiate.
 *
 * It computes exactly what lapsum_backward computes for rows longer than the block path (the
 * two-kernel reduce + map form of Eq. 5), but its scratch - the per-block partial sums, the ticket of
 * the last-block reduction and the two row sums, LAPSUM_STATIC_SCRATCH_BYTES in all - lives in a
 * fixed array inside the library image instead of a caller workspace.  Every GPU that loads the
 * library holds that array until the process exits.
 *
 *  - v, r, grad_r: rows*n device floats; b: rows device floats; all as for lapsum_backward.
 *  - Limits: 1 <= rows <= LAPSUM_STATIC_MAX_ROWS, 1 <= n <= LAPSUM_MAX_N; anything larger returns
 *    LAPSUM_ERR_SHAPE and enqueues nothing.  The current device must have an index below 16
 *    (LAPSUM_ERR_UNSUPPORTED otherwise: the per-device table of scratch addresses has 16 entries).
 *  - The first call on each device looks up the device address of the array (the device must be
 *    current; a failure returns LAPSUM_ERR_CUDA).  Make that first call before any stream capture.
 *  - No cudaMalloc, cudaFree or other allocating call is made, on any call.
 *  - The array is shared by every call in the process and keeps the last call's contents; the entry
 *    point clears the ticket it needs at the start of each call.  Two calls whose kernels overlap on
 *    the GPU (different streams, no dependency) race on the array: serialise them.
 *  - Accuracy: it has only the fp32 b to work from, where lapsum_backward also reads the forward's
 *    (pivot, offset) pair from its workspace.  |r_i - b| / t therefore carries up to ulp(b) / (2 t):
 *    negligible while t >= 1e-2 |b|, a relative error of the gradient of up to ~4e-4 at t = 1e-3 |b|.
 */
#define LAPSUM_STATIC_MAX_ROWS 65536
#define LAPSUM_STATIC_SCRATCH_BYTES 98304
int lapsum_backward_static(const float *v, const float *r, const float *b, int64_t rows, int64_t n, double alpha,
                           float *grad_r, void *stream);

/*
 * One row sharded over several GPUs (Sec. 4, App. B, Alg. 1: every quantity the bracketed solver needs from the
 * row is a sum, a count or a short list, so contiguous shards of the row can be worked on where they live).
 * The library runs the per-shard pieces; the caller - one process per GPU - merges what they leave in the
 * workspace with three small collectives of its own (NCCL, or any other transport):
 *
 *   forward   lapsum_shard_sample     every rank draws the strata of the systematic sample that fall into its
 *                                     shard; the other strata stay 0 in its key buffer
 *             -> sum the K-word key buffers over the ranks (each word is written by exactly one rank)
 *             lapsum_shard_stream     order statistics a_L, a_R from the whole sample (the same on every rank),
 *                                     then the stream pass over the shard: its tails, counts, bucket tables, band
 *             -> sum tails (2 doubles), counts, bucket tables over the ranks; concatenate the bands
 *             lapsum_shard_solve      every rank solves the merged band: the same b everywhere, NaN if the
 *                                     certificate Lap(a_R) <= k <= Lap(a_L) failed (the caller then gathers the
 *                                     row on one GPU and calls lapsum_forward: the full sort is not sharded)
 *             lapsum_shard_mask       p of the shard
 *   backward  lapsum_shard_vjp_partial   the shard's four sums (Eq. 5 and the scalar gradients)
 *             -> sum the 4 doubles over the ranks
 *             lapsum_shard_vjp_apply     grad_r of the shard, grad_k / grad_alpha (the same on every rank)
 *
 * lapsum_shard_describe gives the byte offsets, from the start of the workspace, of the buffers the collectives
 * work on in place.  The workspace is that of ONE shard: lapsum_shard_workspace_bytes / _init size it from the
 * row's total length (sample, band) without the full-sort buffers of an ordinary workspace; it serves only the
 * lapsum_shard_* calls.  fp32 storage, one row, alpha of either sign; all ranks must use the same seed, params,
 * k and alpha.  Nothing here waits on another GPU: every call enqueues kernels on this GPU only.
 */
typedef struct lapsum_shard_layout {
    int64_t K;                 /* sample size (Alg. 1 line 1)                                              */
    int64_t band_capacity;     /* elements of the band buffer                                               */
    size_t off_sample_keys;    /* K uint32: the sample as order-preserving keys; SUM over ranks            */
    size_t off_band_count;     /* 1 uint64: |M| of the shard (may exceed band_capacity: overflow); SUM     */
    size_t off_n_R;            /* 1 uint64: |R| of the shard; SUM                                           */
    size_t off_tails;          /* 2 doubles: S_L, S_R (Eq. 7) of the shard; SUM                            */
    size_t off_bucket_counts;  /* 1024 uint32: scores per first-level bucket of the band; SUM              */
    size_t off_bucket_sums;    /* 2048 uint64: the buckets' two pivoted sums in fixed point; SUM           */
    size_t off_band_keys;      /* band_capacity uint32: the shard's band first (min(|M|, capacity) keys);
                                  the caller puts the concatenation of all shards' bands here               */
    size_t off_vjp_sums;       /* 4 doubles: sum f, sum v f, sum f (r-b), sum v f (r-b) of the shard; SUM  */
} lapsum_shard_layout;

int lapsum_shard_workspace_bytes(int64_t n_total, const lapsum_params *prm, size_t *bytes);
int lapsum_shard_workspace_init(void *ws, size_t bytes, int64_t n_total, const lapsum_params *prm, uint64_t seed, void *stream);
int lapsum_shard_describe(void *ws, lapsum_shard_layout *out);
/* r_shard: this rank's shard_len scores, scores [shard_begin, shard_begin + shard_len) of the row of n_total */
int lapsum_shard_sample(const float *r_shard, int64_t shard_begin, int64_t shard_len, int64_t n_total, double alpha, void *ws,
                        void *stream);
int lapsum_shard_stream(const float *r_shard, int64_t shard_len, int64_t n_total, double k, double alpha, void *ws, void *stream);
/* b: 1 device float out (the row's threshold, NaN on a failed certificate or a band that overflowed) */
int lapsum_shard_solve(int64_t n_total, double k, double alpha, float *b, void *ws, void *stream);
int lapsum_shard_mask(const float *r_shard, int64_t shard_len, int64_t n_total, double alpha, float *p_shard, void *ws,
                      void *stream);
int lapsum_shard_vjp_partial(const float *v_shard, const float *r_shard, int64_t shard_len, int64_t n_total, const float *b,
                             double alpha, void *ws, void *stream);
/* grad_k, grad_alpha: 1 device float each, nullable */
int lapsum_shard_vjp_apply(const float *v_shard, const float *r_shard, int64_t shard_len, int64_t n_total, const float *b,
                           double alpha, float *grad_shard, float *grad_k, float *grad_alpha, void *ws, void *stream);

/* Synchronise `stream`, then copy counters and the last bracket's figures to *out (host). */
int lapsum_status(void *ws, void *stream, lapsum_stats *out);

/*
 * Test hook for the sort step (App. A "after sorting"): every row ascending under the total order on
 * the fp32 bit patterns (-0.0 before +0.0), equal keys by ascending original index.
 * keys_out: rows*n floats.  idx_out: rows*n original indices, or NULL for the keys alone.
 * Which kernel runs:
 *  - block-path workspace, idx_out == NULL: the forward's own kernel for the shape, in the forward's
 *    own launch configuration (16 lanes per row up to 128 scores, else one thread block per row with
 *    the keys in registers, or a cluster of 4 / 8 blocks per row), stopped after its sort;
 *  - block-path workspace, idx_out != NULL: a separate kernel that sorts 64-bit (key, index)
 *    composites in shared memory; no forward runs it (the forward needs no payload);
 *  - longer rows: the radix sort of the forward's full-sort chain: keys only when the workspace was
 *    built with sort_payload = 0 (the default, and what lapsum_forward runs), with the index payload
 *    when built with sort_payload = 1.  idx_out != NULL needs sort_payload = 1
 *    (LAPSUM_ERR_UNSUPPORTED otherwise).
 */
int lapsum_debug_sort_pairs(const float *keys, int64_t rows, int64_t n, float *keys_out, uint32_t *idx_out,
                            void *ws, void *stream);

/*
 * Test hook for the bounded waits of the radix sort (the paper has no counterpart: its full-sort
 * branch, Sec. 4, is a library sort).  A tile of a radix pass waits for the digit counts of the tiles
 * before it; every such wait gives up after a fixed number of polls, raises
 * LAPSUM_ST_LOOKBACK_TIMEOUT, counts itself in lapsum_stats.lookback_timeouts and lets the kernel
 * finish (with an invalid order).  This hook makes that happen without faulting or hanging anything:
 * it runs the histogram and the FIRST radix pass of the forward's full-sort chain on `keys` (n floats,
 * one row) with the pass's ticket counter started at 1, so that tile 0 is never processed and its
 * counts never arrive, and with `spin_limit` polls (1 .. 65536, about a microsecond each) as the bound.
 * Only scratch buffers of the workspace are written.  For workspaces of one row on the full-sort or
 * bracket path with n > 8192 (LAPSUM_ERR_UNSUPPORTED otherwise).
 */
int lapsum_debug_lookback_timeout(const float *keys, int64_t n, int spin_limit, void *ws, void *stream);

/*
 * Test hook for the bracket (Alg. 1 lines 1-3 and 7, Eq. 7-8): runs sampling,
 * order statistics and the stream pass of the bracket path on one row and
 * leaves K, j, l, a_L, a_R, |L|, |M|, |R|, S_L, S_R in the workspace for
 * lapsum_status.  If use_override != 0 the given ends replace the sampled
 * ones (used to provoke the fallback from the host).  y_out (nullable, K
 * floats) receives the noised sample in draw order, band_out (nullable,
 * band_capacity floats) the gathered middle band in arbitrary order.
 */
int lapsum_debug_bracket(const float *r, int64_t n, double k, double alpha, void *ws, void *stream,
                         int use_override, float a_L, float a_R, float *y_out, float *band_out);

/*
 * Forward of one row through the bracket path with caller-chosen bracket ends
 * instead of sampled ones (host-side injection of a failed certificate; the
 * solver then takes its full-sort fallback, Alg. 1 line 5).
 */
int lapsum_forward_with_bracket(const float *r, int64_t n, double k, double alpha, float a_L, float a_R,
                                float *p, float *b, void *ws, void *stream);

/*
 * Per-kernel timing (the paper reports wall-clock means only; this is the
 * library's tracing aid).  After lapsum_profile_enable, every launch of a
 * kernel whose bit (1u << lapsum_kernel) is set in kernel_mask is bracketed by
 * a pair of CUDA events on the caller's stream, up to max_records launches.
 * lapsum_profile_read synchronises the stream and returns the number of
 * recorded launches of one kernel and their summed duration (host out).
 * Enabling allocates CUDA events (host objects, no device memory); events
 * cost about a microsecond each on the stream, so leave profiling off unless
 * a per-kernel figure is wanted.
 */
typedef enum lapsum_kernel {
    LAPSUM_K_BLOCK_FWD = 0,
    LAPSUM_K_BLOCK_BWD = 1,
    LAPSUM_K_HISTOGRAM = 2,
    LAPSUM_K_ONESWEEP = 3,
    LAPSUM_K_TILE_AGG = 4,
    LAPSUM_K_SOLVE = 5,
    LAPSUM_K_CDF_MAP = 6,
    LAPSUM_K_VJP_REDUCE = 7,
    LAPSUM_K_VJP_MAP = 8,
    LAPSUM_K_SAMPLE = 9,
    LAPSUM_K_STREAM_BAND = 10,
    LAPSUM_K_MISC = 11,
    LAPSUM_K_COUNT = 12
} lapsum_kernel;

int lapsum_profile_enable(void *ws, uint32_t kernel_mask, int max_records);
int lapsum_profile_read(void *ws, void *stream, int kernel_id, int64_t *launches, double *total_ms);
int lapsum_profile_disable(void *ws);
const char *lapsum_kernel_name(int kernel_id);

/* Number of kernel launches this library has enqueued since it was loaded. */
int64_t lapsum_launch_count(void);

/* Text for a lapsum_error; the last CUDA error code seen by this thread. */
const char *lapsum_error_string(int err);
int lapsum_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LAPSUM_H */
