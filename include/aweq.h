/*
 * aweq.h -- C ABI of the B200 (sm_100a) AWEQ calibration library.
 *
 * AWEQ (arXiv 2311.01305, "Post-Training Quantization with Activation-Weight
 * Equalization for Large Language Models") calibrates one linear layer
 * y = W x (+ bias) from N calibration inputs x_1..x_N in six steps:
 *   1. per-channel min / max / mean of the inputs            aweq_stats
 *   2. per-input-channel range of the weights                aweq_wrange
 *   3. equalisation factors s (Eq. 10) and diagnostics       aweq_factors
 *   4. fold s into W and quantise (Eq. 3, Eq. 1-2), pack     aweq_equalize_quantize
 *   5. statistical bias correction (Eq. 11-15)               aweq_bias_correct
 *   6. 8-bit quantisation of the equalised inputs (W8A8)     aweq_quant_act
 * aweq_layer_pass runs all six for one input and the matrices it feeds.
 * Around the pass: aweq_fold_scale folds diag(s)^-1 into the producer of an input
 * (Section 3.1); aweq_forward_check (W8A8) and aweq_forward_check_weights (weight-only)
 * measure what Eq. 11 names, E[y~ - y], for a calibrated layer on the tensor cores.
 *
 * General rules
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned
 *     by the caller.  The library allocates no device memory and keeps no
 *     per-call state; scratch memory is passed in as `ws` (size from
 *     aweq_workspace_bytes, 256-byte aligned, contents irrelevant on entry).
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) and the call returns without synchronising.
 *   - The return value is the result of host-side validation and of the
 *     launches.  When it is not AWEQ_OK nothing was enqueued (validation) or
 *     the CUDA error is reported (AWEQ_ERR_CUDA); no exception crosses the ABI.
 *   - Conditions found on the device are counted into *st (may be NULL); the
 *     caller zeroes it and reads it back after synchronising.
 *   - Matrices are row-major with the innermost dimension contiguous.
 *     X is [N x C_in] with row pitch ldx elements, W is [C_out x C_in] with
 *     row pitch ldw elements ("channel i" of the paper is always the input
 *     channel, a column of both).  16-bit elements are fp16 or bf16.
 *     Base pointers of X and W must be 16-byte aligned, ldx / ldw and C_in
 *     multiples of 8; a violation is an error code, never a fault.
 *   - Outputs are overwritten completely unless `accumulate` is set.
 *   - Floating-point decisions that produce integer codes are taken in IEEE
 *     binary32, round to nearest even, without fused multiply-add:
 *     v^ = fl(v * scale), Step = fl(fl(hi - lo) / (2^b - 1)),
 *     inv = fl(1 / Step), Z = -rint(fl(lo * inv)),
 *     q = clamp(rint(fl(v^ * inv)) + Z, 0, 2^b - 1).
 *     A constant vector (hi == lo) takes Step = |lo| (1 if lo == 0).
 */
#ifndef AWEQ_H
#define AWEQ_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    AWEQ_OK = 0,
    AWEQ_ERR_NULL = 1,        /* a required pointer is NULL */
    AWEQ_ERR_SHAPE = 2,       /* a size is <= 0, not a multiple of 8, or too large */
    AWEQ_ERR_ALIGN = 3,       /* a base pointer or pitch breaks the alignment rule */
    AWEQ_ERR_DTYPE = 4,
    AWEQ_ERR_BITS = 5,        /* bit-width outside 2..8 */
    AWEQ_ERR_GROUP = 6,       /* group size not a power of two in [8, 256] or not dividing C_in */
    AWEQ_ERR_WORKSPACE = 7,   /* ws is NULL, misaligned or smaller than aweq_workspace_bytes */
    AWEQ_ERR_CUDA = 8,        /* a CUDA call failed; see aweq_last_cuda_error */
    AWEQ_ERR_UNSUPPORTED = 9,
    AWEQ_ERR_LIMIT = 10       /* size beyond the built-in scratch of aweq_stats_static */
} aweq_status;

typedef enum { AWEQ_F16 = 0, AWEQ_BF16 = 1 } aweq_dtype;

/* Granularity of one (Step, Z) pair: the whole tensor; one row (an output
 * channel of W, a token of X); or a group of `group` consecutive input
 * channels inside one row of W. */
typedef enum { AWEQ_PER_TENSOR = 0, AWEQ_PER_ROW = 1, AWEQ_PER_GROUP = 2 } aweq_gran;

/* Device-side condition counters.  nonfinite: channels / vectors whose
 * statistics were Inf or NaN; zero_range: dead channels (factor forced to 1);
 * wait_timeout: a bounded wait inside a kernel gave up (results of that call
 * are invalid). */
typedef struct {
    unsigned long long nonfinite;
    unsigned long long zero_range;
    unsigned long long wait_timeout;
    unsigned long long reserved;
} aweq_dev_status;

typedef enum {
    AWEQ_OP_STATS = 1,
    AWEQ_OP_WRANGE = 2,
    AWEQ_OP_EQUALIZE_QUANTIZE = 4,
    AWEQ_OP_BIAS_CORRECT = 5,
    AWEQ_OP_QUANT_ACT = 6
} aweq_op;

/* Host helpers (no CUDA calls). */
const char *aweq_strerror(aweq_status code);
const char *aweq_last_cuda_error(void);          /* text of the last CUDA error seen by this thread */
int aweq_version(void);
/* Number of kernels this library has launched in this process (diagnostic). */
unsigned long long aweq_launch_count(void);
/* Launch geometry the library would use for an operation on a rows x cols matrix (host logic
 * only, no CUDA call; for diagnostics and tests).  op is AWEQ_OP_STATS / AWEQ_OP_WRANGE (the
 * column reduction), AWEQ_OP_EQUALIZE_QUANTIZE (row-wise weights) or AWEQ_OP_QUANT_ACT (per
 * token).  plan[8] receives
 *   column reduction: {CTAs, threads (256, 320 or 384 consumers and a producer warp), shared bytes
 *                      (128 + stages x rows per stage x slab width x 16: two to four stages),
 *                      column slabs, slab width in 16-byte vectors, row splits, row phases, rows per stage}
 *   row quantisers:   {CTAs, threads, shared bytes, threads per row, vectors per thread,
 *                      rows per stage, stages, kernel: 2 plain loads without stages (rows per stage
 *                      and stages are 0 then; step 4 at every width, step 6 up to 36864 columns),
 *                      3 shared-memory stages with every row shared by a cluster of two CTAs (step 6
 *                      beyond 36864 columns; threads per row = twice the threads of a CTA, shared
 *                      bytes for half-rows)}
 * Returns AWEQ_ERR_SHAPE when the shape is not supported, AWEQ_ERR_UNSUPPORTED for other ops. */
aweq_status aweq_plan_query(int op, long long rows, long long cols, long long plan[8]);

/* Scratch bytes an operation needs for the given shape: rows x cols is
 * N x C_in for AWEQ_OP_STATS / AWEQ_OP_QUANT_ACT and C_out x C_in for the
 * weight operations.  Returns 0 when the operation needs none. */
size_t aweq_workspace_bytes(int op, long long rows, long long cols, int bits, int gran, int group);

/*
 * Step 1 -- calibration statistics (Section 3.2: the range of channel i is its
 * maximum minus its minimum over all inputs; Section 3.3, last paragraph: E[x]
 * is gathered in the same sweep as the factors).
 *   xmin[j] = min_n X[n,j], xmax[j] = max_n X[n,j]  (exact)
 *   xmean[j] = (1/N) sum_n X[n,j]  (binary32 partial sums over at most 8 rows,
 *              folded into binary64; final division in binary64)
 * X: [N x C_in] 16-bit, read once.  xmin, xmax, xmean: float[C_in], written.
 * xsum: double[C_in], count: long long[1] -- optional running state; both
 * required when accumulate != 0, in which case xmin / xmax / xsum / count
 * hold the result of earlier chunks on entry and the merged result on exit
 * (calibration data can be streamed in chunks; also the hook for sharding
 * tokens over devices).  N == 0 is allowed (identity).
 * ws: aweq_workspace_bytes(AWEQ_OP_STATS, N, C_in, 0, 0, 0).
 */
aweq_status aweq_stats(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx,
                       float *xmin, float *xmax, float *xmean,
                       double *xsum, long long *count, int accumulate,
                       void *ws, size_t ws_bytes, aweq_dev_status *st, void *stream);

/*
 * Step 1 for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of aweq_stats, same kernels, same
 * results.)  Some callers have no way to provide `ws`: code running inside a
 * framework whose allocator they must not touch, plug-ins that are handed
 * tensors but no allocation service, or a latency-critical section where a
 * cudaMalloc (which synchronises the device) is not acceptable.  For them the
 * scratch is a fixed array inside the library image: about 4.6 MiB of device
 * memory on every GPU that loads the library, held until the process exits.
 * Limits: C_in <= 16384 (a multiple of 8); N >= 1; no running state (no
 * accumulate).  Anything larger returns AWEQ_ERR_LIMIT and enqueues nothing.
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  The call
 * allocates and frees nothing.  All calls on a device share the one array, and
 * it keeps what the last call left there: nothing in it has to be cleared,
 * because each call writes every partial it later reads, but two calls whose
 * kernels may overlap on the GPU (different streams, no ordering between them)
 * would overwrite each other's partials -- order such calls yourself.
 * Other arguments and results as for aweq_stats.
 */
aweq_status aweq_stats_static(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx,
                              float *xmin, float *xmax, float *xmean, aweq_dev_status *st, void *stream);

/*
 * Step 2 -- per-input-channel weight range (Section 3.2, same definition
 * applied to W): wmin[j] = min_o W[o,j], wmax[j] = max_o W[o,j].
 * accumulate != 0 merges with the values already in wmin / wmax, which gives
 * matrices that share one input (q/k/v, gate/up) a common range.
 * ws: aweq_workspace_bytes(AWEQ_OP_WRANGE, C_out, C_in, 0, 0, 0).
 */
aweq_status aweq_wrange(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ldw,
                        float *wmin, float *wmax, int accumulate,
                        void *ws, size_t ws_bytes, aweq_dev_status *st, void *stream);

/*
 * Step 3 -- equalisation factors (Eq. 10) and the quantities of Eq. 4-8.
 *   r^X_j = xmax_j - xmin_j, r^W_j = wmax_j - wmin_j
 *   s_j = (1/r^W_j) sqrt(r^X_j r^W_j)   (Eq. 10 evaluated in binary64 and rounded
 *                                       once to binary32; = sqrt(r^X_j / r^W_j))
 *   rinv_j = 1 / s_j, mu_hat_j = xmean_j * rinv_j  (E[x^] of the equalised input)
 *   a dead channel (range <= 0 or not finite) gets s_j = 1 and is counted in
 *   st->zero_range.
 * All arrays float[C_in]; s, rinv, mu_hat required, pX, pW optional
 * (p_j = r_j / R with R the tensor range, Eq. 4).
 * scalars: optional double[8] = { R^X, R^W, R^X^, R^W^ (tensor ranges after
 * equalisation), objective of Eq. 5 before and after, the max*max product of
 * Eq. 8 before (s = 1) and after }.  C_in <= 1048576.
 */
aweq_status aweq_factors(const float *xmin, const float *xmax, const float *xmean,
                         const float *wmin, const float *wmax, long long C_in,
                         float *s, float *rinv, float *mu_hat, float *pX, float *pW, double *scalars,
                         aweq_dev_status *st, void *stream);

/*
 * Step 3 with the criterion AWEQ argues against, for comparison.  Section 3.1 starts from the
 * per-channel equalisation that balances the LARGEST MAGNITUDES of activations and weights;
 * the paper's point is that balancing the channel RANGES (Eq. 4-10) does better.  This entry
 * feeds Eq. 10 with max|x_j| and max|w_j| instead of the ranges,
 *   s_j = (1 / max|w_j|) sqrt(max|x_j| max|w_j|)   ( = sqrt(max|x_j| / max|w_j|) ),
 * everything else (rinv, mu_hat, the range-based diagnostics, dead channels, rounding) as in
 * aweq_factors, so that the two criteria can be put through the same quantiser and forward check.
 */
aweq_status aweq_factors_absmax(const float *xmin, const float *xmax, const float *xmean,
                                const float *wmin, const float *wmax, long long C_in,
                                float *s, float *rinv, float *mu_hat, float *pX, float *pW, double *scalars,
                                aweq_dev_status *st, void *stream);

/*
 * Step 4 -- fold s into W and quantise (Eq. 3: W^ = diag(s) W, so input
 * channel j of every row is multiplied by s_j; Eq. 1-2 on every row or group).
 * One pass over W: rescale, range, quantise and pack are fused.
 * s: float[C_in] or NULL (no equalisation: the round-to-nearest baseline of
 * Section 4.2).  mu_hat: float[C_in] or NULL; when given with epsmu,
 *   epsmu[o] = sum_j (Step (q - Z) - W^[o,j]) mu_hat[j]     (eps . E[x^], Eq. 15)
 * is produced in the same pass (binary32 accumulation, fixed order).
 * bits in 2..8.  gran: AWEQ_PER_ROW (one pair per output channel),
 * AWEQ_PER_GROUP (group: power of two in [8, 256] dividing C_in) or
 * AWEQ_PER_TENSOR.  Per-row mode supports C_in <= 40960.
 * codes: unsigned char[C_out x C_in*bits/8], the little-endian bit stream of
 * each row: code i at bits [i*bits, (i+1)*bits) (8-bit: one per byte; 4-bit:
 * two per byte, low nibble first; 3-bit: eight codes per three bytes).
 * step: float, zp: int, one per row ([C_out]), per group ([C_out x C_in/group])
 * or a single pair.  epsmu: float[C_out] or NULL.
 * ws: aweq_workspace_bytes(AWEQ_OP_EQUALIZE_QUANTIZE, C_out, C_in, bits, gran, group).
 * Non-finite elements never fault.  An infinite element makes Step infinite and every code of
 * its row / group equal to the zero-point's clamp, as Eq. 1 evaluated literally gives.  A NaN
 * element is ignored by the extremes (Step, Z and every other code are as if it were absent);
 * the codes of the eight consecutive columns that share its 16-byte input vector are unspecified.
 * The same holds for step 6.
 */
aweq_status aweq_equalize_quantize(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ldw,
                                   const float *s, const float *mu_hat,
                                   int bits, aweq_gran gran, int group,
                                   unsigned char *codes, float *step, int *zp, float *epsmu,
                                   void *ws, size_t ws_bytes, aweq_dev_status *st, void *stream);

/*
 * Step 5 -- bias correction (Eq. 11-15 and the sentence after them: the
 * expected output error eps E[x] is subtracted from the output, which for a
 * linear layer is a change of its bias):
 *   bias_out[o] = bias_in[o] - sum_j eps[o,j] mu_hat[j],  eps = W~ - W^.
 * Two routes.  Fused: epsmu != NULL is the sum produced by step 4 and the
 * weight arguments are ignored.  Standalone: epsmu == NULL and the sum is
 * recomputed from W, s, the packed codes, step, zp and mu_hat.
 * bias_in: 16-bit [C_out] of type bias_dt, or NULL for a layer without bias
 * (the correction then creates one).  bias_out: 16-bit [C_out] (may be NULL);
 * bias_out_f32: float[C_out] (may be NULL); at least one must be given.
 */
aweq_status aweq_bias_correct(const float *epsmu,
                              const void *W, aweq_dtype dt, const float *s, const unsigned char *codes,
                              const float *step, const int *zp, const float *mu_hat,
                              long long C_out, long long C_in, long long ldw, int bits, aweq_gran gran, int group,
                              const void *bias_in, void *bias_out, float *bias_out_f32, aweq_dtype bias_dt,
                              aweq_dev_status *st, void *stream);

/*
 * Step 6 -- quantise the equalised inputs X^ = X diag(s)^-1 (Eq. 3) with
 * Eq. 1-2 (the activation half of the W8A8 setting of Section 4.4).
 * rinv: float[C_in] (1 / s) or NULL (no equalisation).  bits in 2..8, one code
 * per byte.  gran: AWEQ_PER_ROW = one (Step, Z) per token, computed from that
 * row; AWEQ_PER_TENSOR = a static range: tensor_lo_hi is float[2] = { lo, hi }
 * of X^ (for instance min_j xmin_j rinv_j and max_j xmax_j rinv_j from step 1)
 * and step / zp receive one pair.  Per-token mode supports C_in <= 40960.
 * Xq: unsigned char[N x C_in] (dense rows); step: float[N]; zp: int[N].
 */
aweq_status aweq_quant_act(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx,
                           const float *rinv, int bits, aweq_gran gran, const float *tensor_lo_hi,
                           unsigned char *Xq, float *step, int *zp,
                           aweq_dev_status *st, void *stream);

/*
 * One calibration pass for one input X and the n_w weight matrices it feeds,
 * all six steps in order on `stream` (steps 1-2, then 3, then 4-5 per matrix,
 * then 6 when Xq != NULL).  Per-channel vectors are float[C_in]; the arrays of
 * pointers and sizes are HOST arrays of length n_w, their elements device
 * pointers.  bias_in / bias_out / bias_out_f32 may be NULL, as may their
 * entries (see aweq_bias_correct).  flags: AWEQ_FLAG_* below.
 * ws must hold aweq_layer_pass_workspace_bytes().
 */
#define AWEQ_FLAG_NO_EQUALIZE 1      /* s = 1: plain round-to-nearest */
#define AWEQ_FLAG_NO_BIAS_CORRECT 2  /* skip step 5 */
/* Run only part of the pass (any combination; none of the three = the whole pass).  The parts
 * communicate through the per-channel arrays of the argument block, so a caller can put them
 * on different streams -- the shared-memory-staged, HBM-bound sweeps on one, the short
 * issue-bound weight kernels on another, where they fit beside a running sweep -- ordering
 * them with its own events and giving each stream its own `ws`:
 *   REDUCE  steps 1-2 (column reductions: writes xmin, xmax, xmean, wmin, wmax)
 *   QUANT   steps 3-5 (reads them; writes s, rinv, mu_hat, codes, Step, Z, biases)
 *   ACT     step 6 (reads rinv; writes Xq, act_step, act_zp) */
#define AWEQ_FLAG_PHASE_REDUCE 4
#define AWEQ_FLAG_PHASE_QUANT 8
#define AWEQ_FLAG_PHASE_ACT 16
#define AWEQ_FLAG_ABSMAX_CRITERION 32   /* step 3 through aweq_factors_absmax (comparison criterion) */
/* Token-sharded calibration (Section 3.3: the statistics are over all N inputs, wherever they
 * are held): the QUANT part first re-forms xmin, xmax and xmean = sum / count from the exchange
 * buffers stat_negmin_max / stat_sum_count of the argument block, which the caller has merged
 * over the shards between the REDUCE and the QUANT part (one MAX and one SUM all-reduce). */
#define AWEQ_FLAG_MERGED_STATS 64

typedef struct {
    /* input */
    const void *X; aweq_dtype dt; long long N, C_in, ldx;
    /* weights sharing this input (host arrays of length n_w) */
    int n_w;
    const void *const *W; const long long *C_out; const long long *ldw;
    int bits; aweq_gran gran; int group;
    const void *const *bias_in; void *const *bias_out; float *const *bias_out_f32;
    /* per-matrix outputs (host arrays of device pointers) */
    unsigned char *const *codes; float *const *step; int *const *zp; float *const *epsmu;
    /* per-channel outputs */
    float *xmin, *xmax, *xmean, *wmin, *wmax, *s, *rinv, *mu_hat;
    float *pX, *pW; double *scalars;             /* optional */
    /* activation quantisation (optional: Xq == NULL skips step 6) */
    unsigned char *Xq; float *act_step; int *act_zp; int act_bits;
    int flags;
    /* optional profiling hooks: cudaEvent_t handles (or NULL) recorded on `stream`
     * immediately before and after step 1 and step 6 */
    void *ev_stats_begin, *ev_stats_end, *ev_act_begin, *ev_act_end;
    /* optional exchange form of the step-1 statistics, both or neither; when given, the REDUCE
     * part also writes
     *   stat_negmin_max = float[2 C_in]   = { -xmin_j (j < C_in), xmax_j (j < C_in) }
     *   stat_sum_count  = double[C_in + 1] = { sum_n X[n,j] (j < C_in), N }
     * so that an element-wise MAX of the first and SUM of the second over several token shards
     * are the statistics of their union (see AWEQ_FLAG_MERGED_STATS) */
    float *stat_negmin_max; double *stat_sum_count;
} aweq_layer_args;

size_t aweq_layer_pass_workspace_bytes(const aweq_layer_args *args);
/* 1 when the pass takes steps 1 and 2 of this input in ONE launch (at most three matrices of at most
 * 400 MB together share the input: every CTA of the statistics sweep then also reduces its share of
 * their rows), else 0.
 * The profiling hooks around step 1 then bracket both steps.  Host logic only. */
int aweq_layer_pass_fuses_ranges(const aweq_layer_args *args);
aweq_status aweq_layer_pass(const aweq_layer_args *args, void *ws, size_t ws_bytes,
                            aweq_dev_status *st, void *stream);

/* ---- Folding diag(s)^-1 into the producer of a layer input (Section 3.1, text after Eq. 3:
 * the division by s is fused into the previous block) -------------------------------------
 *     out[r, c] = round16( float(P[r, c]) * rinv[r] )     r < rows, c < cols
 * (binary32 product, one round-to-nearest-even to the 16-bit type).  P is a 16-bit row-major
 * matrix with pitch ld elements: the weight matrix of the linear layer whose output channel
 * r is input channel r of the calibrated layer (rows = C_in of that layer), or, with
 * cols = 1, a bias vector or a normalisation layer's gain / shift.  rinv[rows] is step 3's
 * 1/s.  out (pitch ld_out) may be P itself (in place) but must not otherwise overlap it.
 * Any cols >= 1; 16-byte vector accesses are used when cols, ld, ld_out are multiples of 8
 * and both pointers are 16-byte aligned.  Device pointers; enqueued on `stream`. */
aweq_status aweq_fold_scale(const void *P, aweq_dtype dt, long long rows, long long cols, long long ld,
                            const float *rinv, void *out, long long ld_out, void *stream);

/* ---- Signed relabelling of 8-bit codes ------------------------------------------------------
 * Eq. 1 gives unsigned codes q in [0, 255] and a zero-point Z; consumers that take signed 8-bit
 * operands use q' = q - 128 and Z' = Z - 128 (saturating), which de-quantise to the same values,
 * Step (q' - Z') = Step (q - Z).  codes: n bytes, one 8-bit code each (step-6 activations or 8-bit
 * step-4 weights); out: n bytes, may be codes itself (in place).  zp / zp_out: nz zero-points, or
 * both NULL.  Device pointers; enqueued on `stream`. */
aweq_status aweq_relabel_signed(const unsigned char *codes, long long n, signed char *out,
                                const int *zp, long long nz, int *zp_out, void *stream);

/* ---- Forward check of a calibrated W8A8 layer (Eq. 11; the quantity ablated in the AWE / BC
 * table) ------------------------------------------------------------------------------------
 * Compares, on the calibration tokens, the quantised layer
 *     y~[n,o] = sum_k Step^x_n (Xq[n,k] - Z^x_n) * Step^w_o (Wq[o,k] - Z^w_o) + bias_q[o]
 * (Eq. 1-2 de-quantisation of the step-6 activation codes and of the 8-bit per-row step-4
 * weight codes; bias_q is the corrected bias of Eq. 15) with the 16-bit layer
 *     y[n,o] = sum_k X[n,k] W[o,k] + bias[o]
 * (equalisation leaves this product unchanged, Eq. 3).  Both contractions run on the tensor
 * cores: the integer one exactly (int32 accumulation, zero-points folded in afterwards in
 * 64-bit integers), the 16-bit one with binary32 accumulation.  Outputs (device):
 *   mean_err[C_out]  binary64, (1/N) sum_n (y~[n,o] - y[n,o])      -- E[y~_j - y_j] of Eq. 11
 *   sums[4]          binary64: sum (y~ - y)^2, sum y^2, sum_o mean_err[o]^2, N * C_out
 * Layout: Xq [N x C_in] and Wq [C_out x C_in] one byte per code, X and W 16-bit, all
 * row-major, contiguous (no pitch) and 16-byte aligned; act_step/act_zp [N], w_step/w_zp
 * [C_out]; bias (16-bit, [C_out]) may be NULL (a layer without bias); bias_q (binary32,
 * [C_out]) may be NULL: the quantised layer then keeps `bias` (no bias correction).
 * C_in must be a multiple of 16, C_out a multiple of 8 (AWEQ_ERR_SHAPE otherwise).
 * ws: aweq_forward_check_workspace_bytes(N, C_in, C_out) bytes, 256-byte aligned; nothing is
 * allocated.  Everything is enqueued on `stream`; the caller owns all buffers.
 * Returns AWEQ_ERR_UNSUPPORTED when the library was built without the tensor-core GEMM. */
size_t aweq_forward_check_workspace_bytes(long long N, long long C_in, long long C_out);
aweq_status aweq_forward_check(const unsigned char *Xq, const float *act_step, const int *act_zp,
                               const unsigned char *Wq, const float *w_step, const int *w_zp,
                               const float *bias_q, const void *X, const void *W, aweq_dtype dt,
                               const void *bias, long long N, long long C_in, long long C_out,
                               double *mean_err, double *sums, void *ws, size_t ws_bytes, void *stream);

/* ---- Forward check of a weight-only layer (Eq. 11; any bit-width and granularity of step 4) --
 * The quantised layer keeps 16-bit activations: with x^ = x diag(s)^-1 (Eq. 3, rinv = 1/s from
 * step 3, NULL = no equalisation) and W~ = Step (q - Z) the de-quantised step-4 codes,
 *     y~[n,o] = sum_j (X[n,j] rinv[j]) W~[o,j] + bias_q[o]        y[n,o] = sum_j X[n,j] W[o,j] + bias[o]
 * and the outputs are those of aweq_forward_check (mean_err[C_out], sums[4]; bias_q NULL = the
 * layer keeps bias).  The library forms dW = W~ rinv - W once; the mean error, linear in x, is
 * E[x] . dW from the binary64 column sums of X and the unrounded dW; the sums of squares come
 * from two 16-bit tensor-core GEMMs per token chunk, X round16(dW)^T (the error) and X W^T.
 * codes / step / zp / bits / gran / group exactly as aweq_equalize_quantize wrote them; X and W
 * contiguous, 16-byte aligned; C_in a multiple of 16 and within the range of aweq_stats, C_out
 * a multiple of 8.
 * ws: aweq_forward_check_weights_workspace_bytes(N, C_in, C_out), 256-byte aligned. */
size_t aweq_forward_check_weights_workspace_bytes(long long N, long long C_in, long long C_out);
aweq_status aweq_forward_check_weights(const unsigned char *codes, const float *step, const int *zp, int bits,
                                       aweq_gran gran, int group, const float *rinv, const float *bias_q,
                                       const void *X, const void *W, aweq_dtype dt, const void *bias,
                                       long long N, long long C_in, long long C_out, double *mean_err,
                                       double *sums, void *ws, size_t ws_bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* AWEQ_H */
