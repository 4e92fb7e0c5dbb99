// The C ABI: host-side validation, workspace sizing and the composition of the
// six calibration steps into one layer pass.  No device memory is allocated
// here and nothing synchronises.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "common.cuh"
#include "kernels.h"

namespace aweq {

static std::atomic<unsigned long long> g_launches{0};
static thread_local char g_cuda_error[256] = "";

void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

aweq_status cuda_failed(cudaError_t e)
{
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return AWEQ_ERR_CUDA;
}

// AWEQ_LOG=1 in the environment: one line per entry-point call on stderr (shapes and the
// algorithmic bytes the call moves); read once.
static bool log_enabled()
{
    static const bool on = [] { const char *e = getenv("AWEQ_LOG"); return e && e[0] && e[0] != '0'; }();
    return on;
}
#define AWEQ_LOGF(...)                                       \
    do {                                                     \
        if (::aweq::log_enabled()) fprintf(stderr, "[aweq] " __VA_ARGS__); \
    } while (0)

static inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
static inline size_t round256(size_t n) { return (n + 255) & ~(size_t)255; }

static aweq_status check_matrix(const void *M, aweq_dtype dt, long long rows, long long cols, long long ld,
                                bool allow_zero_rows)
{
    if (!M) return AWEQ_ERR_NULL;
    if (dt != AWEQ_F16 && dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (cols <= 0 || (cols % 8) != 0 || cols > (1ll << 30)) return AWEQ_ERR_SHAPE;
    if (rows < 0 || (rows == 0 && !allow_zero_rows) || rows > (1ll << 40)) return AWEQ_ERR_SHAPE;
    if (ld < cols || (ld % 8) != 0) return AWEQ_ERR_ALIGN;
    if (!aligned(M, 16)) return AWEQ_ERR_ALIGN;
    return AWEQ_OK;
}

static aweq_status check_quant(int bits, int gran, int group, long long cols)
{
    if (bits < 2 || bits > 8) return AWEQ_ERR_BITS;
    if (gran != AWEQ_PER_TENSOR && gran != AWEQ_PER_ROW && gran != AWEQ_PER_GROUP) return AWEQ_ERR_UNSUPPORTED;
    if (gran == AWEQ_PER_GROUP) {
        if (group < 8 || group > 256 || (group & (group - 1)) != 0 || (cols % group) != 0) return AWEQ_ERR_GROUP;
    }
    return AWEQ_OK;
}

static aweq_status check_ws(void *ws, size_t ws_bytes, size_t need)
{
    if (need == 0) return AWEQ_OK;
    if (!ws || !aligned(ws, 256) || ws_bytes < need) return AWEQ_ERR_WORKSPACE;
    return AWEQ_OK;
}

static size_t eq_ws_bytes(long long rows, long long cols, int bits, int gran, int group)
{
    // per group of 128: the (window, row) partial sums of eps . E[x^]
    if (gran == AWEQ_PER_GROUP) return groupquant_supported(bits, group) ? round256(groupquant_ws_bytes(rows, cols)) : 0;
    if (gran != AWEQ_PER_TENSOR) return 0;
    // per-tensor: column extremes of W (2 x float[cols]) + lo/hi + the column-reduction scratch
    return round256((size_t)cols * 8) + 256 + colreduce_ws_bytes(rows, cols);
}

}  // namespace aweq

using namespace aweq;

extern "C" {

const char *aweq_strerror(aweq_status code)
{
    switch (code) {
    case AWEQ_OK: return "ok";
    case AWEQ_ERR_NULL: return "a required pointer is NULL";
    case AWEQ_ERR_SHAPE: return "bad shape (sizes must be positive, C_in a multiple of 8 and within the supported range)";
    case AWEQ_ERR_ALIGN: return "bad alignment (16-byte base pointers, row pitch a multiple of 8 elements and >= C_in)";
    case AWEQ_ERR_DTYPE: return "unknown 16-bit element type";
    case AWEQ_ERR_BITS: return "bit-width must be in 2..8";
    case AWEQ_ERR_GROUP: return "group size must be a power of two in [8, 256] that divides C_in";
    case AWEQ_ERR_WORKSPACE: return "workspace missing, misaligned (256 bytes) or too small";
    case AWEQ_ERR_CUDA: return "a CUDA call failed";
    case AWEQ_ERR_UNSUPPORTED: return "unsupported mode";
    case AWEQ_ERR_LIMIT: return "size beyond the built-in scratch of aweq_stats_static (C_in <= 16384)";
    }
    return "unknown status";
}

const char *aweq_last_cuda_error(void) { return g_cuda_error; }
int aweq_version(void) { return 101; }
unsigned long long aweq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

aweq_status aweq_plan_query(int op, long long rows, long long cols, long long plan[8])
{
    if (!plan) return AWEQ_ERR_NULL;
    if (rows <= 0 || cols <= 0 || cols % 8 || cols > (1ll << 30)) return AWEQ_ERR_SHAPE;
    if (op == AWEQ_OP_STATS || op == AWEQ_OP_WRANGE) {
        colreduce_describe(rows, cols, plan);
        return AWEQ_OK;
    }
    if (op == AWEQ_OP_EQUALIZE_QUANTIZE || op == AWEQ_OP_QUANT_ACT)
        return rowquant_describe(rows, cols, op == AWEQ_OP_EQUALIZE_QUANTIZE, plan) ? AWEQ_OK : AWEQ_ERR_SHAPE;
    return AWEQ_ERR_UNSUPPORTED;
}

size_t aweq_workspace_bytes(int op, long long rows, long long cols, int bits, int gran, int group)
{
    if (cols <= 0 || rows < 0) return 0;
    switch (op) {
    case AWEQ_OP_STATS:
    case AWEQ_OP_WRANGE: return colreduce_ws_bytes(rows, cols);
    case AWEQ_OP_EQUALIZE_QUANTIZE: return eq_ws_bytes(rows, cols, bits, gran, group);
    default: return 0;
    }
}

aweq_status aweq_stats(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx, float *xmin,
                       float *xmax, float *xmean, double *xsum, long long *count, int accumulate, void *ws,
                       size_t ws_bytes, aweq_dev_status *st, void *stream)
{
    aweq_status rc = check_matrix(X, dt, N, C_in, ldx, true);
    if (rc != AWEQ_OK) return rc;
    if (!xmin || !xmax || !xmean) return AWEQ_ERR_NULL;
    if (accumulate && (!xsum || !count)) return AWEQ_ERR_NULL;
    if (!aligned(xmin, 16) || !aligned(xmax, 16) || !aligned(xmean, 4) || (xsum && !aligned(xsum, 8)))
        return AWEQ_ERR_ALIGN;
    rc = check_ws(ws, ws_bytes, colreduce_ws_bytes(N, C_in));
    if (rc != AWEQ_OK) return rc;
    AWEQ_LOGF("aweq_stats N=%lld C_in=%lld ld=%lld dtype=%d accumulate=%d bytes=%lld\n", N, C_in, ldx, (int)dt, accumulate,
              2 * N * C_in);
    return run_stats(X, dt, N, C_in, ldx, xmin, xmax, xmean, xsum, count, accumulate, ws, st, (cudaStream_t)stream);
}

aweq_status aweq_wrange(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ldw, float *wmin,
                        float *wmax, int accumulate, void *ws, size_t ws_bytes, aweq_dev_status *st, void *stream)
{
    aweq_status rc = check_matrix(W, dt, C_out, C_in, ldw, false);
    if (rc != AWEQ_OK) return rc;
    if (!wmin || !wmax) return AWEQ_ERR_NULL;
    rc = check_ws(ws, ws_bytes, colreduce_ws_bytes(C_out, C_in));
    if (rc != AWEQ_OK) return rc;
    AWEQ_LOGF("aweq_wrange C_out=%lld C_in=%lld accumulate=%d bytes=%lld\n", C_out, C_in, accumulate, 2 * C_out * C_in);
    return run_wrange(W, dt, C_out, C_in, ldw, wmin, wmax, accumulate, ws, st, (cudaStream_t)stream);
}

aweq_status aweq_factors(const float *xmin, const float *xmax, const float *xmean, const float *wmin,
                         const float *wmax, long long C_in, float *s, float *rinv, float *mu_hat, float *pX,
                         float *pW, double *scalars, aweq_dev_status *st, void *stream)
{
    if (!xmin || !xmax || !xmean || !wmin || !wmax || !s || !rinv || !mu_hat) return AWEQ_ERR_NULL;
    if (C_in <= 0 || C_in > (1ll << 20)) return AWEQ_ERR_SHAPE;
    return run_factors(xmin, xmax, xmean, wmin, wmax, C_in, s, rinv, mu_hat, pX, pW, scalars, st,
                       (cudaStream_t)stream);
}

aweq_status aweq_factors_absmax(const float *xmin, const float *xmax, const float *xmean, const float *wmin,
                                const float *wmax, long long C_in, float *s, float *rinv, float *mu_hat, float *pX,
                                float *pW, double *scalars, aweq_dev_status *st, void *stream)
{
    if (!xmin || !xmax || !xmean || !wmin || !wmax || !s || !rinv || !mu_hat) return AWEQ_ERR_NULL;
    if (C_in <= 0 || C_in > (1ll << 20)) return AWEQ_ERR_SHAPE;
    return run_factors(xmin, xmax, xmean, wmin, wmax, C_in, s, rinv, mu_hat, pX, pW, scalars, st,
                       (cudaStream_t)stream, 1);
}

static aweq_status equalize_quantize_impl(const void *W, aweq_dtype dt, long long C_out, long long C_in,
                                          long long ldw, const float *s, const float *mu_hat, int bits,
                                          aweq_gran gran, int group, unsigned char *codes, float *step, int *zp,
                                          float *epsmu, const BiasIO &bias, void *ws, size_t ws_bytes,
                                          aweq_dev_status *st, void *stream)
{
    aweq_status rc = check_matrix(W, dt, C_out, C_in, ldw, false);
    if (rc != AWEQ_OK) return rc;
    rc = check_quant(bits, gran, group, C_in);
    if (rc != AWEQ_OK) return rc;
    if (!codes || !step || !zp) return AWEQ_ERR_NULL;
    if (!aligned(codes, 16) || (s && !aligned(s, 16)) || (mu_hat && !aligned(mu_hat, 16))) return AWEQ_ERR_ALIGN;
    rc = check_ws(ws, ws_bytes, eq_ws_bytes(C_out, C_in, bits, gran, group));
    if (rc != AWEQ_OK) return rc;
    AWEQ_LOGF("aweq_equalize_quantize C_out=%lld C_in=%lld bits=%d gran=%d group=%d bytes=%lld\n", C_out, C_in, bits,
              (int)gran, group, 2 * C_out * C_in + C_out * C_in * bits / 8);
    cudaStream_t cs = (cudaStream_t)stream;
    if (gran == AWEQ_PER_ROW) {
        if (!rowquant_supported(C_out, C_in)) return AWEQ_ERR_SHAPE;
        return run_rowquant(W, dt, C_out, C_in, ldw, s, mu_hat, bits, true, codes, step, zp, epsmu, bias, st, cs);
    }
    if (gran == AWEQ_PER_GROUP && groupquant_supported(bits, group))
        return run_groupquant(W, dt, C_out, C_in, ldw, s, mu_hat, bits, codes, step, zp, epsmu, bias, ws, cs);
    if (gran == AWEQ_PER_GROUP)
        return run_warpquant(W, dt, C_out, C_in, ldw, s, mu_hat, bits, true, group, nullptr, codes, step, zp, epsmu,
                             bias, st, cs);
    // per tensor: column extremes of W -> extremes of diag(s) W -> static-range quantiser
    char *base = reinterpret_cast<char *>(ws);
    float *cmin = reinterpret_cast<float *>(base);
    float *cmax = cmin + C_in;
    float *lo_hi = reinterpret_cast<float *>(base + round256((size_t)C_in * 8));
    void *ws2 = base + round256((size_t)C_in * 8) + 256;
    rc = run_wrange(W, dt, C_out, C_in, ldw, cmin, cmax, 0, ws2, st, cs);
    if (rc != AWEQ_OK) return rc;
    rc = run_scaled_tensor_range(cmin, cmax, s, C_in, lo_hi, cs);
    if (rc != AWEQ_OK) return rc;
    return run_warpquant(W, dt, C_out, C_in, ldw, s, mu_hat, bits, true, 0, lo_hi, codes, step, zp, epsmu, bias, st,
                         cs);
}

aweq_status aweq_equalize_quantize(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ldw,
                                   const float *s, const float *mu_hat, int bits, aweq_gran gran, int group,
                                   unsigned char *codes, float *step, int *zp, float *epsmu, void *ws,
                                   size_t ws_bytes, aweq_dev_status *st, void *stream)
{
    const BiasIO none = {nullptr, nullptr, nullptr, 0};
    return equalize_quantize_impl(W, dt, C_out, C_in, ldw, s, mu_hat, bits, gran, group, codes, step, zp, epsmu, none,
                                  ws, ws_bytes, st, stream);
}

aweq_status aweq_bias_correct(const float *epsmu, const void *W, aweq_dtype dt, const float *s,
                              const unsigned char *codes, const float *step, const int *zp, const float *mu_hat,
                              long long C_out, long long C_in, long long ldw, int bits, aweq_gran gran, int group,
                              const void *bias_in, void *bias_out, float *bias_out_f32, aweq_dtype bias_dt,
                              aweq_dev_status *st, void *stream)
{
    (void)st;
    if (C_out <= 0) return AWEQ_ERR_SHAPE;
    if (!bias_out && !bias_out_f32) return AWEQ_ERR_NULL;
    if (bias_dt != AWEQ_F16 && bias_dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (epsmu) return run_bias_apply(epsmu, bias_in, bias_out, bias_out_f32, bias_dt, C_out, (cudaStream_t)stream);
    aweq_status rc = check_matrix(W, dt, C_out, C_in, ldw, false);
    if (rc != AWEQ_OK) return rc;
    rc = check_quant(bits, gran, group, C_in);
    if (rc != AWEQ_OK) return rc;
    if (!codes || !step || !zp || !mu_hat) return AWEQ_ERR_NULL;
    return run_bias_gemv(W, dt, C_out, C_in, ldw, s, codes, step, zp, mu_hat, bits, gran, group, bias_in, bias_out,
                         bias_out_f32, bias_dt, (cudaStream_t)stream);
}

aweq_status aweq_quant_act(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx,
                           const float *rinv, int bits, aweq_gran gran, const float *tensor_lo_hi,
                           unsigned char *Xq, float *step, int *zp, aweq_dev_status *st, void *stream)
{
    aweq_status rc = check_matrix(X, dt, N, C_in, ldx, false);
    if (rc != AWEQ_OK) return rc;
    if (bits < 2 || bits > 8) return AWEQ_ERR_BITS;
    if (!Xq || !step || !zp) return AWEQ_ERR_NULL;
    if (!aligned(Xq, 16) || (rinv && !aligned(rinv, 16))) return AWEQ_ERR_ALIGN;
    AWEQ_LOGF("aweq_quant_act N=%lld C_in=%lld bits=%d gran=%d bytes=%lld\n", N, C_in, bits, (int)gran, 3 * N * C_in + 8 * N);
    cudaStream_t cs = (cudaStream_t)stream;
    if (gran == AWEQ_PER_ROW) {
        if (!rowquant_supported(N, C_in)) return AWEQ_ERR_SHAPE;
        const BiasIO none = {nullptr, nullptr, nullptr, 0};
        return run_rowquant(X, dt, N, C_in, ldx, rinv, nullptr, bits, false, Xq, step, zp, nullptr, none, st, cs);
    }
    if (gran == AWEQ_PER_TENSOR) {
        if (!tensor_lo_hi) return AWEQ_ERR_NULL;
        const BiasIO none = {nullptr, nullptr, nullptr, 0};
        return run_warpquant(X, dt, N, C_in, ldx, rinv, nullptr, bits, false, 0, tensor_lo_hi, Xq, step, zp, nullptr,
                             none, st, cs);
    }
    return AWEQ_ERR_UNSUPPORTED;
}

// ------------------------------------------------------------------ layer pass
// workspace layout: [column-reduction scratch | scratch of step 4]
static size_t layer_ws_parts(const aweq_layer_args *a, size_t *col_part)
{
    size_t col = stats_wrange_fusable(a->N, a->C_in, a->C_out, a->n_w) ? colreduce_fused_ws_bytes(a->N, a->C_in)
                                                     : colreduce_ws_bytes(a->N, a->C_in);
    size_t eq = 0;
    for (int i = 0; i < a->n_w; ++i) {
        size_t c = colreduce_ws_bytes(a->C_out[i], a->C_in);
        if (c > col) col = c;
        size_t e = eq_ws_bytes(a->C_out[i], a->C_in, a->bits, a->gran, a->group);
        if (e > eq) eq = e;
    }
    col = round256(col);
    if (col_part) *col_part = col;
    return col + round256(eq);
}

int aweq_layer_pass_fuses_ranges(const aweq_layer_args *args)
{
    return args && args->C_out && stats_wrange_fusable(args->N, args->C_in, args->C_out, args->n_w) ? 1 : 0;
}

size_t aweq_layer_pass_workspace_bytes(const aweq_layer_args *args)
{
    if (!args || args->n_w <= 0 || !args->C_out || args->C_in <= 0) return 0;
    return layer_ws_parts(args, nullptr);
}

// A profiling hook.  While the stream is being captured into a CUDA graph an ordinary record would
// only become an edge of the graph; as an external record it becomes a node of its own, so the
// event is recorded anew on every replay and can be read back afterwards.
static cudaError_t record_hook(void *ev, cudaStream_t cs)
{
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    cudaError_t e = cudaStreamIsCapturing(cs, &cap);
    if (e != cudaSuccess) return e;
    return cudaEventRecordWithFlags((cudaEvent_t)ev, cs,
                                    cap == cudaStreamCaptureStatusActive ? cudaEventRecordExternal : cudaEventRecordDefault);
}

aweq_status aweq_layer_pass(const aweq_layer_args *a, void *ws, size_t ws_bytes, aweq_dev_status *st, void *stream)
{
    if (!a) return AWEQ_ERR_NULL;
    if (a->n_w <= 0 || !a->W || !a->C_out || !a->ldw || !a->codes || !a->step || !a->zp) return AWEQ_ERR_NULL;
    if (!a->xmin || !a->xmax || !a->xmean || !a->wmin || !a->wmax || !a->s || !a->rinv || !a->mu_hat)
        return AWEQ_ERR_NULL;
    aweq_status rc = check_matrix(a->X, a->dt, a->N, a->C_in, a->ldx, false);
    if (rc != AWEQ_OK) return rc;
    rc = check_quant(a->bits, a->gran, a->group, a->C_in);
    if (rc != AWEQ_OK) return rc;
    for (int i = 0; i < a->n_w; ++i) {
        rc = check_matrix(a->W[i], a->dt, a->C_out[i], a->C_in, a->ldw[i], false);
        if (rc != AWEQ_OK) return rc;
        if (!a->codes[i] || !a->step[i] || !a->zp[i]) return AWEQ_ERR_NULL;
    }
    const bool bc = !(a->flags & AWEQ_FLAG_NO_BIAS_CORRECT);
    if (bc && (!a->epsmu || (!a->bias_out && !a->bias_out_f32))) return AWEQ_ERR_NULL;
    for (int i = 0; bc && i < a->n_w; ++i) {
        if (!a->epsmu[i]) return AWEQ_ERR_NULL;
        if (!(a->bias_out && a->bias_out[i]) && !(a->bias_out_f32 && a->bias_out_f32[i])) return AWEQ_ERR_NULL;
    }
    if (a->Xq && (!a->act_step || !a->act_zp)) return AWEQ_ERR_NULL;
    if ((a->stat_negmin_max == nullptr) != (a->stat_sum_count == nullptr)) return AWEQ_ERR_NULL;
    if ((a->flags & AWEQ_FLAG_MERGED_STATS) && !a->stat_negmin_max) return AWEQ_ERR_NULL;
    if (a->stat_negmin_max && (!aligned(a->stat_negmin_max, 4) || !aligned(a->stat_sum_count, 8))) return AWEQ_ERR_ALIGN;
    size_t col_part = 0;
    const size_t need = layer_ws_parts(a, &col_part);
    rc = check_ws(ws, ws_bytes, need);
    if (rc != AWEQ_OK) return rc;
    char *base = reinterpret_cast<char *>(ws);
    void *ws_col = base;
    void *ws_eq = base + col_part;
    const size_t ws_eq_bytes = need - col_part;

    cudaStream_t cs = (cudaStream_t)stream;
    const int kAllPhases = AWEQ_FLAG_PHASE_REDUCE | AWEQ_FLAG_PHASE_QUANT | AWEQ_FLAG_PHASE_ACT;
    const int phases = (a->flags & kAllPhases) ? (a->flags & kAllPhases) : kAllPhases;
    // steps 1-2
    if (phases & AWEQ_FLAG_PHASE_REDUCE) {
        if (a->ev_stats_begin) AWEQ_CUDA_OK(record_hook(a->ev_stats_begin, cs));
        if (!aligned(a->xmin, 16) || !aligned(a->xmax, 16) || !aligned(a->xmean, 4)) return AWEQ_ERR_ALIGN;
        if (stats_wrange_fusable(a->N, a->C_in, a->C_out, a->n_w)) {
            // steps 1 and 2 in one launch: every CTA of the sweep also takes its share of the rows of the
            // matrices this input feeds (they have the same columns), so step 2 has no launch, fill or
            // drain of its own.  The hook interval then covers both steps.
            AWEQ_LOGF("aweq_stats + aweq_wrange x%d N=%lld C_in=%lld bytes=%lld (one launch)\n", a->n_w, a->N, a->C_in,
                      2 * a->N * a->C_in);
            rc = run_stats_wrange(a->X, a->dt, a->N, a->C_in, a->ldx, a->xmin, a->xmax, a->xmean, a->W, a->C_out, a->ldw,
                                  a->n_w, a->wmin, a->wmax, ws_col, st, cs, a->stat_negmin_max, a->stat_sum_count);
            if (rc != AWEQ_OK) return rc;
            if (a->ev_stats_end) AWEQ_CUDA_OK(record_hook(a->ev_stats_end, cs));
        } else {
            if (a->stat_negmin_max) {
                // the sweep that also leaves the exchange form of the statistics
                AWEQ_LOGF("aweq_stats N=%lld C_in=%lld (with exchange buffers) bytes=%lld\n", a->N, a->C_in, 2 * a->N * a->C_in);
                rc = run_stats(a->X, a->dt, a->N, a->C_in, a->ldx, a->xmin, a->xmax, a->xmean, nullptr, nullptr, 0, ws_col,
                               st, cs, a->stat_negmin_max, a->stat_sum_count);
            } else {
                rc = aweq_stats(a->X, a->dt, a->N, a->C_in, a->ldx, a->xmin, a->xmax, a->xmean, nullptr, nullptr, 0, ws_col,
                                col_part, st, stream);
            }
            if (rc != AWEQ_OK) return rc;
            if (a->ev_stats_end) AWEQ_CUDA_OK(record_hook(a->ev_stats_end, cs));
            // step 2: the matrices share the input, hence one range per input channel over all of them
            AWEQ_LOGF("aweq_wrange x%d C_in=%lld\n", a->n_w, a->C_in);
            rc = run_wrange_multi(a->W, a->C_out, a->ldw, a->n_w, a->dt, a->C_in, a->wmin, a->wmax, 0, ws_col, st, cs);
            if (rc != AWEQ_OK) return rc;
        }
    }
    const bool eq = !(a->flags & AWEQ_FLAG_NO_EQUALIZE);
    // without equalisation the layer sees x itself, so E[x^] = E[x]
    const float *s_used = eq ? a->s : nullptr;
    const float *rinv_used = eq ? a->rinv : nullptr;
    const float *mu_used = eq ? a->mu_hat : a->xmean;
    if (phases & AWEQ_FLAG_PHASE_QUANT) {
    if (a->flags & AWEQ_FLAG_MERGED_STATS) {
        rc = run_stats_from_exchange(a->stat_negmin_max, a->stat_sum_count, a->C_in, a->xmin, a->xmax, a->xmean, cs);
        if (rc != AWEQ_OK) return rc;
    }
    // step 3
    rc = ((a->flags & AWEQ_FLAG_ABSMAX_CRITERION) ? aweq_factors_absmax : aweq_factors)(
        a->xmin, a->xmax, a->xmean, a->wmin, a->wmax, a->C_in, a->s, a->rinv, a->mu_hat, a->pX, a->pW, a->scalars, st,
        stream);
    if (rc != AWEQ_OK) return rc;
    // steps 4-5 per matrix: the corrected bias is written by the quantiser itself
    for (int i = 0; i < a->n_w; ++i) {
        float *em = bc ? a->epsmu[i] : nullptr;
        BiasIO bias = {nullptr, nullptr, nullptr, a->dt == AWEQ_BF16};
        if (bc) {
            bias.in = reinterpret_cast<const uint16_t *>(a->bias_in ? a->bias_in[i] : nullptr);
            bias.out = reinterpret_cast<uint16_t *>(a->bias_out ? a->bias_out[i] : nullptr);
            bias.out_f32 = a->bias_out_f32 ? a->bias_out_f32[i] : nullptr;
        }
        rc = equalize_quantize_impl(a->W[i], a->dt, a->C_out[i], a->C_in, a->ldw[i], s_used, bc ? mu_used : nullptr,
                                    a->bits, a->gran, a->group, a->codes[i], a->step[i], a->zp[i], em, bias, ws_eq,
                                    ws_eq_bytes, st, stream);
        if (rc != AWEQ_OK) return rc;
    }
    }
    // step 6
    if (a->Xq && (phases & AWEQ_FLAG_PHASE_ACT)) {
        if (a->ev_act_begin) AWEQ_CUDA_OK(record_hook(a->ev_act_begin, cs));
        rc = aweq_quant_act(a->X, a->dt, a->N, a->C_in, a->ldx, rinv_used, a->act_bits ? a->act_bits : 8, AWEQ_PER_ROW,
                            nullptr, a->Xq, a->act_step, a->act_zp, st, stream);
        if (rc != AWEQ_OK) return rc;
        if (a->ev_act_end) AWEQ_CUDA_OK(record_hook(a->ev_act_end, cs));
    }
    return AWEQ_OK;
}

// ------------------------------------------------------------------ folding 1/s into the producer
aweq_status aweq_fold_scale(const void *P, aweq_dtype dt, long long rows, long long cols, long long ld,
                            const float *rinv, void *out, long long ld_out, void *stream)
{
    if (!P || !rinv || !out) return AWEQ_ERR_NULL;
    if (dt != AWEQ_F16 && dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (rows <= 0 || cols <= 0 || rows > (1ll << 40) || cols > (1ll << 30)) return AWEQ_ERR_SHAPE;
    if (ld < cols || ld_out < cols) return AWEQ_ERR_ALIGN;
    if (!aligned(P, 2) || !aligned(out, 2) || !aligned(rinv, 4)) return AWEQ_ERR_ALIGN;
    AWEQ_LOGF("aweq_fold_scale rows=%lld cols=%lld bytes=%lld\n", rows, cols, 4 * rows * cols + 4 * rows);
    return run_fold_scale(P, dt, rows, cols, ld, rinv, out, ld_out, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ signed relabelling
aweq_status aweq_relabel_signed(const unsigned char *codes, long long n, signed char *out, const int *zp, long long nz,
                                int *zp_out, void *stream)
{
    if (!codes || !out) return AWEQ_ERR_NULL;
    if ((zp == nullptr) != (zp_out == nullptr)) return AWEQ_ERR_NULL;
    if (n <= 0 || nz < 0 || (zp && nz == 0)) return AWEQ_ERR_SHAPE;
    return run_relabel_signed(codes, n, out, zp, zp ? nz : 0, zp_out, (cudaStream_t)stream);
}

// ------------------------------------------------------------------ forward check
size_t aweq_forward_check_workspace_bytes(long long N, long long C_in, long long C_out)
{
    if (N <= 0 || C_in <= 0 || C_out <= 0) return 0;
    return forward_check_ws_bytes(N, C_in, C_out);
}

aweq_status aweq_forward_check(const unsigned char *Xq, const float *act_step, const int *act_zp,
                               const unsigned char *Wq, const float *w_step, const int *w_zp, const float *bias_q,
                               const void *X, const void *W, aweq_dtype dt, const void *bias, long long N,
                               long long C_in, long long C_out, double *mean_err, double *sums, void *ws,
                               size_t ws_bytes, void *stream)
{
    if (!Xq || !act_step || !act_zp || !Wq || !w_step || !w_zp || !X || !W || !mean_err || !sums) return AWEQ_ERR_NULL;
    if (dt != AWEQ_F16 && dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (N <= 0 || C_in <= 0 || C_out <= 0 || C_in % 16 || C_out % 8) return AWEQ_ERR_SHAPE;
    if (C_in > (1ll << 30) || C_out > (1ll << 30) || N > (1ll << 34)) return AWEQ_ERR_SHAPE;
    if (!aligned(Xq, 16) || !aligned(Wq, 16) || !aligned(X, 16) || !aligned(W, 16)) return AWEQ_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < forward_check_ws_bytes(N, C_in, C_out)) return AWEQ_ERR_WORKSPACE;
    AWEQ_LOGF("aweq_forward_check N=%lld C_in=%lld C_out=%lld flops=%.3e\n", N, C_in, C_out, 4.0 * N * C_in * C_out);
    return run_forward_check(Xq, act_step, act_zp, Wq, w_step, w_zp, bias_q, X, W, dt, bias, N, C_in, C_out, mean_err,
                             sums, ws, ws_bytes, (cudaStream_t)stream);
}

size_t aweq_forward_check_weights_workspace_bytes(long long N, long long C_in, long long C_out)
{
    if (N <= 0 || C_in <= 0 || C_out <= 0) return 0;
    return forward_check_weights_ws_bytes(N, C_in, C_out);
}

aweq_status aweq_forward_check_weights(const unsigned char *codes, const float *step, const int *zp, int bits,
                                       aweq_gran gran, int group, const float *rinv, const float *bias_q,
                                       const void *X, const void *W, aweq_dtype dt, const void *bias, long long N,
                                       long long C_in, long long C_out, double *mean_err, double *sums, void *ws,
                                       size_t ws_bytes, void *stream)
{
    if (!codes || !step || !zp || !X || !W || !mean_err || !sums) return AWEQ_ERR_NULL;
    if (dt != AWEQ_F16 && dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (N <= 0 || C_in <= 0 || C_out <= 0 || C_in % 16 || C_out % 8) return AWEQ_ERR_SHAPE;
    if (C_in > (1ll << 30) || C_out > (1ll << 30) || N > (1ll << 34)) return AWEQ_ERR_SHAPE;
    aweq_status rc = check_quant(bits, gran, group, C_in);
    if (rc != AWEQ_OK) return rc;
    if (!aligned(X, 16) || !aligned(W, 16) || (rinv && !aligned(rinv, 16))) return AWEQ_ERR_ALIGN;
    if (!ws || !aligned(ws, 256) || ws_bytes < forward_check_weights_ws_bytes(N, C_in, C_out)) return AWEQ_ERR_WORKSPACE;
    AWEQ_LOGF("aweq_forward_check_weights N=%lld C_in=%lld C_out=%lld bits=%d flops=%.3e\n", N, C_in, C_out, bits,
              4.0 * N * C_in * C_out);
    return run_forward_check_weights(codes, step, zp, bits, gran, group, rinv, bias_q, X, W, dt, bias, N, C_in, C_out,
                                     mean_err, sums, ws, ws_bytes, (cudaStream_t)stream);
}

}  // extern "C"
