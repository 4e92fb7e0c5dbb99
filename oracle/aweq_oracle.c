/*
 * AWEQ calibration pass -- plain CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, obviously-correct statement of what one AWEQ
 * per-linear-layer calibration pass computes (arXiv 2311.01305).  It exists so
 * that the CUDA library can be checked against something that was written
 * from the paper and shares nothing with it: no headers, helpers, tables or
 * constants are common to the two.  Only tests, the smoke check and the
 * CPU-baseline leg of the benchmark may call it; it is never a fallback.
 *
 * Everything is a scalar loop in the order the paper states the operation.
 * Sums are fp64.  Where an integer code depends on floating point (Eq. 1-2)
 * the decision is taken in IEEE binary32 with round-to-nearest-even and no
 * fused multiply-add (build with -ffp-contract=off), which is the precision
 * the quantised layer itself uses.
 *
 * Passages followed
 *   stats / ranges ....... Section 3.2, text below Eq. 4 (channel range =
 *                          max - min of a channel; tensor range = max - min
 *                          over all channels); Section 3.3, last paragraph
 *                          (E[x] is gathered together with S).
 *   factors .............. Eq. 10 (literal form), Eq. 4 (precision p = r/R),
 *                          Eq. 5 (objective), Eq. 8 (max*max form).
 *   equalisation ......... Eq. 3 (X diag(s)^-1 and diag(s) W).
 *   quantiser ............ Eq. 1 and Eq. 2.
 *   bias correction ...... Eq. 11 - Eq. 15 and the sentence after them
 *                          (subtract eps * E[x]); eps = W~ - W.
 *   forward check ........ Eq. 11 (E[y~ - y]) evaluated on data from the
 *                          Eq. 1-2 de-quantised codes and the 16-bit layer.
 *
 * Conventions the paper does not fix (parity unpinned: both sides simply
 * follow the same rule):
 *   - dead channels (a zero or non-finite range): s = 1;
 *   - a constant vector (Step would be 0): Step = |lo|, or 1 when lo == 0;
 *   - zero-point and rounded values saturate to the int32 range (the rule is
 *     this build's; what it gives is pinned by hand-worked vectors);
 *   - sub-byte code packing: 4-bit two per byte, low nibble first; 3-bit as a
 *     dense little-endian bit stream, eight codes per three bytes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F16 0
#define ORACLE_BF16 1
#define ORACLE_PER_TENSOR 0
#define ORACLE_PER_ROW 1
#define ORACLE_PER_GROUP 2

/* ------------------------------------------------------------------ */
/* 16-bit storage formats, decoded by their published bit layouts.     */
/* ------------------------------------------------------------------ */

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static float decode_f16(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1f;
    int frac = h & 0x3ff;
    double v;
    if (expo == 0)
        v = ldexp((double)frac, -24);            /* subnormal: frac * 2^-24 */
    else if (expo == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    return (float)(sign ? -v : v);
}

/* bfloat16: the upper half of an IEEE binary32. */
static float decode_bf16(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return f;
}

static float decode16(uint16_t h, int dtype)
{
    return dtype == ORACLE_F16 ? decode_f16(h) : decode_bf16(h);
}

/* Round a double to the nearest 16-bit value (ties to even), one rounding. */
static uint16_t encode16(double x, int dtype)
{
    int mant_bits = dtype == ORACLE_F16 ? 10 : 7;
    int emin = dtype == ORACLE_F16 ? -14 : -126;      /* smallest normal exponent */
    int emax = dtype == ORACLE_F16 ? 15 : 127;
    int ebias = dtype == ORACLE_F16 ? 15 : 127;
    int ebits = dtype == ORACLE_F16 ? 5 : 8;
    uint16_t sign = (uint16_t)(signbit(x) ? 1u << 15 : 0);
    if (isnan(x))
        return (uint16_t)(sign | (((1u << ebits) - 1) << mant_bits) | 1u);
    double a = fabs(x);
    if (a == 0.0)
        return sign;
    int e;
    (void)frexp(a, &e);                 /* a = m * 2^e with m in [0.5, 1) */
    e -= 1;                             /* a = m' * 2^e with m' in [1, 2)  */
    if (e < emin)
        e = emin;
    /* spacing of representable values in this binade */
    double ulp = ldexp(1.0, e - mant_bits);
    double q = nearbyint(a / ulp);      /* default rounding mode: ties to even */
    if (q >= ldexp(1.0, mant_bits + 1)) {   /* rounded up into the next binade */
        q /= 2.0;
        e += 1;
    }
    if (e > emax || isinf(a))
        return (uint16_t)(sign | (((1u << ebits) - 1) << mant_bits));
    uint32_t qi = (uint32_t)q;
    if (qi < (1u << mant_bits))         /* subnormal result (e == emin) */
        return (uint16_t)(sign | qi);
    return (uint16_t)(sign | ((uint32_t)(e + ebias) << mant_bits) | (qi - (1u << mant_bits)));
}

void oracle_decode16(const uint16_t *in, int dtype, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = decode16(in[i], dtype);
}

void oracle_encode16(const double *in, int dtype, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i)
        out[i] = encode16(in[i], dtype);
}

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0)
        omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------ */
/* Step 1: per-channel min, max and mean of the calibration inputs.    */
/* Section 3.2 (channel range) and Section 3.3 (E[x] gathered in the   */
/* same sweep).  X is [N x C] row-major with row pitch ld elements.    */
/* xsum (optional) receives the fp64 column sums.                      */
/* ------------------------------------------------------------------ */
void oracle_stats(const uint16_t *X, int dtype, int64_t N, int64_t C, int64_t ld,
                  float *xmin, float *xmax, float *xmean, double *xsum)
{
    /* channels are independent; each one is reduced over n = 0..N-1 in order */
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < C; ++j) {
        float lo = INFINITY, hi = -INFINITY;
        double sum = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            float v = decode16(X[n * ld + j], dtype);
            if (v < lo) lo = v;
            if (v > hi) hi = v;
            sum += (double)v;
        }
        xmin[j] = lo;
        xmax[j] = hi;
        xmean[j] = N > 0 ? (float)(sum / (double)N) : 0.0f;
        if (xsum)
            xsum[j] = sum;
    }
}

/* ------------------------------------------------------------------ */
/* Step 2: per-input-channel weight range.  W is [C_out x C_in]; the    */
/* channel index i of the paper is the input channel, shared with X.   */
/* accumulate != 0 merges with the values already in wmin/wmax, which   */
/* is how several matrices fed by one input get one common range.      */
/* ------------------------------------------------------------------ */
void oracle_wrange(const uint16_t *W, int dtype, int64_t C_out, int64_t C_in, int64_t ld,
                   float *wmin, float *wmax, int accumulate)
{
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < C_in; ++j) {
        float lo = accumulate ? wmin[j] : INFINITY;
        float hi = accumulate ? wmax[j] : -INFINITY;
        for (int64_t o = 0; o < C_out; ++o) {
            float v = decode16(W[o * ld + j], dtype);
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
        wmin[j] = lo;
        wmax[j] = hi;
    }
}

/* ------------------------------------------------------------------ */
/* Step 3: equalisation factors.                                        */
/*   r^X_i = xmax_i - xmin_i, r^W_i = wmax_i - wmin_i  (binary32)       */
/*   s_i = (1 / r^W_i) * sqrt(r^X_i * r^W_i)            Eq. 10, fp64,   */
/*         rounded once to binary32                                     */
/*   rinv_i = 1 / s_i,  mu_hat_i = xmean_i * rinv_i  (E[x^] of Eq. 15   */
/*         for the equalised input x^ = x / s)                          */
/*   p^X_i = r^X_i / R^X,  p^W_i = r^W_i / R^W          Eq. 4, with R   */
/*         the tensor range (global max - global min)                   */
/* scalars[0..7]: R^X, R^W, R^X^ , R^W^ (tensor ranges after            */
/*   equalisation), objective of Eq. 5 before and after, and the        */
/*   max*max product of Eq. 8 before (s = 1) and after.                 */
/* Returns the number of dead channels (s forced to 1).                 */
/* ------------------------------------------------------------------ */
int64_t oracle_factors(const float *xmin, const float *xmax, const float *xmean,
                       const float *wmin, const float *wmax, int64_t C,
                       float *s, float *rinv, float *mu_hat, float *pX, float *pW,
                       double *scalars, int criterion)
{
    int64_t dead = 0;
    double gxlo = INFINITY, gxhi = -INFINITY, gwlo = INFINITY, gwhi = -INFINITY;
    double exlo = INFINITY, exhi = -INFINITY, ewlo = INFINITY, ewhi = -INFINITY;
    double max_rx = 0, max_rw = 0, max_erx = 0, max_erw = 0;
    for (int64_t i = 0; i < C; ++i) {
        float rx = xmax[i] - xmin[i];
        float rw = wmax[i] - wmin[i];
        float si = 1.0f;
        /* criterion 0: the channel ranges (Eq. 4-10).  criterion 1, for comparison: the largest
         * magnitudes, which is what the per-channel equalisation of Section 3.1 balances. */
        float cx = criterion ? fmaxf(fabsf(xmin[i]), fabsf(xmax[i])) : rx;
        float cw = criterion ? fmaxf(fabsf(wmin[i]), fabsf(wmax[i])) : rw;
        int ok = isfinite(rx) && isfinite(rw) && cx > 0.0f && cw > 0.0f && isfinite(cx) && isfinite(cw);
        if (ok) {
            double sd = (1.0 / (double)cw) * sqrt((double)cx * (double)cw);
            si = (float)sd;
            if (!(isfinite(si) && si > 0.0f) || !isfinite(1.0f / si)) {
                si = 1.0f;
                ok = 0;
            }
        }
        if (!ok)
            ++dead;
        s[i] = si;
        rinv[i] = 1.0f / si;
        mu_hat[i] = xmean[i] * rinv[i];
        if (xmin[i] < gxlo) gxlo = xmin[i];
        if (xmax[i] > gxhi) gxhi = xmax[i];
        if (wmin[i] < gwlo) gwlo = wmin[i];
        if (wmax[i] > gwhi) gwhi = wmax[i];
        /* the equalised tensors: channel i of X^ is X_i / s_i, of W^ is s_i W_i */
        double a = (double)(xmin[i] * rinv[i]), b = (double)(xmax[i] * rinv[i]);
        double c = (double)(wmin[i] * si), d = (double)(wmax[i] * si);
        if (a < exlo) exlo = a;
        if (b > exhi) exhi = b;
        if (c < ewlo) ewlo = c;
        if (d > ewhi) ewhi = d;
        if (rx > max_rx) max_rx = rx;
        if (rw > max_rw) max_rw = rw;
        if (b - a > max_erx) max_erx = b - a;
        if (d - c > max_erw) max_erw = d - c;
    }
    double RX = gxhi - gxlo, RW = gwhi - gwlo, EX = exhi - exlo, EW = ewhi - ewlo;
    double obj0 = 0.0, obj1 = 0.0;
    for (int64_t i = 0; i < C; ++i) {
        double rx = (double)(xmax[i] - xmin[i]);
        double rw = (double)(wmax[i] - wmin[i]);
        pX[i] = (float)(rx / RX);
        pW[i] = (float)(rw / RW);
        obj0 += (rx / RX) * (rw / RW);
        double erx = (double)(xmax[i] * rinv[i]) - (double)(xmin[i] * rinv[i]);
        double erw = (double)(wmax[i] * s[i]) - (double)(wmin[i] * s[i]);
        obj1 += (erx / EX) * (erw / EW);
    }
    if (scalars) {
        scalars[0] = RX; scalars[1] = RW; scalars[2] = EX; scalars[3] = EW;
        scalars[4] = obj0; scalars[5] = obj1;
        scalars[6] = max_rx * max_rw; scalars[7] = max_erx * max_erw;
    }
    return dead;
}

/* ------------------------------------------------------------------ */
/* The quantiser of Eq. 1-2 on one vector v[0..n).                      */
/*   Step = (v_max - v_min) / (2^b - 1)                        Eq. 2    */
/*   q    = clamp(round(v / Step) + Z, 0, 2^b - 1)             Eq. 1    */
/* with Z = -round(v_min / Step), so that v_min maps to code 0.         */
/* v / Step is evaluated as v * (1 / Step) with one correctly rounded   */
/* reciprocal per vector (literal_division != 0 divides instead; used   */
/* only to show how rarely the two differ).  round = ties to even.      */
/* ------------------------------------------------------------------ */
static int32_t saturate_i32(float r)
{
    if (isnan(r)) return 0;
    if (r >= 2147483648.0f) return INT32_MAX;
    if (r <= -2147483648.0f) return INT32_MIN;
    return (int32_t)r;
}

static void vector_step_zero(float lo, float hi, int bits, float *step, float *inv, int32_t *zp,
                             int literal_division)
{
    float qmax = (float)((1 << bits) - 1);
    float range = hi - lo;
    float st = range / qmax;
    if (!(st > 0.0f))                       /* constant vector */
        st = lo != 0.0f ? fabsf(lo) : 1.0f;
    float iv = 1.0f / st;
    float z = literal_division ? lo / st : lo * iv;
    *step = st;
    *inv = iv;
    *zp = saturate_i32(-nearbyintf(z));
}

static int32_t code_of(float v, float step, float inv, int32_t zp, int bits, int literal_division)
{
    float t = literal_division ? v / step : v * inv;
    int64_t q = (int64_t)saturate_i32(nearbyintf(t)) + (int64_t)zp;
    int64_t qmax = (1 << bits) - 1;
    if (q < 0) q = 0;
    if (q > qmax) q = qmax;
    return (int32_t)q;
}

void oracle_quantize_vector(const float *v, int64_t n, int bits, int literal_division,
                            float *step, int32_t *zp, int32_t *q)
{
    float lo = INFINITY, hi = -INFINITY, inv;
    for (int64_t i = 0; i < n; ++i) {
        if (v[i] < lo) lo = v[i];
        if (v[i] > hi) hi = v[i];
    }
    vector_step_zero(lo, hi, bits, step, &inv, zp, literal_division);
    for (int64_t i = 0; i < n; ++i)
        q[i] = code_of(v[i], *step, inv, *zp, bits, literal_division);
}

/* Code packing: 8-bit one per byte; 4-bit byte k = q[2k] | q[2k+1] << 4;
 * 3-bit: codes 8k..8k+7 form a 24-bit little-endian word, code i at bits
 * [3i, 3i+3).  General rule for all three: code i occupies bits
 * [i*b, (i+1)*b) of the little-endian bit stream of the row. */
static void put_code(uint8_t *row, int64_t i, int bits, int32_t q)
{
    int64_t bit = i * bits;
    for (int k = 0; k < bits; ++k, ++bit)
        if ((q >> k) & 1)
            row[bit >> 3] |= (uint8_t)(1u << (bit & 7));
}

static int32_t get_code(const uint8_t *row, int64_t i, int bits)
{
    int64_t bit = i * bits;
    int32_t q = 0;
    for (int k = 0; k < bits; ++k, ++bit)
        q |= ((row[bit >> 3] >> (bit & 7)) & 1) << k;
    return q;
}

void oracle_pack(const int32_t *q, int64_t rows, int64_t cols, int bits, uint8_t *out)
{
    int64_t pitch = cols * bits / 8;
    memset(out, 0, (size_t)(rows * pitch));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t i = 0; i < cols; ++i)
            put_code(out + r * pitch, i, bits, q[r * cols + i]);
}

void oracle_unpack(const uint8_t *in, int64_t rows, int64_t cols, int bits, int32_t *q)
{
    int64_t pitch = cols * bits / 8;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t i = 0; i < cols; ++i)
            q[r * cols + i] = get_code(in + r * pitch, i, bits);
}

/* ------------------------------------------------------------------ */
/* Step 4: fold s into W (Eq. 3: W^ = diag(s) W, i.e. input channel j   */
/* of every row is multiplied by s_j) and quantise W^ with Eq. 1-2,     */
/* one (Step, Z) per output row, per group of `group` consecutive input */
/* channels of a row, or per tensor.  s == NULL means no equalisation   */
/* (plain round-to-nearest baseline).                                   */
/* Outputs: packed codes [C_out x C_in*bits/8]; step/zp per row         */
/* ([C_out]), per group ([C_out x C_in/group]) or one pair; and, when   */
/* mu_hat is given, delta[o] = sum_j (W~[o,j] - W^[o,j]) * mu_hat[j]    */
/* in fp64 with W~ = Step * (q - Z) (the eps * E[x] of Eq. 15).         */
/* ------------------------------------------------------------------ */
void oracle_equalize_quantize(const uint16_t *W, int dtype, int64_t C_out, int64_t C_in, int64_t ld,
                              const float *s, const float *mu_hat, int bits, int gran, int64_t group,
                              int literal_division,
                              uint8_t *codes, float *step, int32_t *zp, double *delta)
{
    int64_t pitch = C_in * bits / 8;
    int64_t glen = gran == ORACLE_PER_GROUP ? group : C_in;
    int64_t ngroups = C_in / glen;
    float t_step = 0, t_inv = 0;
    int32_t t_zp = 0;
    if (gran == ORACLE_PER_TENSOR) {
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t o = 0; o < C_out; ++o)
            for (int64_t j = 0; j < C_in; ++j) {
                float w = decode16(W[o * ld + j], dtype);
                float wh = s ? w * s[j] : w;
                if (wh < lo) lo = wh;
                if (wh > hi) hi = wh;
            }
        vector_step_zero(lo, hi, bits, &t_step, &t_inv, &t_zp, literal_division);
        step[0] = t_step;
        zp[0] = t_zp;
    }
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < C_out; ++o) {
        float *wh = (float *)malloc(sizeof(float) * (size_t)C_in);
        uint8_t *row = codes + o * pitch;
        memset(row, 0, (size_t)pitch);
        for (int64_t j = 0; j < C_in; ++j) {
            float w = decode16(W[o * ld + j], dtype);
            wh[j] = s ? w * s[j] : w;           /* one binary32 multiply */
        }
        double acc = 0.0;
        for (int64_t g = 0; g < ngroups; ++g) {
            const float *v = wh + g * glen;
            float st, inv;
            int32_t z;
            if (gran == ORACLE_PER_TENSOR) {
                st = t_step; inv = t_inv; z = t_zp;
            } else {
                float lo = INFINITY, hi = -INFINITY;
                for (int64_t i = 0; i < glen; ++i) {
                    if (v[i] < lo) lo = v[i];
                    if (v[i] > hi) hi = v[i];
                }
                vector_step_zero(lo, hi, bits, &st, &inv, &z, literal_division);
                step[o * ngroups + g] = st;
                zp[o * ngroups + g] = z;
            }
            for (int64_t i = 0; i < glen; ++i) {
                int32_t q = code_of(v[i], st, inv, z, bits, literal_division);
                put_code(row, g * glen + i, bits, q);
                if (mu_hat) {
                    double wq = (double)st * (double)((int64_t)q - (int64_t)z);
                    acc += (wq - (double)v[i]) * (double)mu_hat[g * glen + i];
                }
            }
        }
        if (delta)
            delta[o] = mu_hat ? acc : 0.0;
        free(wh);
    }
}

/* Dequantise packed codes: W~[o,j] = Step * (q - Z), fp64. */
void oracle_dequantize(const uint8_t *codes, const float *step, const int32_t *zp,
                       int64_t rows, int64_t cols, int bits, int gran, int64_t group, double *out)
{
    int64_t pitch = cols * bits / 8;
    int64_t glen = gran == ORACLE_PER_GROUP ? group : cols;
    int64_t ngroups = cols / glen;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t j = 0; j < cols; ++j) {
            int64_t k = gran == ORACLE_PER_TENSOR ? 0 : r * ngroups + j / glen;
            int32_t q = get_code(codes + r * pitch, j, bits);
            out[r * cols + j] = (double)step[k] * (double)((int64_t)q - (int64_t)zp[k]);
        }
}

/* ------------------------------------------------------------------ */
/* Step 5: bias correction, Eq. 15 and the sentence after it: the       */
/* expected output error eps * E[x^] is subtracted, which for a linear  */
/* layer is a change of its bias: bias'[o] = bias[o] - delta[o].        */
/* bias_in == NULL means a layer without bias (zeros).  The result is   */
/* rounded once to binary32 and once to the 16-bit type.                */
/* ------------------------------------------------------------------ */
void oracle_bias_correct(const double *delta, const uint16_t *bias_in, int bias_dtype, int64_t C_out,
                         float *bias_f32, uint16_t *bias_16)
{
    for (int64_t o = 0; o < C_out; ++o) {
        double b = bias_in ? (double)decode16(bias_in[o], bias_dtype) : 0.0;
        double c = b - delta[o];
        bias_f32[o] = (float)c;
        bias_16[o] = encode16(c, bias_dtype);
    }
}

/* The same delta recomputed from stored codes (second route to Eq. 15):
 * delta[o] = sum_j (Step*(q - Z) - W[o,j]*s_j) * mu_hat[j]. */
void oracle_bias_delta_from_codes(const uint16_t *W, int dtype, int64_t C_out, int64_t C_in, int64_t ld,
                                  const float *s, const uint8_t *codes, const float *step,
                                  const int32_t *zp, const float *mu_hat, int bits, int gran,
                                  int64_t group, double *delta)
{
    int64_t pitch = C_in * bits / 8;
    int64_t glen = gran == ORACLE_PER_GROUP ? group : C_in;
    int64_t ngroups = C_in / glen;
    for (int64_t o = 0; o < C_out; ++o) {
        double acc = 0.0;
        for (int64_t j = 0; j < C_in; ++j) {
            int64_t k = gran == ORACLE_PER_TENSOR ? 0 : o * ngroups + j / glen;
            float w = decode16(W[o * ld + j], dtype);
            float wh = s ? w * s[j] : w;
            int32_t q = get_code(codes + o * pitch, j, bits);
            double wq = (double)step[k] * (double)((int64_t)q - (int64_t)zp[k]);
            acc += (wq - (double)wh) * (double)mu_hat[j];
        }
        delta[o] = acc;
    }
}

/* ------------------------------------------------------------------ */
/* Step 6: 8-bit quantisation of the equalised activations              */
/* X^ = X diag(s)^-1 (Eq. 3) with Eq. 1-2, one (Step, Z) per token row  */
/* or one pair for the whole tensor (lo_hi given: the static range).    */
/* rinv == NULL means no equalisation.                                  */
/* ------------------------------------------------------------------ */
void oracle_quant_act(const uint16_t *X, int dtype, int64_t N, int64_t C, int64_t ld,
                      const float *rinv, int gran, const float *lo_hi, int bits,
                      int literal_division, uint8_t *Xq, float *step, int32_t *zp)
{
    float t_step = 0, t_inv = 0;
    int32_t t_zp = 0;
    if (gran == ORACLE_PER_TENSOR) {
        vector_step_zero(lo_hi[0], lo_hi[1], bits, &t_step, &t_inv, &t_zp, literal_division);
        step[0] = t_step;
        zp[0] = t_zp;
    }
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        float *xh = (float *)malloc(sizeof(float) * (size_t)C);
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t j = 0; j < C; ++j) {
            float x = decode16(X[n * ld + j], dtype);
            xh[j] = rinv ? x * rinv[j] : x;
            if (xh[j] < lo) lo = xh[j];
            if (xh[j] > hi) hi = xh[j];
        }
        float st = t_step, inv = t_inv;
        int32_t z = t_zp;
        if (gran != ORACLE_PER_TENSOR) {
            vector_step_zero(lo, hi, bits, &st, &inv, &z, literal_division);
            step[n] = st;
            zp[n] = z;
        }
        for (int64_t j = 0; j < C; ++j)
            Xq[n * C + j] = (uint8_t)code_of(xh[j], st, inv, z, bits, literal_division);
        free(xh);
    }
}

/* ------------------------------------------------------------------ */
/* Forward check of a calibrated W8A8 layer.  Eq. 11 names the         */
/* expected output error E[y~_j - y_j] that quantisation leaves behind */
/* and that bias correction (Eq. 15) removes; this routine evaluates   */
/* it, and the output MSE, straight from the definitions, in fp64:     */
/*   y~[n,o] = sum_k Step^x_n (Xq[n,k]-Z^x_n) Step^w_o (Wq[o,k]-Z^w_o) */
/*             + bias_q[o]                 (Eq. 1-2 de-quantisation)   */
/*   y[n,o]  = sum_k X[n,k] W[o,k] + bias[o]   (the 16-bit layer; the  */
/*             product is unchanged by equalisation, Eq. 3)            */
/*   mean_err[o] = (1/N) sum_n (y~ - y),                               */
/*   sums = { sum (y~-y)^2, sum y^2, sum_o mean_err[o]^2, N*C_out }.   */
/* One byte per code; bias may be NULL (zeros); bias_q may be NULL:    */
/* the quantised layer then keeps bias (no correction applied).       */
/* ------------------------------------------------------------------ */
void oracle_forward_check(const uint8_t *Xq, const float *act_step, const int32_t *act_zp,
                          const uint8_t *Wq, const float *w_step, const int32_t *w_zp, const float *bias_q,
                          const uint16_t *X, const uint16_t *W, int dtype, const uint16_t *bias,
                          int64_t N, int64_t C_in, int64_t C_out, double *mean_err, double *sums)
{
    double *sq = (double *)calloc((size_t)C_out * 2, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < C_out; ++o) {
        double sd = 0.0, sd2 = 0.0, sy2 = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            double yq = 0.0, y = 0.0;
            for (int64_t k = 0; k < C_in; ++k) {
                double xq = (double)act_step[n] * (double)((int64_t)Xq[n * C_in + k] - (int64_t)act_zp[n]);
                double wq = (double)w_step[o] * (double)((int64_t)Wq[o * C_in + k] - (int64_t)w_zp[o]);
                yq += xq * wq;
                y += (double)decode16(X[n * C_in + k], dtype) * (double)decode16(W[o * C_in + k], dtype);
            }
            if (bias) y += (double)decode16(bias[o], dtype);
            if (bias_q) yq += (double)bias_q[o];
            else if (bias) yq += (double)decode16(bias[o], dtype);   /* uncorrected: the layer keeps its bias */
            double d = yq - y;
            sd += d;
            sd2 += d * d;
            sy2 += y * y;
        }
        mean_err[o] = sd / (double)N;
        sq[2 * o] = sd2;
        sq[2 * o + 1] = sy2;
    }
    sums[0] = sums[1] = sums[2] = 0.0;
    for (int64_t o = 0; o < C_out; ++o) {
        sums[0] += sq[2 * o];
        sums[1] += sq[2 * o + 1];
        sums[2] += mean_err[o] * mean_err[o];
    }
    sums[3] = (double)N * (double)C_out;
    free(sq);
}

/* ------------------------------------------------------------------ */
/* Folding diag(s)^-1 into the producer of a layer input (Section 3.1, */
/* after Eq. 3: X^ = X diag(s)^-1 is obtained by scaling what produces */
/* X -- row j of the previous linear layer and element j of its bias,  */
/* or the gain and shift of a normalisation layer -- by 1/s_j).        */
/*   out[r,c] = round16( (binary32) P[r,c] * rinv[r] )                 */
/* ------------------------------------------------------------------ */
void oracle_fold_scale(const uint16_t *P, int dtype, int64_t rows, int64_t cols, const float *rinv, uint16_t *out)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            volatile float prod = decode16(P[r * cols + c], dtype) * rinv[r];
            out[r * cols + c] = encode16((double)prod, dtype);
        }
}

/* ------------------------------------------------------------------ */
/* Forward check of a weight-only layer: Eq. 11 evaluated on data with */
/* 16-bit activations.  The equalised input is x^ = x * rinv (Eq. 3;   */
/* rinv is the binary32 1/s of step 3, NULL = ones) and the weights    */
/* are the de-quantised step-4 codes W~ = Step (q - Z) (Eq. 1-2), at   */
/* any bit-width and granularity:                                      */
/*   y~[n,o] = sum_j x^[n,j] W~[o,j] + bias_q[o]                       */
/*   y[n,o]  = sum_j X[n,j] W[o,j] + bias[o]                           */
/* Outputs as oracle_forward_check.  Everything in binary64.           */
/* ------------------------------------------------------------------ */
void oracle_forward_check_weights(const uint8_t *codes, const float *step, const int32_t *zp, int bits, int gran,
                                  int64_t group, const float *rinv, const float *bias_q, const uint16_t *X,
                                  const uint16_t *W, int dtype, const uint16_t *bias, int64_t N, int64_t C_in,
                                  int64_t C_out, double *mean_err, double *sums)
{
    int64_t pitch = C_in * bits / 8;
    int64_t glen = gran == ORACLE_PER_GROUP ? group : C_in;
    int64_t ngroups = C_in / glen;
    double *sq = (double *)calloc((size_t)C_out * 2, sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < C_out; ++o) {
        double *wq = (double *)malloc((size_t)C_in * sizeof(double));
        double *w = (double *)malloc((size_t)C_in * sizeof(double));
        for (int64_t j = 0; j < C_in; ++j) {
            int64_t k = gran == ORACLE_PER_TENSOR ? 0 : o * ngroups + j / glen;
            int32_t q = get_code(codes + o * pitch, j, bits);
            wq[j] = (double)step[k] * (double)((int64_t)q - (int64_t)zp[k]);
            w[j] = (double)decode16(W[o * C_in + j], dtype);
        }
        double sd = 0.0, sd2 = 0.0, sy2 = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            double yq = 0.0, y = 0.0;
            for (int64_t j = 0; j < C_in; ++j) {
                double x = (double)decode16(X[n * C_in + j], dtype);
                double xh = rinv ? x * (double)rinv[j] : x;
                yq += xh * wq[j];
                y += x * w[j];
            }
            if (bias) y += (double)decode16(bias[o], dtype);
            if (bias_q) yq += (double)bias_q[o];
            else if (bias) yq += (double)decode16(bias[o], dtype);
            double d = yq - y;
            sd += d;
            sd2 += d * d;
            sy2 += y * y;
        }
        mean_err[o] = sd / (double)N;
        sq[2 * o] = sd2;
        sq[2 * o + 1] = sy2;
        free(wq);
        free(w);
    }
    sums[0] = sums[1] = sums[2] = 0.0;
    for (int64_t o = 0; o < C_out; ++o) {
        sums[0] += sq[2 * o];
        sums[1] += sq[2 * o + 1];
        sums[2] += mean_err[o] * mean_err[o];
    }
    sums[3] = (double)N * (double)C_out;
    free(sq);
}

/* ------------------------------------------------------------------ */
/* Signed relabelling of 8-bit codes (Eq. 1 with the code range moved   */
/* from [0, 255] to [-128, 127]): q' = q - 128, Z' = Z - 128, so that   */
/* Step (q' - Z') = Step (q - Z).  Z' saturates to the int32 range like */
/* every zero-point here.  codes: n bytes; zp / zp_out: nz values or    */
/* NULL.                                                               */
/* ------------------------------------------------------------------ */
void oracle_relabel_signed(const uint8_t *codes, int64_t n, int8_t *out, const int32_t *zp, int64_t nz,
                           int32_t *zp_out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = (int8_t)((int)codes[i] - 128);
    if (zp && zp_out)
        for (int64_t k = 0; k < nz; ++k) {
            int64_t z = (int64_t)zp[k] - 128;
            if (z < (int64_t)INT32_MIN) z = (int64_t)INT32_MIN;
            zp_out[k] = (int32_t)z;
        }
}
