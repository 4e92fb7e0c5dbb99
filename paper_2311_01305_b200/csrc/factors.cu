// Step 3: equalisation factors and the diagnostics of Eq. 4-8.
//
//   r^X_j = xmax_j - xmin_j, r^W_j = wmax_j - wmin_j            (Section 3.2)
//   s_j   = (1 / r^W_j) sqrt(r^X_j r^W_j)                        (Eq. 10, binary64, one rounding)
//   rinv_j = 1 / s_j,  mu_hat_j = xmean_j * rinv_j               (E[x^], Eq. 15)
//   p^X_j = r^X_j / R^X, p^W_j = r^W_j / R^W                     (Eq. 4)
//   objective sum_j p^X_j p^W_j before and after equalisation    (Eq. 5)
//   max_j r^X_j/s_j * max_k s_k r^W_k before and after           (Eq. 8)
// C_in values: one CTA, fixed reduction order, negligible time.
#include "common.cuh"

namespace aweq {

constexpr int kFacThreads = 1024;

struct FacRed {
    float xlo, xhi, wlo, whi, exlo, exhi, ewlo, ewhi, mrx, mrw, merx, merw;
};

__device__ __forceinline__ void fac_merge(FacRed &a, const FacRed &b)
{
    a.xlo = fminf(a.xlo, b.xlo); a.xhi = fmaxf(a.xhi, b.xhi);
    a.wlo = fminf(a.wlo, b.wlo); a.whi = fmaxf(a.whi, b.whi);
    a.exlo = fminf(a.exlo, b.exlo); a.exhi = fmaxf(a.exhi, b.exhi);
    a.ewlo = fminf(a.ewlo, b.ewlo); a.ewhi = fmaxf(a.ewhi, b.ewhi);
    a.mrx = fmaxf(a.mrx, b.mrx); a.mrw = fmaxf(a.mrw, b.mrw);
    a.merx = fmaxf(a.merx, b.merx); a.merw = fmaxf(a.merw, b.merw);
}

struct FacOut {
    float s, rinv, mu;
};

// one channel of pass 1: the factor, its reciprocal, E[x^], and the running extremes
__device__ __forceinline__ FacOut fac_channel(float lo, float hi, float mean, float wl, float wh, FacRed &a,
                                              unsigned int &dead, int criterion)
{
    const float rx = __fsub_rn(hi, lo), rw = __fsub_rn(wh, wl);
    // what Eq. 10 is fed: the channel ranges (the paper's criterion), or the largest magnitudes (the
    // criterion of the per-channel equalisation it starts from, Section 3.1) for comparison
    const float cx = criterion ? fmaxf(fabsf(lo), fabsf(hi)) : rx;
    const float cw = criterion ? fmaxf(fabsf(wl), fabsf(wh)) : rw;
    float sj = 1.0f;
    bool ok = isfinite(rx) && isfinite(rw) && cx > 0.0f && cw > 0.0f && isfinite(cx) && isfinite(cw);
    if (ok) {
        // Eq. 10 as printed, in binary64, rounded once to binary32
        sj = (float)__dmul_rn(__ddiv_rn(1.0, (double)cw), __dsqrt_rn(__dmul_rn((double)cx, (double)cw)));
        if (!(isfinite(sj) && sj > 0.0f) || !isfinite(__fdiv_rn(1.0f, sj))) {
            sj = 1.0f;
            ok = false;
        }
    }
    if (!ok) ++dead;
    const float ri = __fdiv_rn(1.0f, sj);
    const float exl = __fmul_rn(lo, ri), exh = __fmul_rn(hi, ri);
    const float ewl = __fmul_rn(wl, sj), ewh = __fmul_rn(wh, sj);
    a.xlo = fminf(a.xlo, lo); a.xhi = fmaxf(a.xhi, hi);
    a.wlo = fminf(a.wlo, wl); a.whi = fmaxf(a.whi, wh);
    a.exlo = fminf(a.exlo, exl); a.exhi = fmaxf(a.exhi, exh);
    a.ewlo = fminf(a.ewlo, ewl); a.ewhi = fmaxf(a.ewhi, ewh);
    a.mrx = fmaxf(a.mrx, rx); a.mrw = fmaxf(a.mrw, rw);
    a.merx = fmaxf(a.merx, exh - exl); a.merw = fmaxf(a.merw, ewh - ewl);
    FacOut o;
    o.s = sj; o.rinv = ri; o.mu = __fmul_rn(mean, ri);
    return o;
}

// one channel of pass 2: p^X, p^W and the two objective terms (reciprocals of the tensor ranges given)
__device__ __forceinline__ void fac_precision(float lo, float hi, float wl, float wh, float sj, float ri, double iRX,
                                              double iRW, double iEX, double iEW, float &px, float &pw, double &o0,
                                              double &o1)
{
    const double rx = (double)__fsub_rn(hi, lo), rw = (double)__fsub_rn(wh, wl);
    const double erx = (double)__fmul_rn(hi, ri) - (double)__fmul_rn(lo, ri);
    const double erw = (double)__fmul_rn(wh, sj) - (double)__fmul_rn(wl, sj);
    const double a = rx * iRX, b = rw * iRW;
    px = (float)a;
    pw = (float)b;
    o0 += a * b;
    o1 += (erx * iEX) * (erw * iEW);
}

__global__ void __launch_bounds__(kFacThreads)
factors_kernel(const float *__restrict__ xmin, const float *__restrict__ xmax, const float *__restrict__ xmean,
               const float *__restrict__ wmin, const float *__restrict__ wmax, int C, float *__restrict__ s,
               float *__restrict__ rinv, float *__restrict__ mu_hat, float *__restrict__ pX, float *__restrict__ pW,
               double *__restrict__ scalars, aweq_dev_status *st, int criterion)
{
    __shared__ FacRed red[kFacThreads / 32];
    __shared__ FacRed total;
    __shared__ double dsum[2][kFacThreads / 32];
    __shared__ unsigned int dead_count;
    if (threadIdx.x == 0) dead_count = 0;
    pdl_begin();
    __syncthreads();

    // four channels per thread and step (128-bit loads) when the arrays allow it
    const bool vec4 = ((reinterpret_cast<uintptr_t>(xmin) | reinterpret_cast<uintptr_t>(xmax) |
                        reinterpret_cast<uintptr_t>(xmean) | reinterpret_cast<uintptr_t>(wmin) |
                        reinterpret_cast<uintptr_t>(wmax) | reinterpret_cast<uintptr_t>(s) |
                        reinterpret_cast<uintptr_t>(rinv) | reinterpret_cast<uintptr_t>(mu_hat) |
                        reinterpret_cast<uintptr_t>(pX) | reinterpret_cast<uintptr_t>(pW)) & 15) == 0;
    const int nquad = vec4 ? C / 4 : 0;

    FacRed a;
    a.xlo = a.wlo = a.exlo = a.ewlo = INFINITY;
    a.xhi = a.whi = a.exhi = a.ewhi = -INFINITY;
    a.mrx = a.mrw = a.merx = a.merw = 0.0f;
    unsigned int dead = 0;
    for (int q = threadIdx.x; q < nquad; q += kFacThreads) {
        const float4 lo = ldg_f4(xmin + 4 * q), hi = ldg_f4(xmax + 4 * q), me = ldg_f4(xmean + 4 * q);
        const float4 wl = ldg_f4(wmin + 4 * q), wh = ldg_f4(wmax + 4 * q);
        const FacOut o0 = fac_channel(lo.x, hi.x, me.x, wl.x, wh.x, a, dead, criterion);
        const FacOut o1 = fac_channel(lo.y, hi.y, me.y, wl.y, wh.y, a, dead, criterion);
        const FacOut o2 = fac_channel(lo.z, hi.z, me.z, wl.z, wh.z, a, dead, criterion);
        const FacOut o3 = fac_channel(lo.w, hi.w, me.w, wl.w, wh.w, a, dead, criterion);
        *reinterpret_cast<float4 *>(s + 4 * q) = make_float4(o0.s, o1.s, o2.s, o3.s);
        *reinterpret_cast<float4 *>(rinv + 4 * q) = make_float4(o0.rinv, o1.rinv, o2.rinv, o3.rinv);
        *reinterpret_cast<float4 *>(mu_hat + 4 * q) = make_float4(o0.mu, o1.mu, o2.mu, o3.mu);
    }
    for (int j = 4 * nquad + threadIdx.x; j < C; j += kFacThreads) {
        const FacOut o = fac_channel(xmin[j], xmax[j], xmean[j], wmin[j], wmax[j], a, dead, criterion);
        s[j] = o.s;
        rinv[j] = o.rinv;
        mu_hat[j] = o.mu;
    }
    // block reduction of the twelve extremes
    const uint32_t full = 0xffffffffu;
    a.xlo = redux_min(a.xlo, full); a.xhi = redux_max(a.xhi, full);
    a.wlo = redux_min(a.wlo, full); a.whi = redux_max(a.whi, full);
    a.exlo = redux_min(a.exlo, full); a.exhi = redux_max(a.exhi, full);
    a.ewlo = redux_min(a.ewlo, full); a.ewhi = redux_max(a.ewhi, full);
    a.mrx = redux_max(a.mrx, full); a.mrw = redux_max(a.mrw, full);
    a.merx = redux_max(a.merx, full); a.merw = redux_max(a.merw, full);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    if (dead) atomicAdd(&dead_count, dead);
    __syncthreads();
    if (threadIdx.x == 0) {
        FacRed t = red[0];
        for (int k = 1; k < kFacThreads / 32; ++k) fac_merge(t, red[k]);
        total = t;
        if (st && dead_count) atomicAdd(&st->zero_range, (unsigned long long)dead_count);
    }
    if (!pX && !pW && !scalars) return;
    __syncthreads();
    const FacRed t = total;
    const double RX = (double)t.xhi - (double)t.xlo, RW = (double)t.whi - (double)t.wlo;
    const double EX = (double)t.exhi - (double)t.exlo, EW = (double)t.ewhi - (double)t.ewlo;
    const double iRX = 1.0 / RX, iRW = 1.0 / RW, iEX = 1.0 / EX, iEW = 1.0 / EW;

    double o0 = 0.0, o1 = 0.0;
    for (int q = threadIdx.x; q < nquad; q += kFacThreads) {
        const float4 lo = ldg_f4(xmin + 4 * q), hi = ldg_f4(xmax + 4 * q);
        const float4 wl = ldg_f4(wmin + 4 * q), wh = ldg_f4(wmax + 4 * q);
        const float4 sj = *reinterpret_cast<const float4 *>(s + 4 * q), ri = *reinterpret_cast<const float4 *>(rinv + 4 * q);
        float4 px, pw;
        fac_precision(lo.x, hi.x, wl.x, wh.x, sj.x, ri.x, iRX, iRW, iEX, iEW, px.x, pw.x, o0, o1);
        fac_precision(lo.y, hi.y, wl.y, wh.y, sj.y, ri.y, iRX, iRW, iEX, iEW, px.y, pw.y, o0, o1);
        fac_precision(lo.z, hi.z, wl.z, wh.z, sj.z, ri.z, iRX, iRW, iEX, iEW, px.z, pw.z, o0, o1);
        fac_precision(lo.w, hi.w, wl.w, wh.w, sj.w, ri.w, iRX, iRW, iEX, iEW, px.w, pw.w, o0, o1);
        if (pX) *reinterpret_cast<float4 *>(pX + 4 * q) = px;
        if (pW) *reinterpret_cast<float4 *>(pW + 4 * q) = pw;
    }
    for (int j = 4 * nquad + threadIdx.x; j < C; j += kFacThreads) {
        float px, pw;
        fac_precision(xmin[j], xmax[j], wmin[j], wmax[j], s[j], rinv[j], iRX, iRW, iEX, iEW, px, pw, o0, o1);
        if (pX) pX[j] = px;
        if (pW) pW[j] = pw;
    }
    if (scalars) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            o0 += __shfl_xor_sync(full, o0, o);
            o1 += __shfl_xor_sync(full, o1, o);
        }
        if ((threadIdx.x & 31) == 0) {
            dsum[0][threadIdx.x >> 5] = o0;
            dsum[1][threadIdx.x >> 5] = o1;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            double b0 = 0.0, b1 = 0.0;
            for (int k = 0; k < kFacThreads / 32; ++k) {
                b0 += dsum[0][k];
                b1 += dsum[1][k];
            }
            scalars[0] = RX; scalars[1] = RW; scalars[2] = EX; scalars[3] = EW;
            scalars[4] = b0; scalars[5] = b1;
            scalars[6] = (double)t.mrx * (double)t.mrw;
            scalars[7] = (double)t.merx * (double)t.merw;
        }
    }
}

aweq_status run_factors(const float *xmin, const float *xmax, const float *xmean, const float *wmin,
                        const float *wmax, long long C, float *s, float *rinv, float *mu_hat, float *pX, float *pW,
                        double *scalars, aweq_dev_status *st, cudaStream_t stream, int criterion)
{
    AWEQ_LAUNCH(factors_kernel, dim3(1), dim3(kFacThreads), 0, stream, xmin, xmax, xmean, wmin, wmax, (int)C, s, rinv,
                mu_hat, pX, pW, scalars, st, criterion);
    return AWEQ_OK;
}

}  // namespace aweq
