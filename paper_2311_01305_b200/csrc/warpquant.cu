// Eq. 1-2 quantiser with a per-column scale where the (Step, Z) pair belongs to
// a short group of consecutive columns or to the whole tensor:
//   - step 4 in per-group mode (W^ = diag(s) W, Eq. 3; one pair per `group`
//     consecutive input channels of a row -- the 4-bit / 3-bit, group-128 case),
//   - step 4 and step 6 in per-tensor mode (a static range given up front).
//
// A group of g columns is g/8 adjacent lanes of a warp, each holding one
// 16-byte vector, so the group extremes are a single redux.sync over a lane
// sub-mask and nothing has to be staged: one warp walks one row, 32 vectors per
// step, with the next step's vectors already in flight.  Scale, quantise and
// pack are fused; 4-bit codes leave as one 32-bit word per lane, 3-bit codes are
// regrouped by four lanes into three 32-bit words with shuffles, so all stores
// are coalesced.  The optional eps.E[x^] row sum of Eq. 15 is accumulated per
// lane in binary32 and reduced over the warp in a fixed order.
#include "common.cuh"

namespace aweq {

struct WarpQuantParams {
    const uint16_t *X;
    long long nrows, ld;
    int nvec;
    const float *scale;
    const float *mu;
    unsigned char *out;
    long long out_pitch;
    float *step;
    int *zp;
    float *epsmu;
    int bits;
    int lanes_per_group;        // group / 8 (group mode)
    int ngroups;                // groups per row (group mode)
    const float *lo_hi;         // static mode: device float[2]
    aweq_dev_status *st;
};

constexpr int kWqWarps = 8;

template <class D, bool STATIC, bool MU, bool BYTES_OUT>
__global__ void __launch_bounds__(kWqWarps * 32)
warpquant_kernel(const WarpQuantParams p)
{
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * kWqWarps + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * kWqWarps;
    const int qmax = (1 << p.bits) - 1;
    const int L = p.lanes_per_group;
    const uint32_t gmask = STATIC ? 0xffffffffu
                                  : (L >= 32 ? 0xffffffffu : (((1u << L) - 1u) << (lane & ~(L - 1))));
    const int niter = (p.nvec + 31) / 32;
    const bool quad3 = !BYTES_OUT && p.bits == 3 && (p.nvec % 4 == 0);
    const int vec_bytes = BYTES_OUT ? 8 : p.bits;

    QParams qs;
    if (STATIC) {
        qs = make_qparams(p.lo_hi[0], p.lo_hi[1], qmax);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            p.step[0] = qs.step;
            p.zp[0] = qs.zp;
        }
    }

    for (long long row = warp0; row < p.nrows; row += nwarps) {
        const uint16_t *xrow = p.X + row * p.ld;
        unsigned char *orow = p.out + row * p.out_pitch;
        float eacc = 0.0f;
        uint4 nxt = make_uint4(0, 0, 0, 0);
        if (lane < p.nvec) nxt = ldg_stream(xrow + (size_t)lane * 8);
        for (int it = 0; it < niter; ++it) {
            const int idx = it * 32 + lane;
            const bool active = idx < p.nvec;
            const uint4 raw = nxt;
            if (idx + 32 < p.nvec) nxt = ldg_stream(xrow + (size_t)(idx + 32) * 8);
            const uint32_t amask = __ballot_sync(0xffffffffu, active);
            if (active) {
                float v[8];
                widen8<D>(raw, v);
                if (p.scale) {
                    float sc[8];
                    load8(p.scale + (size_t)idx * 8, sc);
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = __fmul_rn(v[e], sc[e]);
                }
                QParams q;
                if (STATIC) {
                    q = qs;
                } else {
                    float lo = v[0], hi = v[0];
#pragma unroll
                    for (int e = 1; e < 8; ++e) {
                        lo = fminf(lo, v[e]);
                        hi = fmaxf(hi, v[e]);
                    }
                    if (L > 1) {
                        lo = redux_min(lo, gmask);
                        hi = redux_max(hi, gmask);
                    }
                    q = make_qparams(lo, hi, qmax);
                    if ((lane & (L - 1)) == 0) {
                        const long long g = row * p.ngroups + idx / L;
                        p.step[g] = q.step;
                        p.zp[g] = q.zp;
                    }
                }
                uint32_t u[8];
                uint32_t K;
                float mu8[8];
                if (MU) load8(p.mu + (size_t)idx * 8, mu8);
                if (q.fast) {
                    const float hic = (float)(qmax - q.zp);
                    const float loc = (float)(-q.zp);
                    K = (uint32_t)(q.zp - kMagicBits);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        float t = fminf(__fmul_rn(v[e], q.inv), hic);
                        if (STATIC) t = fmaxf(t, loc);
                        const float uf = __fadd_rn(t, kMagic);
                        u[e] = __float_as_uint(uf);
                        if (MU) {
                            const float rq = __fsub_rn(uf, kMagic);
                            const float eps = __fmaf_rn(q.step, rq, -v[e]);
                            eacc = __fmaf_rn(eps, mu8[e], eacc);
                        }
                    }
                } else {
                    K = 0u;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int c = code_generic(v[e], q.inv, q.zp, qmax);
                        u[e] = (uint32_t)c;
                        if (MU) {
                            const float rq = (float)((long long)c - (long long)q.zp);
                            const float eps = __fmaf_rn(q.step, rq, -v[e]);
                            eacc = __fmaf_rn(eps, mu8[e], eacc);
                        }
                    }
                }
                if (BYTES_OUT || p.bits == 8) {
                    const uint32_t kp = K * 0x01010101u;
                    uint2 w;
                    w.x = u[0] + (u[1] << 8) + (u[2] << 16) + (u[3] << 24) + kp;
                    w.y = u[4] + (u[5] << 8) + (u[6] << 16) + (u[7] << 24) + kp;
                    *reinterpret_cast<uint2 *>(orow + (size_t)idx * 8) = w;
                } else if (p.bits <= 4) {
                    uint32_t w = 0, m = 0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        w += u[e] << (e * p.bits);
                        m += 1u << (e * p.bits);
                    }
                    w += K * m;
                    if (p.bits == 4) {
                        *reinterpret_cast<uint32_t *>(orow + (size_t)idx * 4) = w;
                    } else if (p.bits == 2) {
                        *reinterpret_cast<uint16_t *>(orow + (size_t)idx * 2) = (uint16_t)w;
                    } else if (quad3) {
                        // four lanes hold 4 x 24 bits = three 32-bit words
                        w &= 0x00FFFFFFu;
                        const int q4 = lane & 3;
                        const uint32_t up = __shfl_down_sync(amask, w, 1);       // next lane's 24 bits
                        uint32_t word;
                        if (q4 == 0) word = w | (up << 24);
                        else if (q4 == 1) word = (w >> 8) | (up << 16);
                        else word = (w >> 16) | (up << 8);
                        if (q4 < 3)
                            *reinterpret_cast<uint32_t *>(orow + (size_t)(idx >> 2) * 12 + q4 * 4) = word;
                    } else {
                        unsigned char *d = orow + (size_t)idx * 3;
                        d[0] = (unsigned char)w;
                        d[1] = (unsigned char)(w >> 8);
                        d[2] = (unsigned char)(w >> 16);
                    }
                } else {
                    unsigned long long w = 0;
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        w |= (unsigned long long)((u[e] + K) & (uint32_t)qmax) << (e * p.bits);
                    unsigned char *d = orow + (size_t)idx * vec_bytes;
                    for (int k = 0; k < p.bits; ++k) d[k] = (unsigned char)(w >> (8 * k));
                }
            }
        }
        if (MU) {
            eacc = warp_sum(eacc);
            if (lane == 0) p.epsmu[row] = eacc;
        }
    }
}

// lo = min_j fl(cmin_j * scale_j), hi = max_j fl(cmax_j * scale_j): the extremes of
// the scaled tensor from its per-column extremes (scale_j > 0 keeps the order).
__global__ void scaled_tensor_range_kernel(const float *__restrict__ cmin, const float *__restrict__ cmax,
                                           const float *__restrict__ scale, int C, float *lo_hi)
{
    __shared__ float slo[32], shi[32];
    float lo = INFINITY, hi = -INFINITY;
    for (int j = threadIdx.x; j < C; j += blockDim.x) {
        const float sc = scale ? scale[j] : 1.0f;
        lo = fminf(lo, __fmul_rn(cmin[j], sc));
        hi = fmaxf(hi, __fmul_rn(cmax[j], sc));
    }
    lo = redux_min(lo, 0xffffffffu);
    hi = redux_max(hi, 0xffffffffu);
    if ((threadIdx.x & 31) == 0) {
        slo[threadIdx.x >> 5] = lo;
        shi[threadIdx.x >> 5] = hi;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int k = 1; k < (int)(blockDim.x >> 5); ++k) {
            lo = fminf(lo, slo[k]);
            hi = fmaxf(hi, shi[k]);
        }
        lo_hi[0] = lo;
        lo_hi[1] = hi;
    }
}

aweq_status run_scaled_tensor_range(const float *cmin, const float *cmax, const float *scale, long long C,
                                    float *lo_hi, cudaStream_t stream)
{
    scaled_tensor_range_kernel<<<1, 1024, 0, stream>>>(cmin, cmax, scale, (int)C, lo_hi);
    AWEQ_LAUNCH_CHECK();
    return AWEQ_OK;
}

template <class D, bool STATIC, bool MU, bool BYTES_OUT>
static aweq_status launch_wq(const WarpQuantParams &p, cudaStream_t stream)
{
    long long blocks = (p.nrows + kWqWarps - 1) / kWqWarps;
    const long long cap = (long long)kSmCount * 8 * 4;      // a few waves; warps stride over the rows beyond that
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    warpquant_kernel<D, STATIC, MU, BYTES_OUT><<<(unsigned)blocks, kWqWarps * 32, 0, stream>>>(p);
    AWEQ_LAUNCH_CHECK();
    return AWEQ_OK;
}

// group > 0: per-group mode; group == 0: static mode with lo_hi.
aweq_status run_warpquant(const void *X, aweq_dtype dt, long long nrows, long long cols, long long ld,
                          const float *scale, const float *mu, int bits, bool weights, int group,
                          const float *lo_hi, unsigned char *out, float *step, int *zp, float *epsmu,
                          aweq_dev_status *st, cudaStream_t stream)
{
    WarpQuantParams p;
    p.X = reinterpret_cast<const uint16_t *>(X);
    p.nrows = nrows; p.ld = ld; p.nvec = (int)(cols / 8);
    p.scale = scale; p.mu = mu; p.out = out;
    p.out_pitch = weights ? cols * bits / 8 : cols;
    p.step = step; p.zp = zp; p.epsmu = epsmu; p.bits = bits;
    p.lanes_per_group = group > 0 ? group / 8 : 32;
    p.ngroups = group > 0 ? (int)(cols / group) : 1;
    p.lo_hi = lo_hi; p.st = st;
    const bool has_mu = weights && mu && epsmu;
    const bool is_static = group == 0;
#define AWEQ_WQ_GO(DT)                                                                   \
    if (!weights) return is_static ? launch_wq<DT, true, false, true>(p, stream)         \
                                   : launch_wq<DT, false, false, true>(p, stream);       \
    if (is_static) return has_mu ? launch_wq<DT, true, true, false>(p, stream)           \
                                 : launch_wq<DT, true, false, false>(p, stream);         \
    return has_mu ? launch_wq<DT, false, true, false>(p, stream)                         \
                  : launch_wq<DT, false, false, false>(p, stream);
    if (dt == AWEQ_F16) { AWEQ_WQ_GO(F16) }
    AWEQ_WQ_GO(BF16)
#undef AWEQ_WQ_GO
}

}  // namespace aweq
