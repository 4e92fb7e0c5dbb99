// Eq. 1-2 quantiser with a per-column scale where the (Step, Z) pair belongs to
// a short group of consecutive columns or to the whole tensor:
//   - step 4 in per-group mode (W^ = diag(s) W, Eq. 3; one pair per `group`
//     consecutive input channels of a row -- the 4-bit / 3-bit, group-128 case),
//   - step 4 and step 6 in per-tensor mode (a static range given up front).
//
// A group of g columns is g/8 adjacent lanes of a warp, each holding one
// 16-byte vector, so the group extremes are a single redux.sync over a lane
// sub-mask and nothing has to be staged.  One warp walks one row, one vector
// per lane (256 columns) per step with the next step's load already in flight;
// many such warps per SM hide each other's latency (the kernel is bound by
// instruction issue, so every per-element instruction counts).
// The per-element work uses the packed binary32
// instructions of sm_100 (two multiplies / adds / FMAs per instruction):
// scale, multiply by 1/Step, add the rounding constant, and the three
// operations of the eps . E[x^] term of Eq. 15.  The upper clamp of Eq. 1 is
// decided once per group: it can only fire when rint(hi / Step) + Z exceeds
// 2^b - 1, which needs a rounding tie; such groups, and groups whose
// zero-point is too large for the add-constant rounding, take the literal
// cvt.rni path.  4-bit codes leave as one 32-bit word per lane, 3-bit codes are
// regrouped by four lanes into three 32-bit words with shuffles, so stores are
// coalesced.
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
    BiasIO bias;             // when out / out_f32 is set, the corrected bias is written with epsmu
    int bits;
    int lanes_per_group;        // group / 8 (group mode)
    int log2_lanes;             // log2 of it
    int ngroups;                // groups per row (group mode)
    const float *lo_hi;         // static mode: device float[2]
    aweq_dev_status *st;
};

constexpr int kWqWarps = 8;

// store the codes u[i] + K of one vector; BITS == 0 means "runtime bits"
template <int BITS, bool BYTES_OUT>
__device__ __forceinline__ void store_vec(unsigned char *orow, int idx, const uint32_t (&u)[8], uint32_t K, int bits,
                                          bool active, bool quad3, int lane)
{
    const int b = BITS ? BITS : bits;
    if (BYTES_OUT || b == 8) {
        const uint32_t kp = K * 0x01010101u;
        uint2 w;
        w.x = u[0] + (u[1] << 8) + (u[2] << 16) + (u[3] << 24) + kp;
        w.y = u[4] + (u[5] << 8) + (u[6] << 16) + (u[7] << 24) + kp;
        if (active) *reinterpret_cast<uint2 *>(orow + (size_t)idx * 8) = w;
    } else if (b <= 4) {
        uint32_t w = 0, m = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            w += u[e] << (e * b);
            m += 1u << (e * b);
        }
        w += K * m;
        if (b == 4) {
            if (active) *reinterpret_cast<uint32_t *>(orow + (size_t)idx * 4) = w;
        } else if (b == 2) {
            if (active) *reinterpret_cast<uint16_t *>(orow + (size_t)idx * 2) = (uint16_t)w;
        } else if (quad3) {
            // four lanes hold 4 x 24 bits = three 32-bit words (all lanes take part in the shuffle)
            w &= 0x00FFFFFFu;
            const int q4 = lane & 3;
            const uint32_t up = __shfl_down_sync(0xffffffffu, w, 1);
            uint32_t word;
            if (q4 == 0) word = w | (up << 24);
            else if (q4 == 1) word = (w >> 8) | (up << 16);
            else word = (w >> 16) | (up << 8);
            if (active && q4 < 3) *reinterpret_cast<uint32_t *>(orow + (size_t)(idx >> 2) * 12 + q4 * 4) = word;
        } else if (active) {
            unsigned char *d = orow + (size_t)idx * 3;
            d[0] = (unsigned char)w;
            d[1] = (unsigned char)(w >> 8);
            d[2] = (unsigned char)(w >> 16);
        }
    } else if (active) {
        unsigned long long w = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) w |= (unsigned long long)((u[e] + K) & ((1u << b) - 1u)) << (e * b);
        unsigned char *d = orow + (size_t)idx * b;
        for (int k = 0; k < b; ++k) d[k] = (unsigned char)(w >> (8 * k));
    }
}

// FULL: the row is a whole number of 32-vector steps, so no lane is ever past its end.
template <class D, int BITS, bool STATIC, bool MU, bool BYTES_OUT, bool FULL>
__global__ void __launch_bounds__(kWqWarps * 32, 4)
warpquant_kernel(const WarpQuantParams p)
{
    pdl_begin();
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * kWqWarps + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * kWqWarps;
    const int bits = BITS ? BITS : p.bits;
    const int qmax = (1 << bits) - 1;
    const int L = p.lanes_per_group;
    const uint32_t gmask = (STATIC || L >= 32) ? 0xffffffffu : (((1u << L) - 1u) << (lane & ~(L - 1)));
    const int nsteps = (p.nvec + 31) / 32;
    const bool quad3 = !BYTES_OUT && bits == 3 && (p.nvec % 4 == 0);
    const float2 magic2 = make_float2(kMagic, kMagic), nmagic2 = make_float2(-kMagic, -kMagic);
    const float2 one2 = make_float2(1.0f, 1.0f);

    QParams qs;
    int qs_flags = 0;
    if (STATIC) {
        qs = make_qparams(p.lo_hi[0], p.lo_hi[1], qmax);
        qs_flags = (qs.fast ? kQFast : 0) | kQNoClamp;    // the range is external: both clamps are applied explicitly
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            p.step[0] = qs.step;
            p.zp[0] = qs.zp;
        }
    }

    for (long long row = warp0; row < p.nrows; row += nwarps) {
        const uint16_t *xrow = p.X + row * p.ld;
        unsigned char *orow = p.out + row * p.out_pitch;
        float *step_row = STATIC ? p.step : p.step + row * p.ngroups;
        int *zp_row = STATIC ? p.zp : p.zp + row * p.ngroups;
        float2 eneg = make_float2(0.0f, 0.0f);                 // minus the running eps . mu sum
        uint4 nxt = (FULL || lane < p.nvec) ? ldg_stream(xrow + (size_t)lane * 8) : make_uint4(0, 0, 0, 0);
        float buf_step = 0.0f;                                 // (Step, Z) of the group whose index in the current
        int buf_zp = 0;                                        // window of 32 groups is this lane
        for (int it = 0; it < nsteps; ++it) {
            const int idx = it * 32 + lane;
            const bool active = FULL || idx < p.nvec;
            float w[8];
            widen8<D>(nxt, w);
            nxt = idx + 32 < p.nvec ? ldg_stream(xrow + (size_t)(idx + 32) * 8) : make_uint4(0, 0, 0, 0);
            float2 w2[4];
            if (p.scale && active) {
                const float4 s0 = ldg_f4(p.scale + (size_t)idx * 8), s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
                w2[0] = __fmul2_rn(make_float2(w[0], w[1]), make_float2(s0.x, s0.y));
                w2[1] = __fmul2_rn(make_float2(w[2], w[3]), make_float2(s0.z, s0.w));
                w2[2] = __fmul2_rn(make_float2(w[4], w[5]), make_float2(s1.x, s1.y));
                w2[3] = __fmul2_rn(make_float2(w[6], w[7]), make_float2(s1.z, s1.w));
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) w2[k] = make_float2(w[2 * k], w[2 * k + 1]);
            }
            float mu8[8];
            if (MU) {
                if (active) load8(p.mu + (size_t)idx * 8, mu8);
                else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) mu8[e] = 0.0f;
                }
            }
            QParams q;
            int fl;
            if (STATIC) {
                q = qs;
                fl = qs_flags;
            } else {
                float a = fmin3(w2[0].x, w2[0].y, w2[1].x), b = fmax3(w2[0].x, w2[0].y, w2[1].x);
                a = fmin3(a, w2[1].y, w2[2].x); b = fmax3(b, w2[1].y, w2[2].x);
                a = fmin3(a, w2[2].y, w2[3].x); b = fmax3(b, w2[2].y, w2[3].x);
                a = fminf(a, w2[3].y); b = fmaxf(b, w2[3].y);
                if (L == 16) {
                    // two groups per warp: a full-mask reduction per group with the other half's lanes
                    // neutral costs a third of what one reduction over a 16-lane sub-mask does (the two
                    // halves name different masks, which the hardware does not take in one go)
                    const bool upper = lane >= 16;
                    const float a0 = redux_min(upper ? INFINITY : a, 0xffffffffu);
                    const float a1 = redux_min(upper ? a : INFINITY, 0xffffffffu);
                    const float b0 = redux_max(upper ? -INFINITY : b, 0xffffffffu);
                    const float b1 = redux_max(upper ? b : -INFINITY, 0xffffffffu);
                    a = upper ? a1 : a0;
                    b = upper ? b1 : b0;
                } else if (L > 1) {
                    a = redux_min(a, gmask);
                    b = redux_max(b, gmask);
                }
                q = make_qparams(a, b, qmax);
                fl = qflags(q, b, qmax);
                // (Step, Z) pairs are collected in registers -- lane l keeps group l of the current window
                // of 32 groups, fetched from the first lane of that group in the step that formed it --
                // and leave as one coalesced store per window instead of a scattered one per step
                const int gps = 32 >> p.log2_lanes;                       // groups per step
                const int wpos = it & (L - 1);                            // step within the window (L steps)
                const int src = (lane & (gps - 1)) << p.log2_lanes;       // first lane of "my" group in its step
                const float sh_step = __shfl_sync(0xffffffffu, q.step, src);
                const int sh_zp = __shfl_sync(0xffffffffu, q.zp, src);
                if ((lane >> (5 - p.log2_lanes)) == wpos) {
                    buf_step = sh_step;
                    buf_zp = sh_zp;
                }
                if (wpos == L - 1 || it == nsteps - 1) {
                    const int g0 = (it - wpos) * gps;                     // first group of the window
                    if (g0 + lane < p.ngroups) {
                        step_row[g0 + lane] = buf_step;
                        zp_row[g0 + lane] = buf_zp;
                    }
                }
            }
            const bool all_lean = __all_sync(0xffffffffu, !active || fl == (kQFast | kQNoClamp));
            uint32_t u[8];
            uint32_t K;
            if (all_lean) {
                K = (uint32_t)(q.zp - kMagicBits);
                const float2 inv2 = make_float2(q.inv, q.inv);
                const float2 nstep2 = make_float2(-q.step, -q.step);
                const float hic = (float)(qmax - q.zp), loc = (float)(-q.zp);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    float2 t = __fmul2_rn(w2[k], inv2);
                    if (STATIC) {
                        t.x = fmaxf(fminf(t.x, hic), loc);
                        t.y = fmaxf(fminf(t.y, hic), loc);
                    }
                    // t * 1 + magic: the same value as t + magic, but as a single FMA that
                    // cannot be merged with the multiply that produced t (the assembler was
                    // seen to contract a packed multiply followed by a packed add, which
                    // changes the rounding at exact .5 ties)
                    const float2 uf = __ffma2_rn(t, one2, magic2);
                    u[2 * k] = __float_as_uint(uf.x);
                    u[2 * k + 1] = __float_as_uint(uf.y);
                    if (MU) {
                        const float2 rq = __fadd2_rn(uf, nmagic2);                 // q - Z, exact
                        const float2 neps = __ffma2_rn(nstep2, rq, w2[k]);         // -(Step (q - Z) - w^)
                        eneg = __ffma2_rn(neps, make_float2(mu8[2 * k], mu8[2 * k + 1]), eneg);
                    }
                }
            } else {
                K = 0u;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int c0 = code_generic(w2[k].x, q.inv, q.zp, qmax), c1 = code_generic(w2[k].y, q.inv, q.zp, qmax);
                    u[2 * k] = (uint32_t)c0;
                    u[2 * k + 1] = (uint32_t)c1;
                    if (MU) {
                        const float r0 = (float)((long long)c0 - (long long)q.zp), r1 = (float)((long long)c1 - (long long)q.zp);
                        eneg.x = __fmaf_rn(__fmaf_rn(-q.step, r0, w2[k].x), mu8[2 * k], eneg.x);
                        eneg.y = __fmaf_rn(__fmaf_rn(-q.step, r1, w2[k].y), mu8[2 * k + 1], eneg.y);
                    }
                }
            }
            store_vec<BITS, BYTES_OUT>(orow, idx, u, K, bits, active, quad3, lane);
        }
        if (MU) {
            const float tot = -warp_sum(__fadd_rn(eneg.x, eneg.y));
            if (lane == 0) {
                p.epsmu[row] = tot;
                if (p.bias.out || p.bias.out_f32) write_bias(row, tot, p.bias.in, p.bias.out, p.bias.out_f32, p.bias.bf16);
            }
        }
    }
}

// lo = min_j fl(cmin_j * scale_j), hi = max_j fl(cmax_j * scale_j): the extremes of
// the scaled tensor from its per-column extremes (scale_j > 0 keeps the order).
__global__ void scaled_tensor_range_kernel(const float *__restrict__ cmin, const float *__restrict__ cmax,
                                           const float *__restrict__ scale, int C, float *lo_hi)
{
    __shared__ float slo[32], shi[32];
    pdl_begin();
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
    AWEQ_LAUNCH(scaled_tensor_range_kernel, dim3(1), dim3(1024), 0, stream, cmin, cmax, scale, (int)C, lo_hi);
    return AWEQ_OK;
}

template <class D, int BITS, bool STATIC, bool MU, bool BYTES_OUT>
static aweq_status launch_wq(const WarpQuantParams &p, cudaStream_t stream)
{
    long long blocks = (p.nrows + kWqWarps - 1) / kWqWarps;
    const long long cap = (long long)kSmCount * 8 * 4;      // a few waves; warps stride over the rows beyond that
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (p.nvec % 32 == 0)
        AWEQ_LAUNCH((warpquant_kernel<D, BITS, STATIC, MU, BYTES_OUT, true>), dim3((unsigned)blocks), dim3(kWqWarps * 32),
                    0, stream, p);
    else
        AWEQ_LAUNCH((warpquant_kernel<D, BITS, STATIC, MU, BYTES_OUT, false>), dim3((unsigned)blocks),
                    dim3(kWqWarps * 32), 0, stream, p);
    return AWEQ_OK;
}

template <class D, bool STATIC, bool MU>
static aweq_status launch_wq_bits(const WarpQuantParams &p, cudaStream_t stream)
{
    switch (p.bits) {
    case 8: return launch_wq<D, 8, STATIC, MU, false>(p, stream);
    case 4: return launch_wq<D, 4, STATIC, MU, false>(p, stream);
    case 3: return launch_wq<D, 3, STATIC, MU, false>(p, stream);
    default: return launch_wq<D, 0, STATIC, MU, false>(p, stream);
    }
}

// group > 0: per-group mode; group == 0: static mode with lo_hi.
aweq_status run_warpquant(const void *X, aweq_dtype dt, long long nrows, long long cols, long long ld,
                          const float *scale, const float *mu, int bits, bool weights, int group,
                          const float *lo_hi, unsigned char *out, float *step, int *zp, float *epsmu,
                          const BiasIO &bias, aweq_dev_status *st, cudaStream_t stream)
{
    WarpQuantParams p;
    p.X = reinterpret_cast<const uint16_t *>(X);
    p.nrows = nrows; p.ld = ld; p.nvec = (int)(cols / 8);
    p.scale = scale; p.mu = mu; p.out = out;
    p.out_pitch = weights ? cols * bits / 8 : cols;
    p.step = step; p.zp = zp; p.epsmu = epsmu; p.bits = bits; p.bias = bias;
    p.lanes_per_group = group > 0 ? group / 8 : 32;
    p.log2_lanes = 0;
    while ((1 << p.log2_lanes) < p.lanes_per_group) ++p.log2_lanes;
    p.ngroups = group > 0 ? (int)(cols / group) : 1;
    p.lo_hi = lo_hi; p.st = st;
    const bool has_mu = weights && mu && epsmu;
    const bool is_static = group == 0;
#define AWEQ_WQ_GO(DT)                                                                        \
    if (!weights) return launch_wq<DT, 0, true, false, true>(p, stream);                      \
    if (is_static) return has_mu ? launch_wq_bits<DT, true, true>(p, stream)                  \
                                 : launch_wq_bits<DT, true, false>(p, stream);                \
    return has_mu ? launch_wq_bits<DT, false, true>(p, stream)                                \
                  : launch_wq_bits<DT, false, false>(p, stream);
    if (dt == AWEQ_F16) { AWEQ_WQ_GO(F16) }
    AWEQ_WQ_GO(BF16)
#undef AWEQ_WQ_GO
}

}  // namespace aweq
