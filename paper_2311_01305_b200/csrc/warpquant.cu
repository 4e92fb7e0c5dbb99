// Eq. 1-2 quantiser with a per-column scale where the (Step, Z) pair belongs to
// a short group of consecutive columns or to the whole tensor:
//   - step 4 in per-group mode (W^ = diag(s) W, Eq. 3; one pair per `group`
//     consecutive input channels of a row -- the 4-bit / 3-bit, group-128 case),
//   - step 4 and step 6 in per-tensor mode (a static range given up front).
//
// A group of g columns is g/8 adjacent lanes of a warp, each holding one
// 16-byte vector, so the group extremes are a single redux.sync over a lane
// sub-mask and nothing has to be staged.  One warp walks one row, two vectors
// per lane (512 columns, one 32-byte load) per step with the next step's load already in flight;
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

// 32-byte read-once load (two consecutive vectors of one lane)
__device__ __forceinline__ void ldg_stream32(const void *p, uint4 &a, uint4 &b)
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}

// The codes u[h][i] + K of the VPL vectors of a lane, stored as one access where the layout
// allows it (VPL == 2: 16 codes = 16 / 8 / 6 bytes for 8 / 4 / 3 bits).
template <int BITS, bool BYTES_OUT, int VPL>
__device__ __forceinline__ void store_lane(unsigned char *orow, int idxl, const uint32_t (&u)[VPL][8], uint32_t K,
                                           int bits, bool active, bool quad3, bool pair3, int lane)
{
    if (VPL == 1) {
        store_vec<BITS, BYTES_OUT>(orow, idxl, u[0], K, bits, active, quad3, lane);
        return;
    }
    const int b = BITS ? BITS : bits;
    if (BYTES_OUT || b == 8) {
        const uint32_t kp = K * 0x01010101u;
        uint4 w;
        w.x = u[0][0] + (u[0][1] << 8) + (u[0][2] << 16) + (u[0][3] << 24) + kp;
        w.y = u[0][4] + (u[0][5] << 8) + (u[0][6] << 16) + (u[0][7] << 24) + kp;
        w.z = u[VPL - 1][0] + (u[VPL - 1][1] << 8) + (u[VPL - 1][2] << 16) + (u[VPL - 1][3] << 24) + kp;
        w.w = u[VPL - 1][4] + (u[VPL - 1][5] << 8) + (u[VPL - 1][6] << 16) + (u[VPL - 1][7] << 24) + kp;
        if (active) *reinterpret_cast<uint4 *>(orow + (size_t)idxl * 16) = w;
    } else if (b == 4) {
        uint2 w;
        w.x = K * 0x11111111u;
        w.y = w.x;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            w.x += u[0][e] << (4 * e);
            w.y += u[VPL - 1][e] << (4 * e);
        }
        if (active) *reinterpret_cast<uint2 *>(orow + (size_t)idxl * 8) = w;
    } else if (b == 3 && pair3) {
        // 48 bits per lane; two lanes hold three 32-bit words (all lanes take part in the shuffle)
        uint32_t wa = K * 0x249249u, wb = wa;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            wa += u[0][e] << (3 * e);
            wb += u[VPL - 1][e] << (3 * e);
        }
        wa &= 0x00FFFFFFu;
        wb &= 0x00FFFFFFu;
        const uint32_t lo32 = wa | (wb << 24), hi16 = wb >> 8;
        const uint32_t nlo = __shfl_down_sync(0xffffffffu, lo32, 1);       // the odd lane's low word
        uint32_t *dst = reinterpret_cast<uint32_t *>(orow + (size_t)(idxl >> 1) * 12);
        if (active) {
            if ((lane & 1) == 0) {
                dst[0] = lo32;
                dst[1] = hi16 | (nlo << 16);
            } else {
                dst[2] = (lo32 >> 16) | (hi16 << 16);
            }
        }
    } else {
#pragma unroll
        for (int h = 0; h < VPL; ++h) store_vec<BITS, BYTES_OUT>(orow, idxl * VPL + h, u[h], K, bits, active, false, lane);
    }
}

// VPL: 16-byte vectors per lane and step.  Two when the group holds at least 16 columns and
// the row an even number of vectors: the per-group work (Step, 1/Step, Z, their stores) is
// then spread over 16 elements per lane instead of 8.
template <class D, int BITS, bool STATIC, bool MU, bool BYTES_OUT, int VPL>
__global__ void __launch_bounds__(kWqWarps * 32, VPL == 1 ? 4 : 3)
warpquant_kernel(const WarpQuantParams p)
{
    const int lane = threadIdx.x & 31;
    const long long warp0 = (long long)blockIdx.x * kWqWarps + (threadIdx.x >> 5);
    const long long nwarps = (long long)gridDim.x * kWqWarps;
    const int bits = BITS ? BITS : p.bits;
    const int qmax = (1 << bits) - 1;
    const int L = VPL == 1 ? p.lanes_per_group : max(p.lanes_per_group / VPL, 1);   // lanes per group
    const int log2L = VPL == 1 ? p.log2_lanes : max(p.log2_lanes - 1, 0);
    const uint32_t gmask = (STATIC || L >= 32) ? 0xffffffffu : (((1u << L) - 1u) << (lane & ~(L - 1)));
    const int nlv = p.nvec / VPL;                        // lane-vectors per row
    const int nsteps = (nlv + 31) / 32;
    const bool quad3 = !BYTES_OUT && bits == 3 && VPL == 1 && (p.nvec % 4 == 0);
    const bool pair3 = !BYTES_OUT && bits == 3 && VPL == 2 && (p.nvec % 4 == 0);
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
        uint4 nxt[VPL];
#pragma unroll
        for (int h = 0; h < VPL; ++h) nxt[h] = make_uint4(0, 0, 0, 0);
        if (lane < nlv) {
            if (VPL == 2) ldg_stream32(xrow + (size_t)lane * 16, nxt[0], nxt[VPL - 1]);
            else nxt[0] = ldg_stream(xrow + (size_t)lane * 8);
        }
        for (int it = 0; it < nsteps; ++it) {
            const int idxl = it * 32 + lane;                   // lane-vector index
            const bool active = idxl < nlv;
            float2 w2[VPL][4];
#pragma unroll
            for (int h = 0; h < VPL; ++h) {
                float w[8];
                widen8<D>(nxt[h], w);
#pragma unroll
                for (int k = 0; k < 4; ++k) w2[h][k] = make_float2(w[2 * k], w[2 * k + 1]);
            }
#pragma unroll
            for (int h = 0; h < VPL; ++h) nxt[h] = make_uint4(0, 0, 0, 0);
            if (idxl + 32 < nlv) {
                if (VPL == 2) ldg_stream32(xrow + (size_t)(idxl + 32) * 16, nxt[0], nxt[VPL - 1]);
                else nxt[0] = ldg_stream(xrow + (size_t)(idxl + 32) * 8);
            }
            float mu8[VPL][8];
#pragma unroll
            for (int h = 0; h < VPL; ++h) {
                const size_t e0 = ((size_t)idxl * VPL + h) * 8;
                if (p.scale && active) {
                    const float4 s0 = ldg_f4(p.scale + e0), s1 = ldg_f4(p.scale + e0 + 4);
                    w2[h][0] = __fmul2_rn(w2[h][0], make_float2(s0.x, s0.y));
                    w2[h][1] = __fmul2_rn(w2[h][1], make_float2(s0.z, s0.w));
                    w2[h][2] = __fmul2_rn(w2[h][2], make_float2(s1.x, s1.y));
                    w2[h][3] = __fmul2_rn(w2[h][3], make_float2(s1.z, s1.w));
                }
                if (MU) {
                    if (active) load8(p.mu + e0, mu8[h]);
                    else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) mu8[h][e] = 0.0f;
                    }
                }
            }
            QParams q;
            int fl;
            if (STATIC) {
                q = qs;
                fl = qs_flags;
            } else {
                float a = INFINITY, b = -INFINITY;
#pragma unroll
                for (int h = 0; h < VPL; ++h) {
                    a = fminf(fminf(a, w2[h][0].x), w2[h][0].y); b = fmaxf(fmaxf(b, w2[h][0].x), w2[h][0].y);
                    a = fminf(fminf(a, w2[h][1].x), w2[h][1].y); b = fmaxf(fmaxf(b, w2[h][1].x), w2[h][1].y);
                    a = fminf(fminf(a, w2[h][2].x), w2[h][2].y); b = fmaxf(fmaxf(b, w2[h][2].x), w2[h][2].y);
                    a = fminf(fminf(a, w2[h][3].x), w2[h][3].y); b = fmaxf(fmaxf(b, w2[h][3].x), w2[h][3].y);
                }
                if (L > 1) {
                    a = redux_min(a, gmask);
                    b = redux_max(b, gmask);
                }
                q = make_qparams(a, b, qmax);
                fl = qflags(q, b, qmax);
                if (active && (lane & (L - 1)) == 0) {
                    step_row[idxl >> log2L] = q.step;
                    zp_row[idxl >> log2L] = q.zp;
                }
            }
            const bool all_lean = __all_sync(0xffffffffu, !active || fl == (kQFast | kQNoClamp));
            uint32_t u[VPL][8];
            uint32_t K;
            if (all_lean) {
                K = (uint32_t)(q.zp - kMagicBits);
                const float2 inv2 = make_float2(q.inv, q.inv);
                const float2 nstep2 = make_float2(-q.step, -q.step);
                const float hic = (float)(qmax - q.zp), loc = (float)(-q.zp);
#pragma unroll
                for (int h = 0; h < VPL; ++h) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        float2 t = __fmul2_rn(w2[h][k], inv2);
                        if (STATIC) {
                            t.x = fmaxf(fminf(t.x, hic), loc);
                            t.y = fmaxf(fminf(t.y, hic), loc);
                        }
                        // t * 1 + magic: the same value as t + magic, but as a single FMA that
                        // cannot be merged with the multiply that produced t (the assembler was
                        // seen to contract a packed multiply followed by a packed add, which
                        // changes the rounding at exact .5 ties)
                        const float2 uf = __ffma2_rn(t, one2, magic2);
                        u[h][2 * k] = __float_as_uint(uf.x);
                        u[h][2 * k + 1] = __float_as_uint(uf.y);
                        if (MU) {
                            const float2 rq = __fadd2_rn(uf, nmagic2);                 // q - Z, exact
                            const float2 neps = __ffma2_rn(nstep2, rq, w2[h][k]);      // -(Step (q - Z) - w^)
                            eneg = __ffma2_rn(neps, make_float2(mu8[h][2 * k], mu8[h][2 * k + 1]), eneg);
                        }
                    }
                }
            } else {
                K = 0u;
#pragma unroll
                for (int h = 0; h < VPL; ++h) {
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int c0 = code_generic(w2[h][k].x, q.inv, q.zp, qmax);
                        const int c1 = code_generic(w2[h][k].y, q.inv, q.zp, qmax);
                        u[h][2 * k] = (uint32_t)c0;
                        u[h][2 * k + 1] = (uint32_t)c1;
                        if (MU) {
                            const float r0 = (float)((long long)c0 - (long long)q.zp);
                            const float r1 = (float)((long long)c1 - (long long)q.zp);
                            eneg.x = __fmaf_rn(__fmaf_rn(-q.step, r0, w2[h][k].x), mu8[h][2 * k], eneg.x);
                            eneg.y = __fmaf_rn(__fmaf_rn(-q.step, r1, w2[h][k].y), mu8[h][2 * k + 1], eneg.y);
                        }
                    }
                }
            }
            store_lane<BITS, BYTES_OUT, VPL>(orow, idxl, u, K, bits, active, quad3, pair3, lane);
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

template <class D, int BITS, bool STATIC, bool MU, bool BYTES_OUT>
static aweq_status launch_wq(const WarpQuantParams &p, cudaStream_t stream)
{
    long long blocks = (p.nrows + kWqWarps - 1) / kWqWarps;
    const long long cap = (long long)kSmCount * 8 * 4;      // a few waves; warps stride over the rows beyond that
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    // two vectors per lane need an even number of vectors per row, 32-byte aligned rows and
    // groups of at least 16 columns
    const bool two = (p.nvec % 2 == 0) && (p.ld % 16 == 0) && ((reinterpret_cast<uintptr_t>(p.X) & 31) == 0) &&
                     (STATIC || p.lanes_per_group >= 2);
    if (two)
        warpquant_kernel<D, BITS, STATIC, MU, BYTES_OUT, 2><<<(unsigned)blocks, kWqWarps * 32, 0, stream>>>(p);
    else
        warpquant_kernel<D, BITS, STATIC, MU, BYTES_OUT, 1><<<(unsigned)blocks, kWqWarps * 32, 0, stream>>>(p);
    AWEQ_LAUNCH_CHECK();
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
