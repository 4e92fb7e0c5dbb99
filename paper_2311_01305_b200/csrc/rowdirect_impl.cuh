// Row-wise Eq. 1-2 quantiser with plain loads: no shared-memory ring, no bulk copies.
//
// A team of TW warps owns one row at a time and takes rows team by team over the whole
// grid: a thread loads its V 16-byte vectors of the row straight from global memory (all V
// loads in flight), keeps the scaled values in registers, the team agrees on the row's
// extremes (redux.sync, a few words of shared memory and a named barrier when the team has
// more than one warp), every thread forms Step, 1/Step and Z and writes the codes of its
// vectors.  (A two-sweep form for rows too long for a team's registers, with the second sweep
// served by the L2, was measured at 2.3 TB/s and is not kept.)
// Latency is hidden by the number of resident teams rather than by a staging pipeline, which
// suits matrices of a few thousand rows (the weight matrices of step 4), where a persistent
// ring spends most of its time filling and draining.  On the long runs of rows of step 6 the
// resident teams alone leave the kernel waiting for loads (24 warps x 1.5 KB in flight per SM at
// 768 columns): there a team issues the loads of its next row as soon as the current row has
// been unpacked, before the reduction, Step / Z and the codes, and holds as many vectors per thread
// as the registers allow (768 columns 5.45 -> 5.90 TB/s, 3072 5.53 -> 6.39, 5120 5.92 -> 6.07,
// 9216 5.46 -> 6.27, 13824 6.05 -> 6.35, 36864 5.23 -> 6.14).  Shared memory: 768 bytes.
//
// The arithmetic (see rowquant_impl.cuh): binary32, no FMA
// contraction across the two multiplies, ties to even, the literal path when a clamp could
// fire or the zero-point is too large for the add-constant rounding.
#pragma once
#include "rowquant_impl.cuh"

namespace aweq {

constexpr int kRdThreads = 256;
// threads of a CTA: 256 (several teams), or the team itself when it has more than 8 warps
__host__ __device__ constexpr int rd_threads(int TW) { return TW > 8 ? TW * 32 : kRdThreads; }
// CTAs per SM the kernel is compiled for: three while the registers allow it (the next row's
// raw vectors count when they are loaded early), else two; one for a team of a whole CTA
__host__ __device__ constexpr int rd_ctas_per_sm(int TW, int V, bool PF) { return TW > 8 ? 1 : V <= (PF ? 3 : 4) ? 3 : 2; }

struct RdSmem {
    float2 red[2][32];
    float rsum[2][32];
};

template <class D, bool SC_REGS>
__device__ __forceinline__ void rd_scaled(const uint4 &raw, const float *scale, int idx, const float2 (&sc)[4],
                                          float2 (&x)[4])
{
    x[0] = D::to_float2(D::from_bits(raw.x));
    x[1] = D::to_float2(D::from_bits(raw.y));
    x[2] = D::to_float2(D::from_bits(raw.z));
    x[3] = D::to_float2(D::from_bits(raw.w));
    if (SC_REGS) {
#pragma unroll
        for (int k = 0; k < 4; ++k) x[k] = __fmul2_rn(x[k], sc[k]);
    } else if (scale) {
        const float4 s0 = ldg_f4(scale + (size_t)idx * 8), s1 = ldg_f4(scale + (size_t)idx * 8 + 4);
        x[0] = __fmul2_rn(x[0], make_float2(s0.x, s0.y));
        x[1] = __fmul2_rn(x[1], make_float2(s0.z, s0.w));
        x[2] = __fmul2_rn(x[2], make_float2(s1.x, s1.y));
        x[3] = __fmul2_rn(x[3], make_float2(s1.z, s1.w));
    }
}

// codes of one vector (and its share of minus eps . mu), stored
template <bool MU, bool BYTES_OUT>
__device__ __forceinline__ void rd_codes(const float2 (&x)[4], const QParams &q, bool lean, int qmax, int bits,
                                         const float *mu, int idx, unsigned char *dst, float2 &eneg)
{
    uint32_t u[8];
    float mu8[8];
    if (MU) load8(mu + (size_t)idx * 8, mu8);
    if (lean) {
        const uint32_t K = (uint32_t)(q.zp - kMagicBits);
        const float2 inv2 = make_float2(q.inv, q.inv), nstep2 = make_float2(-q.step, -q.step);
        const float2 magic2 = make_float2(kMagic, kMagic), nmagic2 = make_float2(-kMagic, -kMagic);
        const float2 one2 = make_float2(1.0f, 1.0f);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float2 t = __fmul2_rn(x[k], inv2);
            // t * 1 + magic as one FMA: equal to t + magic, and it cannot be contracted with the
            // multiply above (which would change the rounding at exact ties)
            const float2 uf = __ffma2_rn(t, one2, magic2);
            u[2 * k] = __float_as_uint(uf.x);
            u[2 * k + 1] = __float_as_uint(uf.y);
            if (MU) {
                const float2 rq = __fadd2_rn(uf, nmagic2);              // q - Z, exact
                const float2 neps = __ffma2_rn(nstep2, rq, x[k]);       // -(Step (q - Z) - v^)
                eneg = __ffma2_rn(neps, make_float2(mu8[2 * k], mu8[2 * k + 1]), eneg);
            }
        }
        store_codes(dst, u, K, bits, BYTES_OUT);
    } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int c0 = code_generic(x[k].x, q.inv, q.zp, qmax), c1 = code_generic(x[k].y, q.inv, q.zp, qmax);
            u[2 * k] = (uint32_t)c0;
            u[2 * k + 1] = (uint32_t)c1;
            if (MU) {
                const float r0 = (float)((long long)c0 - (long long)q.zp), r1 = (float)((long long)c1 - (long long)q.zp);
                eneg.x = __fmaf_rn(__fmaf_rn(-q.step, r0, x[k].x), mu8[2 * k], eneg.x);
                eneg.y = __fmaf_rn(__fmaf_rn(-q.step, r1, x[k].y), mu8[2 * k + 1], eneg.y);
            }
        }
        store_codes(dst, u, 0u, bits, BYTES_OUT);
    }
}

// V: vectors per thread; TW: warps per team; PF: the loads of the team's next row are issued
// before the current row is reduced and quantised (two rows in flight per team)
template <class D, int V, int TW, bool MU, bool BYTES_OUT, bool PF = false>
__global__ void __launch_bounds__(rd_threads(TW), rd_ctas_per_sm(TW, V, PF))
rowdirect_kernel(const RowQuantParams p)
{
    __shared__ RdSmem sm;
    pdl_begin();
    constexpr int T = TW * 32;
    constexpr int teams = rd_threads(TW) / T;
    constexpr bool SC_REGS = V <= 4;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tm = threadIdx.x / T, tt = threadIdx.x % T;
    const int tw0 = tm * TW;
    const int qmax = (1 << p.bits) - 1;
    const int vec_bytes = BYTES_OUT ? 8 : p.bits;
    int parity = 0;

    float2 sc[SC_REGS ? V : 1][4];
    if (SC_REGS) {
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int idx = tt + v * T;
#pragma unroll
            for (int k = 0; k < 4; ++k) sc[v][k] = make_float2(1.0f, 1.0f);
            if (p.scale && idx < p.nvec) {
                const float4 s0 = ldg_f4(p.scale + (size_t)idx * 8), s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
                sc[v][0] = make_float2(s0.x, s0.y); sc[v][1] = make_float2(s0.z, s0.w);
                sc[v][2] = make_float2(s1.x, s1.y); sc[v][3] = make_float2(s1.z, s1.w);
            }
        }
    }

    const long long nteams = (long long)gridDim.x * teams;
    uint4 raw[V];
    auto load_row = [&](long long row) {
        const uint16_t *xrow = p.X + row * p.ld;
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int idx = tt + v * T;
            raw[v] = make_uint4(0, 0, 0, 0);
            if (v < V - 1 || idx < p.nvec) raw[v] = ldg_stream(xrow + (size_t)idx * 8);
        }
    };
    if (PF && (long long)blockIdx.x * teams + tm < p.nrows) load_row((long long)blockIdx.x * teams + tm);
    for (long long row = (long long)blockIdx.x * teams + tm; row < p.nrows; row += nteams) {
        unsigned char *orow = p.out + row * p.out_pitch;
        float lo = INFINITY, hi = -INFINITY;
        float2 xh[V][4];
        {
            if (!PF) load_row(row);
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int idx = tt + v * T;
                if (v < V - 1 || idx < p.nvec) {
                    rd_scaled<D, SC_REGS>(raw[v], p.scale, idx, sc[SC_REGS ? v : 0], xh[v]);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        lo = fmin3(lo, xh[v][k].x, xh[v][k].y);
                        hi = fmax3(hi, xh[v][k].x, xh[v][k].y);
                    }
                }
            }
            if (PF && row + nteams < p.nrows) load_row(row + nteams);
        }
        lo = redux_min(lo, 0xffffffffu);
        hi = redux_max(hi, 0xffffffffu);
        if (TW > 1) {
            if (lane == 0) sm.red[parity][warp] = make_float2(lo, hi);
            named_bar_sync(1 + tm, T);
            const float2 o = lane < TW ? sm.red[parity][tw0 + lane] : make_float2(INFINITY, -INFINITY);
            lo = redux_min(o.x, 0xffffffffu);
            hi = redux_max(o.y, 0xffffffffu);
        }
        const QParams q = make_qparams(lo, hi, qmax);
        const bool lean = qflags(q, hi, qmax) == (kQFast | kQNoClamp);
        if (tt == 0) {
            p.step[row] = q.step;
            p.zp[row] = q.zp;
        }
        float2 eneg = make_float2(0.0f, 0.0f);
#pragma unroll
        for (int v = 0; v < V; ++v) {
            const int idx = tt + v * T;
            if (v < V - 1 || idx < p.nvec)
                rd_codes<MU, BYTES_OUT>(xh[v], q, lean, qmax, p.bits, p.mu, idx, orow + (size_t)idx * vec_bytes, eneg);
        }
        if (MU) {
            const float eacc = -warp_sum(__fadd_rn(eneg.x, eneg.y));
            if (TW > 1) {
                if (lane == 0) sm.rsum[parity][warp] = eacc;
                named_bar_sync(1 + tm, T);
                if (tt == 0) {
                    float tot = 0.0f;
                    for (int w = 0; w < TW; ++w) tot += sm.rsum[parity][tw0 + w];
                    p.epsmu[row] = tot;
                    if (p.bias.out || p.bias.out_f32) write_bias(row, tot, p.bias.in, p.bias.out, p.bias.out_f32, p.bias.bf16);
                }
            } else if (lane == 0) {
                p.epsmu[row] = eacc;
                if (p.bias.out || p.bias.out_f32) write_bias(row, eacc, p.bias.in, p.bias.out, p.bias.out_f32, p.bias.bf16);
            }
        }
        parity ^= 1;
    }
}

template <class D, int V, int TW, bool MU, bool BYTES_OUT, bool PF = false>
static aweq_status rd_launch_one(const RowQuantParams &p, cudaStream_t stream)
{
    constexpr int teams = rd_threads(TW) / (TW * 32);
    constexpr int per_sm = rd_ctas_per_sm(TW, V, PF);
    long long grid = (p.nrows + teams - 1) / teams;
    if (grid > (long long)kSmCount * per_sm) grid = (long long)kSmCount * per_sm;
    if (grid < 1) grid = 1;
    AWEQ_LAUNCH((rowdirect_kernel<D, V, TW, MU, BYTES_OUT, PF>), dim3((unsigned)grid), dim3(rd_threads(TW)), 0, stream, p);
    return AWEQ_OK;
}

// Largest V of the step-6 shapes: two rows of a team are in flight there, which 128 registers hold
// up to nine vectors per thread (nine spills a few words in the small teams and still measured 5-8 %
// faster than a larger team with five; ten spills over a hundred bytes and loses a quarter).
constexpr int kRdActMaxV = 9;
constexpr int kRdActMaxTeamWarps = 16;

// mode: 0 = activations (one byte per code, next row's loads issued early), 1 = weights with eps.mu
// sums, 2 = weights without
template <class D, int V, int TW>
static aweq_status rd_launch_weights(const RowQuantParams &p, int mode, cudaStream_t stream)
{
    if (mode == 1) return rd_launch_one<D, V, TW, true, false>(p, stream);
    return rd_launch_one<D, V, TW, false, false>(p, stream);
}

template <class D>
static aweq_status rd_launch(const RowQuantParams &p, int team_warps, int V, int mode, cudaStream_t stream)
{
    if (mode == 0) {
        // the shapes plan_rowdirect gives step 6: one warp with 1-9 vectors, larger teams with 5-9
#define AWEQ_RD_ACT(tw, v) if (team_warps == tw && V == v) return rd_launch_one<D, v, tw, false, true, true>(p, stream);
        AWEQ_RD_ACT(1, 1) AWEQ_RD_ACT(1, 2) AWEQ_RD_ACT(1, 3) AWEQ_RD_ACT(1, 4) AWEQ_RD_ACT(1, 5) AWEQ_RD_ACT(1, 6)
        AWEQ_RD_ACT(1, 7) AWEQ_RD_ACT(1, 8) AWEQ_RD_ACT(1, 9)
        AWEQ_RD_ACT(2, 5) AWEQ_RD_ACT(2, 6) AWEQ_RD_ACT(2, 7) AWEQ_RD_ACT(2, 8) AWEQ_RD_ACT(2, 9)
        AWEQ_RD_ACT(4, 5) AWEQ_RD_ACT(4, 6) AWEQ_RD_ACT(4, 7) AWEQ_RD_ACT(4, 8) AWEQ_RD_ACT(4, 9)
        AWEQ_RD_ACT(8, 5) AWEQ_RD_ACT(8, 6) AWEQ_RD_ACT(8, 7) AWEQ_RD_ACT(8, 8) AWEQ_RD_ACT(8, 9)
        AWEQ_RD_ACT(16, 5) AWEQ_RD_ACT(16, 6) AWEQ_RD_ACT(16, 7) AWEQ_RD_ACT(16, 8) AWEQ_RD_ACT(16, 9)
#undef AWEQ_RD_ACT
        return AWEQ_ERR_UNSUPPORTED;
    }
#define AWEQ_RD_CASE(tw, v) if (team_warps == tw && V == v) return rd_launch_weights<D, v, tw>(p, mode, stream);
    AWEQ_RD_CASE(1, 1) AWEQ_RD_CASE(1, 2) AWEQ_RD_CASE(1, 3) AWEQ_RD_CASE(1, 4) AWEQ_RD_CASE(1, 5)
    AWEQ_RD_CASE(1, 6) AWEQ_RD_CASE(1, 7) AWEQ_RD_CASE(1, 8) AWEQ_RD_CASE(1, 9) AWEQ_RD_CASE(1, 10)
    AWEQ_RD_CASE(2, 6) AWEQ_RD_CASE(2, 7) AWEQ_RD_CASE(2, 8) AWEQ_RD_CASE(2, 9) AWEQ_RD_CASE(2, 10)
    AWEQ_RD_CASE(4, 6) AWEQ_RD_CASE(4, 7) AWEQ_RD_CASE(4, 8) AWEQ_RD_CASE(4, 9) AWEQ_RD_CASE(4, 10)
    AWEQ_RD_CASE(8, 6) AWEQ_RD_CASE(8, 7) AWEQ_RD_CASE(8, 8) AWEQ_RD_CASE(8, 9) AWEQ_RD_CASE(8, 10)
    AWEQ_RD_CASE(32, 3) AWEQ_RD_CASE(32, 4) AWEQ_RD_CASE(32, 5)
#undef AWEQ_RD_CASE
    return AWEQ_ERR_UNSUPPORTED;
}

bool plan_rowdirect(long long cols, bool weights, int *team_warps, int *V);
aweq_status run_rowdirect(const RowQuantParams &p, int team_warps, int V, int mode, aweq_dtype dt, cudaStream_t stream);
aweq_status rd_launch_f16(const RowQuantParams &p, int team_warps, int V, int mode, cudaStream_t stream);
aweq_status rd_launch_bf16(const RowQuantParams &p, int team_warps, int V, int mode, cudaStream_t stream);

}  // namespace aweq
