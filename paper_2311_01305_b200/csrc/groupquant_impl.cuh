// Device code of the group-128 quantiser (see groupquant.cu for the design).
#pragma once
#include "common.cuh"

namespace aweq {

constexpr int kGqWarps = 8;

struct GroupQuantParams {
    const uint16_t *W;
    long long nrows, ld;
    int nvec;                   // 16-byte vectors per row
    int nwin;                   // windows of 32 vectors per row
    long long nbatch;           // batches of R rows
    const float *scale;         // s, or NULL
    const float *mu;            // E[x^] (MU only)
    unsigned char *out;
    long long out_pitch;
    float *step;
    int *zp;
    int ngroups;                // groups per row
    float *partial;             // [nwin][prow]: minus the eps . mu sum of a (window, row)
    long long prow;             // nrows rounded up to whole batches
};

template <int BITS>
__device__ __forceinline__ void gq_store(unsigned char *orow, int idx, const uint32_t (&u)[8], uint32_t K, bool active,
                                         int lane)
{
    if (BITS == 8) {
        const uint32_t kp = K * 0x01010101u;
        uint2 w;
        w.x = u[0] + (u[1] << 8) + (u[2] << 16) + (u[3] << 24) + kp;
        w.y = u[4] + (u[5] << 8) + (u[6] << 16) + (u[7] << 24) + kp;
        if (active) *reinterpret_cast<uint2 *>(orow + (size_t)idx * 8) = w;
    } else {
        uint32_t w = 0, m = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            w += u[e] << (e * BITS);
            m += 1u << (e * BITS);
        }
        w += K * m;
        if (BITS == 4) {
            if (active) *reinterpret_cast<uint32_t *>(orow + (size_t)idx * 4) = w;
        } else {
            // 3 bits: four lanes hold 4 x 24 bits = three 32-bit words
            w &= 0x00FFFFFFu;
            const int q4 = lane & 3;
            const uint32_t up = __shfl_down_sync(0xffffffffu, w, 1);
            uint32_t word;
            if (q4 == 0) word = w | (up << 24);
            else if (q4 == 1) word = (w >> 8) | (up << 16);
            else word = (w >> 16) | (up << 8);
            if (active && q4 < 3) *reinterpret_cast<uint32_t *>(orow + (size_t)(idx >> 2) * 12 + q4 * 4) = word;
        }
    }
}

// the eight scaled values of a vector
template <class D>
__device__ __forceinline__ void gq_scaled(const uint4 &raw, const float2 (&s2)[4], float2 (&w2)[4])
{
    float w[8];
    widen8<D>(raw, w);
#pragma unroll
    for (int k = 0; k < 4; ++k) w2[k] = __fmul2_rn(make_float2(w[2 * k], w[2 * k + 1]), s2[k]);
}

// Second pass over a batch: the (1 / Step, Z, Step) of every row's group come from the lane that
// formed them; codes, packing, stores and this lane's share of eps . E[x^] per row (minus it, in
// e[]).  LEAN: every pair of the batch may use the add-constant rounding without a clamp.
template <class D, int BITS, bool MU, int R, bool KEEP, bool LEAN>
__device__ __forceinline__ void gq_codes(const GroupQuantParams &p, uint4 (&raw)[R], float2 (&w2)[KEEP ? R : 1][4],
                                         const float2 (&s2)[4], const float2 (&mu2)[4], const QParams &q,
                                         long long row0, int idx, bool active, int lane, float (&e)[R])
{
    constexpr int qmax = (1 << BITS) - 1;
    const float2 magic2 = make_float2(kMagic, kMagic), nmagic2 = make_float2(-kMagic, -kMagic);
    const float2 one2 = make_float2(1.0f, 1.0f);
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int src = 2 * r + (lane >> 4);
        const float inv = __shfl_sync(0xffffffffu, q.inv, src);
        const int zpv = __shfl_sync(0xffffffffu, q.zp, src);
        const float stp = MU ? __shfl_sync(0xffffffffu, q.step, src) : 0.0f;
        float2(&v)[4] = w2[KEEP ? r : 0];
        if (!KEEP) {
            // formed again on purpose: the empty statement keeps the compiler from holding on to
            // the first pass's values (which is the register use this variant exists to avoid)
            asm volatile("" : "+r"(raw[r].x), "+r"(raw[r].y), "+r"(raw[r].z), "+r"(raw[r].w));
            gq_scaled<D>(raw[r], s2, v);
        }
        uint32_t u[8];
        uint32_t K;
        float2 eneg = make_float2(0.0f, 0.0f);
        if (LEAN) {
            K = (uint32_t)(zpv - kMagicBits);
            const float2 inv2 = make_float2(inv, inv);
            const float2 nstep2 = make_float2(-stp, -stp);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 t = __fmul2_rn(v[k], inv2);
                // t * 1 + magic as one FMA: the same value as t + magic, and it cannot be merged
                // with the multiply that produced t (a packed multiply followed by a packed add
                // was seen to be contracted, which changes the rounding at exact .5 ties)
                const float2 uf = __ffma2_rn(t, one2, magic2);
                u[2 * k] = __float_as_uint(uf.x);
                u[2 * k + 1] = __float_as_uint(uf.y);
                if (MU) {
                    const float2 rq = __fadd2_rn(uf, nmagic2);                 // q - Z, exact
                    const float2 neps = __ffma2_rn(nstep2, rq, v[k]);          // -(Step (q - Z) - w^)
                    eneg = __ffma2_rn(neps, mu2[k], eneg);
                }
            }
        } else {
            K = 0u;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int c0 = code_generic(v[k].x, inv, zpv, qmax), c1 = code_generic(v[k].y, inv, zpv, qmax);
                u[2 * k] = (uint32_t)c0;
                u[2 * k + 1] = (uint32_t)c1;
                if (MU) {
                    const float r0 = (float)((long long)c0 - (long long)zpv), r1 = (float)((long long)c1 - (long long)zpv);
                    eneg.x = __fmaf_rn(__fmaf_rn(-stp, r0, v[k].x), mu2[k].x, eneg.x);
                    eneg.y = __fmaf_rn(__fmaf_rn(-stp, r1, v[k].y), mu2[k].y, eneg.y);
                }
            }
        }
        const bool st_ok = active && row0 + r < p.nrows;
        gq_store<BITS>(p.out + (row0 + r) * p.out_pitch, idx, u, K, st_ok, lane);
        e[r] = __fadd_rn(eneg.x, eneg.y);
    }
}

// R rows per batch (4 or 8); KEEP: the scaled values of a batch stay in registers between the
// two passes (otherwise they are formed again from the 16-bit data, which costs 12 instructions
// per vector and saves 4 registers per row); OCC: CTAs per SM the register budget is set for.
template <class D, int BITS, bool MU, int R, bool KEEP, int OCC>
__global__ void __launch_bounds__(kGqWarps * 32, OCC)
groupquant_kernel(const GroupQuantParams p)
{
    pdl_begin();
    static_assert(R == 4 || R == 8 || R == 16, "rows per batch");
    constexpr int qmax = (1 << BITS) - 1;
    constexpr int KR = KEEP ? R : 1;
    const int lane = threadIdx.x & 31;
    const bool upper = lane >= 16;
    const long long gw = (long long)blockIdx.x * kGqWarps + (threadIdx.x >> 5);
    const long long nw = (long long)gridDim.x * kGqWarps;
    const long long items = p.nbatch * p.nwin;
    const int orow = (lane & (2 * R - 1)) >> 1, ogrp = lane & 1;      // the (row, group) pair this lane forms
    const float2 one2 = make_float2(1.0f, 1.0f);

    int cur_win = -1;
    float2 s2[4], mu2[4];
    for (long long it = gw; it < items; it += nw) {
        const int win = (int)(it % p.nwin);
        const long long row0 = (it / p.nwin) * R;
        const int idx = win * 32 + lane;
        const bool active = idx < p.nvec;
        if (win != cur_win) {
            cur_win = win;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                s2[k] = one2;
                mu2[k] = make_float2(0.0f, 0.0f);
            }
            if (active && p.scale) {
                const float4 a = ldg_f4(p.scale + (size_t)idx * 8), b = ldg_f4(p.scale + (size_t)idx * 8 + 4);
                s2[0] = make_float2(a.x, a.y); s2[1] = make_float2(a.z, a.w);
                s2[2] = make_float2(b.x, b.y); s2[3] = make_float2(b.z, b.w);
            }
            if (MU && active) {
                const float4 a = ldg_f4(p.mu + (size_t)idx * 8), b = ldg_f4(p.mu + (size_t)idx * 8 + 4);
                mu2[0] = make_float2(a.x, a.y); mu2[1] = make_float2(a.z, a.w);
                mu2[2] = make_float2(b.x, b.y); mu2[3] = make_float2(b.z, b.w);
            }
        }
        // ---- all loads of the batch first
        uint4 raw[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            raw[r] = make_uint4(0, 0, 0, 0);
            if (active && row0 + r < p.nrows) raw[r] = ldg_stream(p.W + (row0 + r) * p.ld + (size_t)idx * 8);
        }
        // ---- scaled values and group extremes; lane (orow, ogrp) keeps the extremes of its pair
        float2 w2[KR][4];
        float mya = 0.0f, myb = 1.0f;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float2(&v)[4] = w2[KEEP ? r : 0];
            gq_scaled<D>(raw[r], s2, v);
            float a = fmin3(v[0].x, v[0].y, v[1].x), b = fmax3(v[0].x, v[0].y, v[1].x);
            a = fmin3(a, v[1].y, v[2].x); b = fmax3(b, v[1].y, v[2].x);
            a = fmin3(a, v[2].y, v[3].x); b = fmax3(b, v[2].y, v[3].x);
            a = fminf(a, v[3].y); b = fmaxf(b, v[3].y);
            // one full-mask reduction per group with the other half's lanes neutral (a reduction
            // over a 16-lane sub-mask is slower: the two halves would name different masks)
            const float a0 = redux_min(upper ? INFINITY : a, 0xffffffffu);
            const float a1 = redux_min(upper ? a : INFINITY, 0xffffffffu);
            const float b0 = redux_max(upper ? -INFINITY : b, 0xffffffffu);
            const float b1 = redux_max(upper ? b : -INFINITY, 0xffffffffu);
            if (orow == r) {
                mya = ogrp ? a1 : a0;
                myb = ogrp ? b1 : b0;
            }
        }
        const bool pair_ok = row0 + orow < p.nrows && win * 2 + ogrp < p.ngroups;
        if (!pair_ok) {                 // nothing there: harmless numbers (Step 1 / qmax, Z 0)
            mya = 0.0f;
            myb = 1.0f;
        }
        const QParams q = make_qparams(mya, myb, qmax);
        const int fl = qflags(q, myb, qmax);
        if (pair_ok && lane < 2 * R) {
            const size_t at = (size_t)(row0 + orow) * p.ngroups + win * 2 + ogrp;
            p.step[at] = q.step;
            p.zp[at] = q.zp;
        }
        // bit 2r + g: the pair (row r, group g) may take the add-constant rounding without a clamp
        const uint32_t lean_mask = __ballot_sync(0xffffffffu, fl == (kQFast | kQNoClamp));

        // ---- codes.  A pair leaves the add-constant path only on a rounding tie at the top of
        // its range or with a huge zero-point, so the decision is taken once for the whole batch.
        float e[R];
        if (lean_mask == 0xffffffffu)
            gq_codes<D, BITS, MU, R, KEEP, true>(p, raw, w2, s2, mu2, q, row0, idx, active, lane, e);
        else
            gq_codes<D, BITS, MU, R, KEEP, false>(p, raw, w2, s2, mu2, q, row0, idx, active, lane, e);
        if (MU) {
            // R row sums over 32 lanes: exchange halves, keep half of the rows, repeat; then plain
            // exchanges.  Always the same order, so the sums are reproducible.
            int off = 16;
#pragma unroll
            for (int live = R; live > 1; live >>= 1, off >>= 1) {
                const bool hi = (lane & off) != 0;
#pragma unroll
                for (int i = 0; i < live / 2; ++i) {
                    const float send = hi ? e[i] : e[i + live / 2], keep = hi ? e[i + live / 2] : e[i];
                    e[i] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, off));
                }
            }
#pragma unroll
            for (; off >= 1; off >>= 1) e[0] = __fadd_rn(e[0], __shfl_xor_sync(0xffffffffu, e[0], off));
            // lanes (32 / R) k .. (32 / R) k + 32 / R - 1 now hold row k of the batch
            if ((lane & (32 / R - 1)) == 0) p.partial[(size_t)win * p.prow + row0 + lane / (32 / R)] = e[0];
        }
    }
}

// eps . E[x^] of a row = the sum of its windows' partials, in window order; Eq. 15's bias with it
__global__ void __launch_bounds__(256)
groupquant_finalize_kernel(const float *__restrict__ partial, int nwin, long long prow, long long nrows,
                           float *__restrict__ epsmu, const BiasIO bias)
{
    pdl_begin();
    const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= nrows) return;
    float acc = 0.0f;
    for (int w = 0; w < nwin; ++w) acc = __fadd_rn(acc, partial[(size_t)w * prow + row]);
    const float tot = -acc;
    epsmu[row] = tot;
    if (bias.out || bias.out_f32) write_bias(row, tot, bias.in, bias.out, bias.out_f32, bias.bf16);
}

}  // namespace aweq
