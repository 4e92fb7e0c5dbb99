// Row-wise Eq. 1-2 quantiser with a per-column scale: the kernel behind
// step 4 in per-output-channel mode (W^ = diag(s) W, Eq. 3, quantised per row)
// and step 6 in per-token mode (X^ = X diag(s)^-1 quantised per token).
//
// Every row needs its own minimum and maximum before a single code can be
// produced, so a row must be looked at twice while HBM should see it once.
// The kernel keeps the scaled row on chip: persistent CTAs pull tiles of whole
// rows through a ring of shared-memory stages with 1-D bulk copies (TMA,
// completion on mbarriers; warp 0 issues the copies between its own rows, so
// that a CTA is 8 or 16 warps and the register file divides evenly over the
// four schedulers).  A stage is released as soon as its rows are in registers,
// so its refill overlaps the rest of the work on those rows.  A team of T threads owns one row of the stage at a time,
// each thread holding V 16-byte vectors of the row, already multiplied by the
// column scale, in registers; T is chosen small (few warps per row, V up to
// 10) because everything that happens once per row -- the exchange of the
// extremes, Step, 1/Step, Z -- is repeated by every warp of the team.  The row
// extremes are reduced with redux.sync inside a warp and through a few words of
// shared memory plus a named barrier across the warps of a team; the codes are
// then formed from the registers and stored with coalesced 8-byte (or b-byte)
// stores.
//
// Rounding adds 1.5 * 2^23 in binary32 (rounds to an integer, ties to even, like
// rint).  The lower clamp of Eq. 1 cannot fire when Step and Z come from the
// same vector (t >= fl(lo * inv) implies rint(t) >= -Z); the upper clamp can only
// fire when rint(hi * inv) + Z exceeds 2^b - 1, which is decided once per row.
// Rows where it does, and rows whose zero-point is too large for the rounding
// trick, take the literal cvt.rni path.  Multiplies, the rounding add and the
// eps . E[x^] terms use the packed binary32 instructions of sm_100.
#pragma once
#include "common.cuh"

namespace aweq {

constexpr int kRqStagesMax = 4;
constexpr int kRqMaxV = 10;
constexpr int kRqScaleRegsMaxV = 5;      // up to this many vectors per thread the scales stay in registers

struct RowQuantParams {
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
    int team;             // threads per row (multiple of 32, divides the CTA)
    int rows_per_stage;
    int stages;
    long long ntiles;
    aweq_dev_status *st;
};

struct RowQuantPlan {
    int V, NT, team, rows_per_stage, stages, grid;
    size_t smem;
    long long ntiles;
};

bool plan_rowquant(long long nrows, long long cols, RowQuantPlan *out);
// wide rows of step 6 (rowquant_wide.cu): a plan exists for 10240 < cols <= 40960
bool plan_rowquant_wide(long long nrows, long long cols, RowQuantPlan *out);

struct RqSmem {
    uint64_t full[kRqStagesMax];
    uint64_t empty[kRqStagesMax];
    int abort_flag;
    int pad[15];
    float2 red[2][16];
    float rsum[2][16];
};
constexpr int kRqHeader = 512;
static_assert(sizeof(RqSmem) <= kRqHeader, "header");

// pack eight values u[i] + K (each in [0, 2^b)) into the little-endian bit stream
__device__ __forceinline__ void store_codes(unsigned char *dst, const uint32_t (&u)[8], uint32_t K, int bits, bool bytes_out)
{
    if (bytes_out || bits == 8) {
        const uint32_t kp = K * 0x01010101u;
        uint2 w;
        w.x = u[0] + (u[1] << 8) + (u[2] << 16) + (u[3] << 24) + kp;
        w.y = u[4] + (u[5] << 8) + (u[6] << 16) + (u[7] << 24) + kp;
        *reinterpret_cast<uint2 *>(dst) = w;
    } else if (bits <= 4) {
        uint32_t w = 0, m = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            w += u[i] << (i * bits);
            m += 1u << (i * bits);
        }
        w += K * m;
        if (bits == 4) {
            *reinterpret_cast<uint32_t *>(dst) = w;
        } else if (bits == 2) {
            *reinterpret_cast<uint16_t *>(dst) = (uint16_t)w;
        } else {
            dst[0] = (unsigned char)w;
            dst[1] = (unsigned char)(w >> 8);
            dst[2] = (unsigned char)(w >> 16);
        }
    } else {
        unsigned long long w = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) w |= (unsigned long long)((u[i] + K) & ((1u << bits) - 1)) << (i * bits);
        for (int k = 0; k < bits; ++k) dst[k] = (unsigned char)(w >> (8 * k));
    }
}

// warp 0: is the stage of tile `t` free again (released by every warp after its previous
// use)?  Blocking (bounded) or a single test.  *timed_out is set when a blocking wait gave up.
__device__ __forceinline__ bool rq_stage_free(RqSmem *sm, long long t, int S, bool block, bool *timed_out)
{
    const int s = (int)(t % S);
    const uint32_t use = (uint32_t)(t / S);
    if (use == 0) return true;
    bool ready;
    if (block) {
        ready = mbar_wait(&sm->empty[s], (use - 1) & 1);
        ready = __all_sync(0xffffffffu, ready);
        if (!ready) *timed_out = true;
    } else {
        ready = __all_sync(0xffffffffu, mbar_test(&sm->empty[s], (use - 1) & 1));
    }
    return ready;
}

// warp 0: start the copy of tile `t` of this CTA into its (free) stage.
__device__ __forceinline__ void rq_issue_tile(const RowQuantParams &p, RqSmem *sm, uint4 *stage_base, long long t,
                                              int S, int R, size_t stage_vecs, int lane)
{
    const int s = (int)(t % S);
    const long long row0 = (blockIdx.x + t * gridDim.x) * (long long)R;
    const int rows = (int)min((long long)R, p.nrows - row0);
    const uint32_t row_bytes = (uint32_t)p.nvec * 16u;
    uint4 *dst = stage_base + (size_t)s * stage_vecs;
    if (lane == 0) mbar_arrive_expect_tx(&sm->full[s], (uint32_t)rows * row_bytes);
    __syncwarp();
    if (p.ld == (long long)p.nvec * 8) {
        // the tile is one contiguous range: a copy per 32 KB chunk
        const uint32_t total = (uint32_t)rows * row_bytes;
        const uint32_t chunk = 32768u;
        const char *src = reinterpret_cast<const char *>(p.X + row0 * p.ld);
        for (uint32_t off = lane * chunk; off < total; off += 32u * chunk)
            bulk_g2s(reinterpret_cast<char *>(dst) + off, src + off, min(chunk, total - off), &sm->full[s]);
    } else {
        for (int r = lane; r < rows; r += 32)
            bulk_g2s(dst + (size_t)r * p.nvec, p.X + (row0 + r) * p.ld, row_bytes, &sm->full[s]);
    }
}

template <class D, int V, int NT, bool MU, bool BYTES_OUT>
__global__ void __launch_bounds__(NT, NT <= 256 ? 2 : 1)
rowquant_kernel(const RowQuantParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RqSmem *sm = reinterpret_cast<RqSmem *>(smem_raw);
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw + kRqHeader);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = p.team;
    const int teams = NT / T;
    const int R = p.rows_per_stage;
    const int S = p.stages;
    const size_t stage_vecs = (size_t)R * p.nvec;
    const int qmax = (1 << p.bits) - 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sm->full[s], 1);
            mbar_init(&sm->empty[s], NT / 32);
        }
        sm->abort_flag = 0;
        mbar_init_fence();
    }
    pdl_begin();                 // everything above overlaps the tail of the previous kernel
    __syncthreads();

    // tiles of R rows, dealt round-robin to the persistent CTAs
    const long long my_tiles = p.ntiles > blockIdx.x ? (p.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    // A stage is needed only until its rows sit in registers, so it is released right after
    // the first pass and refilled while Step / Z are formed and the codes are written: up to
    // S tiles are in flight.  warp 0 refills whenever it sees a free stage (single tests
    // after each phase, a bounded wait only when the next tile has not been requested yet).
    // That pays when one row fills a stage and the whole CTA works on it (the widest rows: one
    // tile in flight is then too little); with several rows per stage the stage is released
    // at the end of the tile and refilled at the top of the next one (measured: releasing early
    // costs 5-9 % there).
    constexpr bool early = NT == 512;           // the 512-thread shape is only used with one team
    bool ok = true;
    long long next_issue = 0;                   // warp 0: first tile not yet requested
    if (warp == 0) {
        const int ahead = early ? S : S - 1;
        for (; next_issue < ahead && next_issue < my_tiles; ++next_issue)
            rq_issue_tile(p, sm, stage_base, next_issue, S, R, stage_vecs, lane);
    }
#define AWEQ_RQ_TRY_REFILL()                                                                   \
    if (early && warp == 0 && next_issue < my_tiles) {                                         \
        bool dummy = false;                                                                    \
        if (rq_stage_free(sm, next_issue, S, false, &dummy)) {                                 \
            rq_issue_tile(p, sm, stage_base, next_issue, S, R, stage_vecs, lane);              \
            ++next_issue;                                                                      \
        }                                                                                      \
    }
    {
        const int tm = threadIdx.x / T, tt = threadIdx.x % T;
        const int wpt = T / 32;                       // warps per team
        const int tw0 = tm * wpt;                     // first warp of my team
        int parity = 0;
        // a thread keeps the same columns for every row: their scale factors live in registers
        // (no equalisation = factors of one, which is exact)
        constexpr bool SC_REGS = V <= kRqScaleRegsMaxV;
        float2 sc[SC_REGS ? V : 1][4];
        if (SC_REGS) {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int idx = tt + v * T;
                if (p.scale && idx < p.nvec) {
                    const float4 s0 = ldg_f4(p.scale + (size_t)idx * 8), s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
                    sc[v][0] = make_float2(s0.x, s0.y); sc[v][1] = make_float2(s0.z, s0.w);
                    sc[v][2] = make_float2(s1.x, s1.y); sc[v][3] = make_float2(s1.z, s1.w);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k) sc[v][k] = make_float2(1.0f, 1.0f);
                }
            }
        }
        for (long long k = 0; k < my_tiles; ++k) {
            if (warp == 0 && next_issue < my_tiles && (!early || next_issue <= k)) {
                // late mode: tile k + S - 1 goes into the stage tile k - 1 used; early mode: only a guard
                bool timed_out = false;
                if (rq_stage_free(sm, next_issue, S, true, &timed_out)) {
                    rq_issue_tile(p, sm, stage_base, next_issue, S, R, stage_vecs, lane);
                    ++next_issue;
                }
                if (timed_out) ok = false;
            }
            const int s = (int)(k % S);
            const uint32_t use = (uint32_t)(k / S);
            ok = ok && mbar_wait(&sm->full[s], use & 1) && !*reinterpret_cast<volatile int *>(&sm->abort_flag);
            // the whole team leaves together, or a later team barrier would miss a warp
            ok = wpt > 1 ? named_bar_and(1 + tm, T, ok) : __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const long long row0 = (blockIdx.x + k * gridDim.x) * (long long)R;
            const int rows = (int)min((long long)R, p.nrows - row0);
            const uint4 *tile = stage_base + (size_t)s * stage_vecs;
            if (early && tm >= rows) {                        // no row for this team in a short last tile
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->empty[s]);
            }
            for (int r = tm; r < rows; r += teams) {
                const uint4 *rowp = tile + (size_t)r * p.nvec;
                float2 xh[V][4];
                float lo = INFINITY, hi = -INFINITY;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int idx = tt + v * T;
                    // only the last vector of a thread can fall outside the row
                    if (v < V - 1 || idx < p.nvec) {
                        const uint4 raw = rowp[idx];
                        xh[v][0] = D::to_float2(D::from_bits(raw.x));
                        xh[v][1] = D::to_float2(D::from_bits(raw.y));
                        xh[v][2] = D::to_float2(D::from_bits(raw.z));
                        xh[v][3] = D::to_float2(D::from_bits(raw.w));
                        if (SC_REGS) {
#pragma unroll
                            for (int k4 = 0; k4 < 4; ++k4) xh[v][k4] = __fmul2_rn(xh[v][k4], sc[v][k4]);
                        } else if (p.scale) {
                            const float4 s0 = ldg_f4(p.scale + (size_t)idx * 8), s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
                            xh[v][0] = __fmul2_rn(xh[v][0], make_float2(s0.x, s0.y));
                            xh[v][1] = __fmul2_rn(xh[v][1], make_float2(s0.z, s0.w));
                            xh[v][2] = __fmul2_rn(xh[v][2], make_float2(s1.x, s1.y));
                            xh[v][3] = __fmul2_rn(xh[v][3], make_float2(s1.z, s1.w));
                        }
                        lo = fmin3(lo, xh[v][0].x, xh[v][0].y); hi = fmax3(hi, xh[v][0].x, xh[v][0].y);
                        lo = fmin3(lo, xh[v][1].x, xh[v][1].y); hi = fmax3(hi, xh[v][1].x, xh[v][1].y);
                        lo = fmin3(lo, xh[v][2].x, xh[v][2].y); hi = fmax3(hi, xh[v][2].x, xh[v][2].y);
                        lo = fmin3(lo, xh[v][3].x, xh[v][3].y); hi = fmax3(hi, xh[v][3].x, xh[v][3].y);
                    }
                }
                if (early && r + teams >= rows) {             // my last row of the tile is in registers
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->empty[s]);
                }
                lo = redux_min(lo, 0xffffffffu);
                hi = redux_max(hi, 0xffffffffu);
                if (wpt > 1) {
                    if (lane == 0) sm->red[parity][warp] = make_float2(lo, hi);
                    named_bar_sync(1 + tm, T);
                    // lane l fetches the partial of the team's warp l; one more reduction over the warp
                    const float2 o = lane < wpt ? sm->red[parity][tw0 + lane] : make_float2(INFINITY, -INFINITY);
                    lo = redux_min(o.x, 0xffffffffu);
                    hi = redux_max(o.y, 0xffffffffu);
                }
                AWEQ_RQ_TRY_REFILL()
                const QParams q = make_qparams(lo, hi, qmax);
                const int fl = qflags(q, hi, qmax);
                const long long row = row0 + r;
                if (tt == 0) {
                    p.step[row] = q.step;
                    p.zp[row] = q.zp;
                }
                unsigned char *orow = p.out + row * p.out_pitch;
                const int vec_bytes = BYTES_OUT ? 8 : p.bits;
                float2 eneg = make_float2(0.0f, 0.0f);            // minus the eps . mu partial sum
                if (fl == (kQFast | kQNoClamp)) {
                    // lean path: no clamp can fire in this row; packed multiply and rounding add
                    const uint32_t K = (uint32_t)(q.zp - kMagicBits);
                    const float2 inv2 = make_float2(q.inv, q.inv), nstep2 = make_float2(-q.step, -q.step);
                    const float2 magic2 = make_float2(kMagic, kMagic), nmagic2 = make_float2(-kMagic, -kMagic);
                    const float2 one2 = make_float2(1.0f, 1.0f);
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = tt + v * T;
                        if (v < V - 1 || idx < p.nvec) {
                            uint32_t u[8];
                            float mu8[8];
                            if (MU) load8(p.mu + (size_t)idx * 8, mu8);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float2 t = __fmul2_rn(xh[v][k], inv2);
                                // t * 1 + magic as one FMA: equal to t + magic, and it cannot be
                                // contracted with the multiply above (which would change ties)
                                const float2 uf = __ffma2_rn(t, one2, magic2);
                                u[2 * k] = __float_as_uint(uf.x);
                                u[2 * k + 1] = __float_as_uint(uf.y);
                                if (MU) {
                                    const float2 rq = __fadd2_rn(uf, nmagic2);              // q - Z, exact
                                    const float2 neps = __ffma2_rn(nstep2, rq, xh[v][k]);   // -(Step (q - Z) - v^)
                                    eneg = __ffma2_rn(neps, make_float2(mu8[2 * k], mu8[2 * k + 1]), eneg);
                                }
                            }
                            store_codes(orow + (size_t)idx * vec_bytes, u, K, p.bits, BYTES_OUT);
                        }
                    }
                } else {
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = tt + v * T;
                        if (v < V - 1 || idx < p.nvec) {
                            uint32_t u[8];
                            float mu8[8];
                            if (MU) load8(p.mu + (size_t)idx * 8, mu8);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const int c0 = code_generic(xh[v][k].x, q.inv, q.zp, qmax);
                                const int c1 = code_generic(xh[v][k].y, q.inv, q.zp, qmax);
                                u[2 * k] = (uint32_t)c0;
                                u[2 * k + 1] = (uint32_t)c1;
                                if (MU) {
                                    const float r0 = (float)((long long)c0 - (long long)q.zp);
                                    const float r1 = (float)((long long)c1 - (long long)q.zp);
                                    eneg.x = __fmaf_rn(__fmaf_rn(-q.step, r0, xh[v][k].x), mu8[2 * k], eneg.x);
                                    eneg.y = __fmaf_rn(__fmaf_rn(-q.step, r1, xh[v][k].y), mu8[2 * k + 1], eneg.y);
                                }
                            }
                            store_codes(orow + (size_t)idx * vec_bytes, u, 0u, p.bits, BYTES_OUT);
                        }
                    }
                }
                if (MU) {
                    const float eacc = -warp_sum(__fadd_rn(eneg.x, eneg.y));
                    if (wpt > 1) {
                        if (lane == 0) sm->rsum[parity][warp] = eacc;
                        named_bar_sync(1 + tm, T);
                        if (tt == 0) {
                            float tot = 0.0f;
                            for (int w2 = 0; w2 < wpt; ++w2) tot += sm->rsum[parity][tw0 + w2];
                            p.epsmu[row] = tot;
                            if (p.bias.out || p.bias.out_f32)
                                write_bias(row, tot, p.bias.in, p.bias.out, p.bias.out_f32, p.bias.bf16);
                        }
                    } else if (lane == 0) {
                        p.epsmu[row] = eacc;
                        if (p.bias.out || p.bias.out_f32)
                            write_bias(row, eacc, p.bias.in, p.bias.out, p.bias.out_f32, p.bias.bf16);
                    }
                }
                parity ^= 1;
                AWEQ_RQ_TRY_REFILL()
            }
            if (!early) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->empty[s]);
            }
        }
#undef AWEQ_RQ_TRY_REFILL
        if (!ok && lane == 0) {
            atomicExch(&sm->abort_flag, 1);
            if (p.st) atomicAdd(&p.st->wait_timeout, 1ull);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0 && sm->abort_flag) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) { }
    }
}


template <class D, int V, int NT, bool MU, bool BYTES_OUT>
static aweq_status rq_launch_one(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    auto kern = rowquant_kernel<D, V, NT, MU, BYTES_OUT>;
    AWEQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    AWEQ_LAUNCH(kern, dim3(pl.grid), dim3(NT), pl.smem, stream, p);
    return AWEQ_OK;
}

template <class D, bool MU, bool BYTES_OUT>
static aweq_status rq_launch_v(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
#define AWEQ_RQ_CASE(v)                                                                      \
    case v:                                                                                  \
        return pl.NT == 512 ? rq_launch_one<D, v, 512, MU, BYTES_OUT>(p, pl, stream)         \
                            : rq_launch_one<D, v, 256, MU, BYTES_OUT>(p, pl, stream);
    switch (pl.V) {
        AWEQ_RQ_CASE(1) AWEQ_RQ_CASE(2) AWEQ_RQ_CASE(3) AWEQ_RQ_CASE(4) AWEQ_RQ_CASE(5)
        AWEQ_RQ_CASE(6) AWEQ_RQ_CASE(7) AWEQ_RQ_CASE(8) AWEQ_RQ_CASE(9) AWEQ_RQ_CASE(10)
    }
#undef AWEQ_RQ_CASE
    return AWEQ_ERR_UNSUPPORTED;
}

// mode: 0 = activations (one byte per code), 1 = weights with eps.mu sums, 2 = weights without
template <class D>
static aweq_status rq_launch(const RowQuantParams &p, const RowQuantPlan &pl, int mode, cudaStream_t stream)
{
    if (mode == 0) return rq_launch_v<D, false, true>(p, pl, stream);
    if (mode == 1) return rq_launch_v<D, true, false>(p, pl, stream);
    return rq_launch_v<D, false, false>(p, pl, stream);
}

aweq_status run_rowquant_wide(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream);
// rows of step 6 beyond 24576 channels, each shared by a cluster of two CTAs (rowquant_cluster.cu)
bool plan_rowquant_cluster(long long nrows, long long cols, RowQuantPlan *out);
aweq_status run_rowquant_cluster(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream);
aweq_status rq_launch_f16(const RowQuantParams &p, const RowQuantPlan &pl, int mode, cudaStream_t stream);
aweq_status rq_launch_bf16(const RowQuantParams &p, const RowQuantPlan &pl, int mode, cudaStream_t stream);

}  // namespace aweq
