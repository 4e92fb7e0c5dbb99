// Per-token quantiser of step 6 (8-bit codes of X^ = X diag(s)^-1, Eq. 1-3), tile form.
//
// Where the register-resident row quantiser (rowquant_impl.cuh) gives a row to a team of
// warps that keeps it in registers, this kernel gives a TILE of R rows to the whole CTA and
// reads it twice from the shared-memory stage the bulk copy (TMA) filled:
//   pass 1  x^ = x * (1/s), running min / max of every row of the tile
//   reduce  warp redux -> a few words of shared memory -> ONE THREAD per row forms Step,
//           1/Step, Z (Eq. 2) and writes them (coalesced) -- not one warp per row
//   pass 2  x^ again, codes (Eq. 1), 8-byte coalesced stores
// The CTA is G groups of W threads; group g takes rows g, g + G, ... of the tile and thread c
// of a group owns the column vectors c, c + W, ... (V <= 5 of them) of EVERY row, so the
// factors 1/s of its columns are loaded once per kernel and stay in registers (with 1024
// threads, 64 registers each, those of the fourth and fifth vector sit in shared memory).
// What this buys over the register-resident form: the per-row work that every warp of a team
// repeated (exchange, Step, Z: ~90 instructions) shrinks to two redux and one store per
// warp and row, the factors are never re-read (a 36864-channel factor vector is 147 KB, more
// than L1 keeps beside the stages), and there are two CTA barriers per tile, not per row.
// Tiles arrive through a ring of two (three) stages; warp 0 issues the next tile at the top
// of each iteration.  Every wait is bounded.
#include "rowquant_impl.cuh"

namespace aweq {

constexpr int kRtHeader = 8192;
constexpr int kRtMaxRows = 64;         // rows per tile
constexpr int kRtMaxRed = 512;         // (row, warp-of-group) partials per tile

struct RtSmem {
    RqSmem ring;                       // full / empty barriers, abort flag
    float4 q[kRtMaxRows];              // Step, 1/Step, Z (bits), flags (bits)
    float2 red[kRtMaxRed];             // [row][warp of the row's group]: (lo, hi)
};
static_assert(sizeof(RtSmem) <= kRtHeader, "header");

// vectors per thread whose factors live in registers; the rest (1024-thread shape only) in shared memory
__host__ __device__ constexpr int rt_reg_vectors(int V, int NT) { return NT == 1024 && V > 3 ? 3 : V; }
__host__ __device__ constexpr size_t rt_scale_smem(int V, int NT) { return (size_t)(V - rt_reg_vectors(V, NT)) * NT * 32; }

template <class D, int V, int NT, int RPG>
__global__ void __launch_bounds__(NT, 1) rowquant_tile_kernel(const RowQuantParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RtSmem *sm = reinterpret_cast<RtSmem *>(smem_raw);
    constexpr int VR = rt_reg_vectors(V, NT);
    float4 *ssc = reinterpret_cast<float4 *>(smem_raw + kRtHeader);       // [(v - VR) * 2 + half][thread]
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw + kRtHeader + rt_scale_smem(V, NT));
    constexpr int NW = NT / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int W = NT == 1024 ? NT : p.team;        // threads per row (a multiple of 32; the 1024-thread shape has one group)
    const int G = NT / W;                          // row groups
    const int g = threadIdx.x / W, col = threadIdx.x - g * W;
    const int wpg = W / 32, wig = col >> 5;        // warps per group, my warp within the group
    const int R = p.rows_per_stage, S = p.stages;
    const size_t stage_vecs = (size_t)R * p.nvec;
    const int qmax = (1 << p.bits) - 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sm->ring.full[s], 1);
            mbar_init(&sm->ring.empty[s], NW);
        }
        sm->ring.abort_flag = 0;
        mbar_init_fence();
    }
    pdl_begin();
    __syncthreads();

    const long long my_tiles = p.ntiles > blockIdx.x ? (p.ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    long long next_issue = 0;
    if (warp == 0)
        for (; next_issue < S - 1 && next_issue < my_tiles; ++next_issue)
            rq_issue_tile(p, &sm->ring, stage_base, next_issue, S, R, stage_vecs, lane);

    // the factors of this thread's columns (no equalisation = ones, which is exact)
    float2 sc[VR][4];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int idx = col + v * W;
        float4 s0 = make_float4(1.0f, 1.0f, 1.0f, 1.0f), s1 = s0;
        if (p.scale && idx < p.nvec) {
            s0 = ldg_f4(p.scale + (size_t)idx * 8);
            s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
        }
        if (v < VR) {
            sc[v < VR ? v : 0][0] = make_float2(s0.x, s0.y); sc[v < VR ? v : 0][1] = make_float2(s0.z, s0.w);
            sc[v < VR ? v : 0][2] = make_float2(s1.x, s1.y); sc[v < VR ? v : 0][3] = make_float2(s1.z, s1.w);
        } else {                                   // only this thread reads these back
            ssc[((v - VR) * 2 + 0) * NT + threadIdx.x] = s0;
            ssc[((v - VR) * 2 + 1) * NT + threadIdx.x] = s1;
        }
    }
#define AWEQ_RT_SCALES(v, f)                                                           \
    float2 f[4];                                                                       \
    if (v < VR) {                                                                      \
        f[0] = sc[v < VR ? v : 0][0]; f[1] = sc[v < VR ? v : 0][1];                    \
        f[2] = sc[v < VR ? v : 0][2]; f[3] = sc[v < VR ? v : 0][3];                    \
    } else {                                                                           \
        const float4 a = ssc[((v - VR) * 2 + 0) * NT + threadIdx.x];                   \
        const float4 b = ssc[((v - VR) * 2 + 1) * NT + threadIdx.x];                   \
        f[0] = make_float2(a.x, a.y); f[1] = make_float2(a.z, a.w);                    \
        f[2] = make_float2(b.x, b.y); f[3] = make_float2(b.z, b.w);                    \
    }

    bool ok = true;
    for (long long k = 0; k < my_tiles; ++k) {
        if (warp == 0 && next_issue < my_tiles) {
            // tile k + S - 1 goes into the stage that tile k - 1 released
            bool timed_out = false;
            if (rq_stage_free(&sm->ring, next_issue, S, true, &timed_out)) {
                rq_issue_tile(p, &sm->ring, stage_base, next_issue, S, R, stage_vecs, lane);
                ++next_issue;
            }
            if (timed_out) ok = false;
        }
        const int s = (int)(k % S);
        const uint32_t use = (uint32_t)(k / S);
        ok = ok && mbar_wait(&sm->ring.full[s], use & 1);
        const long long row0 = (blockIdx.x + k * gridDim.x) * (long long)R;
        const int rows = (int)min((long long)R, p.nrows - row0);
        const uint4 *tile = stage_base + (size_t)s * stage_vecs;

        // ---- pass 1: extremes of my group's rows (scaled)
        float lo[RPG], hi[RPG];
#pragma unroll
        for (int i = 0; i < RPG; ++i) { lo[i] = INFINITY; hi[i] = -INFINITY; }
        if (ok) {
#pragma unroll
            for (int i = 0; i < RPG; ++i) {
                const int r = g + i * G;
                if (r < rows) {
                    const uint4 *rowp = tile + (size_t)r * p.nvec;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = col + v * W;
                        if (v < V - 1 || idx < p.nvec) {
                            const uint4 raw = rowp[idx];
                            const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
                            AWEQ_RT_SCALES(v, f)
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w4[c])), f[c]);
                                lo[i] = fminf(fminf(lo[i], x.x), x.y);
                                hi[i] = fmaxf(fmaxf(hi[i], x.x), x.y);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < RPG; ++i) {
            const int r = g + i * G;
            if (r < rows) {
                const float l = redux_min(lo[i], 0xffffffffu), h = redux_max(hi[i], 0xffffffffu);
                if (lane == 0) sm->red[r * wpg + wig] = make_float2(l, h);
            }
        }
        // the barrier doubles as the agreement on a timed-out wait: everybody leaves or nobody
        ok = __syncthreads_and(ok);
        if (!ok) break;
        // ---- one thread per row: Step, 1 / Step, Z
        if ((int)threadIdx.x < rows) {
            const int r = threadIdx.x;
            float l = INFINITY, h = -INFINITY;
            for (int w2 = 0; w2 < wpg; ++w2) {
                const float2 o = sm->red[r * wpg + w2];
                l = fminf(l, o.x);
                h = fmaxf(h, o.y);
            }
            const QParams q = make_qparams(l, h, qmax);
            const int fl = qflags(q, h, qmax);
            sm->q[r] = make_float4(q.step, q.inv, __int_as_float(q.zp), __int_as_float(fl));
            p.step[row0 + r] = q.step;
            p.zp[row0 + r] = q.zp;
        }
        __syncthreads();

        // ---- pass 2: codes
#pragma unroll
        for (int i = 0; i < RPG; ++i) {
            const int r = g + i * G;
            if (r < rows) {
                const float4 qv = sm->q[r];
                const float inv = qv.y;
                const int zp = __float_as_int(qv.z), fl = __float_as_int(qv.w);
                const uint4 *rowp = tile + (size_t)r * p.nvec;
                unsigned char *orow = p.out + (row0 + r) * p.out_pitch;
                const bool lean = fl == (kQFast | kQNoClamp);
                const uint32_t K = (uint32_t)(zp - kMagicBits);
                const float2 inv2 = make_float2(inv, inv), magic2 = make_float2(kMagic, kMagic);
                const float2 one2 = make_float2(1.0f, 1.0f);
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int idx = col + v * W;
                    if (v < V - 1 || idx < p.nvec) {
                        const uint4 raw = rowp[idx];
                        const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
                        uint32_t u[8];
                        AWEQ_RT_SCALES(v, f)
                        if (lean) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w4[c])), f[c]);
                                const float2 t = __fmul2_rn(x, inv2);
                                // t * 1 + magic as one FMA: equal to t + magic, and it cannot be
                                // contracted with the multiply above (which would change ties)
                                const float2 uf = __ffma2_rn(t, one2, magic2);
                                u[2 * c] = __float_as_uint(uf.x);
                                u[2 * c + 1] = __float_as_uint(uf.y);
                            }
                            store_codes(orow + (size_t)idx * 8, u, K, p.bits, true);
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w4[c])), f[c]);
                                u[2 * c] = (uint32_t)code_generic(x.x, inv, zp, qmax);
                                u[2 * c + 1] = (uint32_t)code_generic(x.y, inv, zp, qmax);
                            }
                            store_codes(orow + (size_t)idx * 8, u, 0u, p.bits, true);
                        }
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm->ring.empty[s]);
    }
#undef AWEQ_RT_SCALES
    if (!ok && threadIdx.x == 0) {
        if (p.st) atomicAdd(&p.st->wait_timeout, 1ull);
        // copies that were already requested may still land in this CTA's shared memory
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) { }
    }
    __syncthreads();
}

// Shape of the CTA for a row of nvec vectors: NT threads as G groups of W, V vectors per thread.
// Cost of a row in issue slots ~ (W / 32) * (V * c_vec + c_warp); lanes beyond the row's end
// (V * W > nvec) are paid for in full, so the shapes are ranked by that product first.
bool plan_rowquant_tile(long long nrows, long long cols, RowQuantPlan *out)
{
    const int nvec = (int)(cols / 8);
    if (nvec < 1 || nvec > 5 * 1024) return false;
    static const int kNT[3] = {512, 384, 1024};
    double best = 1e30;
    RowQuantPlan bp = {};
    const size_t row_bytes = (size_t)nvec * 16;
    for (int a = 0; a < 3; ++a) {
        const int NT = kNT[a];
        for (int W = 32; W <= NT; W += 32) {
            if (NT % W) continue;
            const int V = (nvec + W - 1) / W;
            if (V > 5) continue;
            if (NT == 1024 && (V < 3 || W != NT)) continue;          // instantiated for the widest rows only
            const int G = NT / W;
            const size_t budget = 226 * 1024 - kRtHeader - rt_scale_smem(V, NT);
            const int rpg_max = NT == 1024 ? 4 : 16;
            int S = 2;
            long long Rfit = (long long)(budget / (2 * row_bytes));
            int rpg = (int)(Rfit / G);
            if (rpg > rpg_max) rpg = rpg_max;
            if (rpg * G > kRtMaxRows) rpg = kRtMaxRows / G;
            if (rpg * G * (W / 32) > kRtMaxRed) rpg = kRtMaxRed / (G * (W / 32));
            if (rpg < 1) {
                if (G > 1) continue;
                rpg = 1;
                S = (int)(budget / row_bytes);
                if (S < 2) continue;
            } else if (G == 1 && rpg == 1) {
                S = (int)(budget / row_bytes);                        // a third stage when it fits
            }
            if (S > kRqStagesMax) S = kRqStagesMax;
            const int R = rpg * G;
            // issue slots per row, plus the two barriers of a tile spread over its rows
            const double cost = (W / 32) * (V * 56.0 + 8.0) + 2.0 + 600.0 / R + (NT == 1024 ? 0.15 : 0.0) * V * W / 32 * 56.0;
            if (cost < best - 1e-9) {
                best = cost;
                bp.NT = NT; bp.team = W; bp.V = V; bp.rows_per_stage = R; bp.stages = S;
                bp.smem = kRtHeader + rt_scale_smem(V, NT) + (size_t)S * R * row_bytes;
            }
        }
    }
    if (best > 1e29) return false;
    if ((long long)bp.rows_per_stage > nrows) {
        const int G = bp.NT / bp.team;
        bp.rows_per_stage = (int)((nrows + G - 1) / G * G);
    }
    bp.ntiles = (nrows + bp.rows_per_stage - 1) / bp.rows_per_stage;
    long long gsz = kSmCount;
    if (gsz > bp.ntiles) gsz = bp.ntiles;
    bp.grid = (int)(gsz < 1 ? 1 : gsz);
    *out = bp;
    return true;
}

template <class D, int V, int NT, int RPG>
static aweq_status rt_launch_one(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    auto kern = rowquant_tile_kernel<D, V, NT, RPG>;
    AWEQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    AWEQ_LAUNCH(kern, dim3(pl.grid), dim3(NT), pl.smem, stream, p);
    return AWEQ_OK;
}

template <class D>
static aweq_status rt_launch(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
#define AWEQ_RT_CASE(v)                                                                        \
    case v:                                                                                    \
        if (pl.NT == 512) return rt_launch_one<D, v, 512, 16>(p, pl, stream);                  \
        if (pl.NT == 384) return rt_launch_one<D, v, 384, 16>(p, pl, stream);                  \
        break;
    switch (pl.V) { AWEQ_RT_CASE(1) AWEQ_RT_CASE(2) AWEQ_RT_CASE(3) AWEQ_RT_CASE(4) AWEQ_RT_CASE(5) }
#undef AWEQ_RT_CASE
    if (pl.NT == 1024) {
        if (pl.V == 3) return rt_launch_one<D, 3, 1024, 4>(p, pl, stream);
        if (pl.V == 4) return rt_launch_one<D, 4, 1024, 4>(p, pl, stream);
        if (pl.V == 5) return rt_launch_one<D, 5, 1024, 4>(p, pl, stream);
    }
    return AWEQ_ERR_UNSUPPORTED;
}

aweq_status run_rowquant_tile(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream)
{
    return dt == AWEQ_F16 ? rt_launch<F16>(p, pl, stream) : rt_launch<BF16>(p, pl, stream);
}

}  // namespace aweq
