// Per-token quantiser of step 6 for wide rows (12288 to 24576 channels; narrower rows go through
// the plain-load kernel, wider ones through the cluster pair of rowquant_cluster.cu).
//
// A row that no longer fits the registers of a few warps needs a whole team of warps, and then
// every row costs a team-wide exchange.  Here the whole CTA (512 or 768 threads) works on a
// tile of R rows at a time; a thread owns the same V <= 5 column vectors in every row, so their
// factors stay in registers for the whole kernel, and the rows are read twice from shared
// memory instead of being kept in registers:
//   pass 1  x^ = x * (1/s), running min / max of each of the R rows     (no global loads)
//   reduce  warp redux -> shared -> warp r finishes row r: Step, 1/Step, Z (Eq. 2)
//   pass 2  x^ again, codes (Eq. 1), 8-byte coalesced stores
// with two CTA-wide barriers per tile of R rows rather than per row.  Tiles arrive through a
// ring of bulk-copy (TMA) stages; warp 0 issues the next tile at the top of each iteration.
// Every wait is bounded.
#include "rowquant_impl.cuh"

namespace aweq {

constexpr int kRwMaxR = 4;
constexpr int kRwHeader = 4096;

struct RwSmem {
    RqSmem ring;                       // full / empty barriers, abort flag
    float2 red[32][kRwMaxR];           // per-warp (lo, hi) of each row of the tile
    float4 q[kRwMaxR];                 // Step, 1/Step, Z (bits), flags (bits)
};
static_assert(sizeof(RwSmem) <= kRwHeader, "header");

template <class D, int V, int NT>
__global__ void __launch_bounds__(NT, 1) rowquant_wide_kernel(const RowQuantParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RwSmem *sm = reinterpret_cast<RwSmem *>(smem_raw);
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw + kRwHeader);
    constexpr int NW = NT / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
    float2 sc[V][4];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int idx = threadIdx.x + v * NT;
        float4 s0 = make_float4(1.0f, 1.0f, 1.0f, 1.0f), s1 = s0;
        if (p.scale && idx < p.nvec) {
            s0 = ldg_f4(p.scale + (size_t)idx * 8);
            s1 = ldg_f4(p.scale + (size_t)idx * 8 + 4);
        }
        sc[v][0] = make_float2(s0.x, s0.y); sc[v][1] = make_float2(s0.z, s0.w);
        sc[v][2] = make_float2(s1.x, s1.y); sc[v][3] = make_float2(s1.z, s1.w);
    }
#define AWEQ_RW_SCALES(v, f) const float2 (&f)[4] = sc[v];

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

        // ---- pass 1: extremes of the scaled rows
        float lo[kRwMaxR], hi[kRwMaxR];
#pragma unroll
        for (int r = 0; r < kRwMaxR; ++r) { lo[r] = INFINITY; hi[r] = -INFINITY; }
        if (ok) {
#pragma unroll
            for (int r = 0; r < kRwMaxR; ++r) {
                if (r < rows) {
                    const uint4 *rowp = tile + (size_t)r * p.nvec;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = threadIdx.x + v * NT;
                        if (v < V - 1 || idx < p.nvec) {
                            const uint4 raw = rowp[idx];
                            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                            AWEQ_RW_SCALES(v, f)
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), f[c]);
                                lo[r] = fmin3(lo[r], x.x, x.y);
                                hi[r] = fmax3(hi[r], x.x, x.y);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kRwMaxR; ++r) {
            if (r < rows) {
                const float l = redux_min(lo[r], 0xffffffffu), h = redux_max(hi[r], 0xffffffffu);
                if (lane == 0) sm->red[warp][r] = make_float2(l, h);
            }
        }
        // the barrier doubles as the agreement on a timed-out wait: everybody leaves or nobody
        ok = __syncthreads_and(ok);
        if (!ok) break;
        if (warp < rows) {
            const float2 o = lane < NW ? sm->red[lane][warp] : make_float2(INFINITY, -INFINITY);
            const float l = redux_min(o.x, 0xffffffffu), h = redux_max(o.y, 0xffffffffu);
            const QParams q = make_qparams(l, h, qmax);
            const int fl = qflags(q, h, qmax);
            if (lane == 0) {
                sm->q[warp] = make_float4(q.step, q.inv, __int_as_float(q.zp), __int_as_float(fl));
                p.step[row0 + warp] = q.step;
                p.zp[row0 + warp] = q.zp;
            }
        }
        __syncthreads();

        // ---- pass 2: codes
#pragma unroll
        for (int r = 0; r < kRwMaxR; ++r) {
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
                    const int idx = threadIdx.x + v * NT;
                    if (v < V - 1 || idx < p.nvec) {
                        const uint4 raw = rowp[idx];
                        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                        uint32_t u[8];
                        AWEQ_RW_SCALES(v, f)
                        if (lean) {
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), f[c]);
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
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), f[c]);
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
#undef AWEQ_RW_SCALES
    if (!ok && threadIdx.x == 0) {
        if (p.st) atomicAdd(&p.st->wait_timeout, 1ull);
        // copies that were already requested may still land in this CTA's shared memory
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) { }
    }
    __syncthreads();
}

bool plan_rowquant_wide(long long nrows, long long cols, RowQuantPlan *out)
{
    const int nvec = (int)(cols / 8);
    if (nvec <= 1536 || nvec > 4 * 768) return false;
    RowQuantPlan p;
    // up to 20480 columns 512 threads with four or five vectors each; 20481 .. 24576 columns 768 threads
    // with four vectors each, which keeps two rows per stage
    p.NT = nvec <= 5 * 512 ? 512 : 768;
    p.team = p.NT;
    p.V = (nvec + p.NT - 1) / p.NT;
    const size_t row_bytes = (size_t)nvec * 16;
    const size_t budget = 226 * 1024 - kRwHeader;
    int S = 2;
    int R = (int)(budget / (2 * row_bytes));
    if (R > kRwMaxR) R = kRwMaxR;
    if (R < 1) {
        R = 1;
        S = (int)(budget / row_bytes);
        if (S < 2) return false;
    } else if (R == 1) {
        S = (int)(budget / row_bytes);               // a third stage when it fits
    }
    if (S > kRqStagesMax) S = kRqStagesMax;
    if ((long long)R > nrows) R = (int)nrows;
    p.rows_per_stage = R;
    p.stages = S;
    p.smem = kRwHeader + (size_t)S * R * row_bytes;
    p.ntiles = (nrows + R - 1) / R;
    long long g = kSmCount;
    if (g > p.ntiles) g = p.ntiles;
    p.grid = (int)(g < 1 ? 1 : g);
    *out = p;
    return true;
}

template <class D, int V, int NT>
static aweq_status rw_launch_one(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    auto kern = rowquant_wide_kernel<D, V, NT>;
    AWEQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    AWEQ_LAUNCH(kern, dim3(pl.grid), dim3(NT), pl.smem, stream, p);
    return AWEQ_OK;
}

template <class D>
static aweq_status rw_launch(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    if (pl.NT == 768 && pl.V == 4) return rw_launch_one<D, 4, 768>(p, pl, stream);
    if (pl.NT == 512 && pl.V == 4) return rw_launch_one<D, 4, 512>(p, pl, stream);
    if (pl.NT == 512 && pl.V == 5) return rw_launch_one<D, 5, 512>(p, pl, stream);
    return AWEQ_ERR_UNSUPPORTED;
}

aweq_status run_rowquant_wide(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream)
{
    return dt == AWEQ_F16 ? rw_launch<F16>(p, pl, stream) : rw_launch<BF16>(p, pl, stream);
}

}  // namespace aweq
