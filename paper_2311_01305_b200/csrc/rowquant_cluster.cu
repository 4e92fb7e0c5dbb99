// Per-token quantiser of step 6 for the widest rows (more than 36864 channels, where the plain-load
// kernel would need ten vectors per thread and spills): a row is shared by the two CTAs of a
// thread-block cluster.
//
// A row of 40960 fp16 channels is 80 KB.  With one CTA per row only one row fits a stage of a
// bulk-copy ring, the CTA needs 1024 threads, and the factors of its columns do not all fit
// in registers.  Here the two CTAs of a cluster (two SMs) each take half of the columns of the
// same rows: 512 threads, five 16-byte vectors per thread, every factor in registers, tiles of
// two half-rows per stage, which the whole CTA reads twice from shared memory (extremes, then
// codes) with two CTA-wide barriers per tile.  What the two halves must share is
// the pair of extremes of every row (Eq. 2 needs max and min over the whole row): after the first
// pass a warp per row writes the CTA's (lo, hi) into its own and, through distributed shared
// memory, into the peer's exchange slot and arrives on both CTAs' exchange barrier; one lane of every
// warp waits (bounded) for the eight arrivals of the tile, and every thread forms Step, 1/Step and Z from
// the two halves' extremes itself and runs the second pass on its half.  The CTAs of a pair run the same
// tiles in the same order, so the exchange needs no further hand-shake: a slot of parity k & 1 is
// rewritten for tile k + 2 only after its owner has sent its extremes of tile k + 1, which it
// does after reading the slot for tile k.
//
// Waits are bounded as everywhere in this library: a CTA whose wait gives up stops working and
// says so; its peer then runs into the limit of its own wait.  Both reach the cluster-wide
// barrier at the end of the kernel, which keeps a CTA's shared memory alive while the peer may
// still write to it.
#include <mutex>
#include "rowquant_impl.cuh"

namespace aweq {

constexpr int kRcThreads = 512;
constexpr int kRcMaxR = 4;
constexpr int kRcHeader = 4096;
constexpr int kRcStages = 2;

struct RcSmem {
    RqSmem ring;                          // full / empty barriers of the stages, abort flag
    float2 red[kRcThreads / 32][kRcMaxR]; // per-warp (lo, hi) of each row of the tile (this CTA's half)
    float2 xch[2][2][kRcMaxR];            // [tile parity][CTA rank][row]: each half's (lo, hi)
    uint64_t xbar[2];                     // [tile parity]: 4 local + 4 remote arrivals per tile
};
static_assert(sizeof(RcSmem) <= kRcHeader, "header");

template <class D, int V>
__global__ void __launch_bounds__(kRcThreads, 1) rowquant_cluster_kernel(const RowQuantParams p)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    RcSmem *sm = reinterpret_cast<RcSmem *>(smem_raw);
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw + kRcHeader);
    constexpr int NT = kRcThreads, NW = NT / 32, S = kRcStages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(), peer = rank ^ 1u;
    const int R = p.rows_per_stage;
    const int half0 = (p.nvec + 1) / 2;
    const int off = rank ? half0 : 0;                     // first vector of my half
    const int myvec = rank ? p.nvec - half0 : half0;      // vectors of my half
    const size_t stage_vecs = (size_t)R * half0;
    const int qmax = (1 << p.bits) - 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&sm->ring.full[s], 1);
            mbar_init(&sm->ring.empty[s], NW);
        }
        mbar_init(&sm->xbar[0], 2 * kRcMaxR);
        mbar_init(&sm->xbar[1], 2 * kRcMaxR);
        sm->ring.abort_flag = 0;
        mbar_init_fence();
    }
    pdl_begin();
    cluster_sync_all();                  // the peer's barriers exist before anybody arrives on them

    const long long cid = blockIdx.x >> 1, ncl = gridDim.x >> 1;
    const long long my_tiles = p.ntiles > cid ? (p.ntiles - cid + ncl - 1) / ncl : 0;
    long long next_issue = 0;
    // warp 0: copy my half of the rows of tile t into its stage, one bulk copy per row
    auto issue = [&](long long t) {
        const int s = (int)(t % S);
        const long long row0 = (cid + t * ncl) * (long long)R;
        const int rows = (int)min((long long)R, p.nrows - row0);
        uint4 *dst = stage_base + (size_t)s * stage_vecs;
        if (lane == 0) mbar_arrive_expect_tx(&sm->ring.full[s], (uint32_t)rows * (uint32_t)myvec * 16u);
        __syncwarp();
        for (int r = lane; r < rows; r += 32)
            bulk_g2s(dst + (size_t)r * half0, p.X + (row0 + r) * p.ld + (long long)off * 8, (uint32_t)myvec * 16u,
                     &sm->ring.full[s]);
    };
    if (warp == 0)
        for (; next_issue < S - 1 && next_issue < my_tiles; ++next_issue) issue(next_issue);

    // the factors of this thread's columns (no equalisation = ones, which is exact)
    float2 sc[V][4];
#pragma unroll
    for (int v = 0; v < V; ++v) {
        const int idx = threadIdx.x + v * NT;
#pragma unroll
        for (int k = 0; k < 4; ++k) sc[v][k] = make_float2(1.0f, 1.0f);
        if (p.scale && idx < myvec) {
            const float4 s0 = ldg_f4(p.scale + (size_t)(off + idx) * 8), s1 = ldg_f4(p.scale + (size_t)(off + idx) * 8 + 4);
            sc[v][0] = make_float2(s0.x, s0.y); sc[v][1] = make_float2(s0.z, s0.w);
            sc[v][2] = make_float2(s1.x, s1.y); sc[v][3] = make_float2(s1.z, s1.w);
        }
    }

    bool ok = true;
    for (long long k = 0; k < my_tiles; ++k) {
        if (warp == 0 && next_issue < my_tiles) {
            // tile k + S - 1 goes into the stage that tile k - 1 released
            bool timed_out = false;
            if (rq_stage_free(&sm->ring, next_issue, S, &timed_out)) {
                issue(next_issue);
                ++next_issue;
            }
            if (timed_out) ok = false;
        }
        const int s = (int)(k % S);
        ok = ok && mbar_wait(&sm->ring.full[s], (uint32_t)(k / S) & 1);
        const long long row0 = (cid + k * ncl) * (long long)R;
        const int rows = (int)min((long long)R, p.nrows - row0);
        const uint4 *tile = stage_base + (size_t)s * stage_vecs;
        const int par = (int)(k & 1);

        // ---- pass 1: extremes of my half of the scaled rows
        float lo[kRcMaxR], hi[kRcMaxR];
#pragma unroll
        for (int r = 0; r < kRcMaxR; ++r) { lo[r] = INFINITY; hi[r] = -INFINITY; }
        if (ok) {
#pragma unroll
            for (int r = 0; r < kRcMaxR; ++r) {
                if (r < rows) {
                    const uint4 *rowp = tile + (size_t)r * half0;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = threadIdx.x + v * NT;
                        if (v < V - 1 || idx < myvec) {
                            const uint4 raw = rowp[idx];
                            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), sc[v][c]);
                                lo[r] = fmin3(lo[r], x.x, x.y);
                                hi[r] = fmax3(hi[r], x.x, x.y);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int r = 0; r < kRcMaxR; ++r) {
            if (r < rows) {
                const float l = redux_min(lo[r], 0xffffffffu), h = redux_max(hi[r], 0xffffffffu);
                if (lane == 0) sm->red[warp][r] = make_float2(l, h);
            }
        }
        // the barrier doubles as the agreement on a wait that gave up: everybody leaves or nobody
        ok = __syncthreads_and(ok);
        if (!ok) break;
        // ---- exchange: warp r sends this CTA's extremes of row r to both CTAs of the pair
        if (warp < kRcMaxR) {
            if (warp < rows) {
                const float2 o = lane < NW ? sm->red[lane][warp] : make_float2(INFINITY, -INFINITY);
                const float l = redux_min(o.x, 0xffffffffu), h = redux_max(o.y, 0xffffffffu);
                if (lane == 0) {
                    sm->xch[par][rank][warp] = make_float2(l, h);
                    cluster_store_f2(cluster_map(&sm->xch[par][rank][warp], peer), l, h);
                }
            }
            if (lane == 0) {
                mbar_arrive(&sm->xbar[par]);
                cluster_mbar_arrive(cluster_map(&sm->xbar[par], peer));
            }
        }
        {
            // one lane per warp polls; the warp barrier hands what it acquired to the other lanes
            int got = 1;
            if (lane == 0) got = mbar_wait_cluster(&sm->xbar[par], (uint32_t)(k >> 1) & 1) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            __syncwarp();
            if (!got) ok = false;
        }

        // ---- pass 2: Step, 1/Step, Z of the whole row from the two halves' extremes; codes of my half
        if (ok) {
#pragma unroll
            for (int r = 0; r < kRcMaxR; ++r) {
                if (r < rows) {
                    const float2 e0 = sm->xch[par][0][r], e1 = sm->xch[par][1][r];
                    const float l = fminf(e0.x, e1.x), h = fmaxf(e0.y, e1.y);
                    const QParams q = make_qparams(l, h, qmax);
                    const bool lean = qflags(q, h, qmax) == (kQFast | kQNoClamp);
                    if (rank == 0 && threadIdx.x == r) {
                        p.step[row0 + r] = q.step;
                        p.zp[row0 + r] = q.zp;
                    }
                    const uint4 *rowp = tile + (size_t)r * half0;
                    unsigned char *orow = p.out + (row0 + r) * p.out_pitch + (size_t)off * 8;
                    const uint32_t K = (uint32_t)(q.zp - kMagicBits);
                    const float2 inv2 = make_float2(q.inv, q.inv), magic2 = make_float2(kMagic, kMagic);
                    const float2 one2 = make_float2(1.0f, 1.0f);
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const int idx = threadIdx.x + v * NT;
                        if (v < V - 1 || idx < myvec) {
                            const uint4 raw = rowp[idx];
                            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
                            uint32_t u[8];
                            if (lean) {
#pragma unroll
                                for (int c = 0; c < 4; ++c) {
                                    const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), sc[v][c]);
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
                                    const float2 x = __fmul2_rn(D::to_float2(D::from_bits(w[c])), sc[v][c]);
                                    u[2 * c] = (uint32_t)code_generic(x.x, q.inv, q.zp, qmax);
                                    u[2 * c + 1] = (uint32_t)code_generic(x.y, q.inv, q.zp, qmax);
                                }
                                store_codes(orow + (size_t)idx * 8, u, 0u, p.bits, true);
                            }
                        }
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm->ring.empty[s]);
    }
    if (!ok && threadIdx.x == 0) {
        if (p.st) atomicAdd(&p.st->wait_timeout, 1ull);
        // copies that were already requested may still land in this CTA's shared memory
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) { }
    }
    __syncthreads();
    cluster_sync_all();                  // nobody leaves while its peer may still write into its exchange slots
}

// Shape for a row width: two CTAs per row, 512 threads each, as many half-rows per stage (at most four)
// as two stages leave room for.  Needs an even split into whole vectors only in the sense that
// both halves are at most 2560 vectors.
bool plan_rowquant_cluster(long long nrows, long long cols, RowQuantPlan *out)
{
    const int nvec = (int)(cols / 8);
    if (nvec <= 4608 || nvec > 5120) return false;
    const int half0 = (nvec + 1) / 2;
    RowQuantPlan p;
    p.NT = kRcThreads;
    p.team = 2 * kRcThreads;
    p.V = (half0 + kRcThreads - 1) / kRcThreads;
    if (p.V > 5) return false;
    const size_t half_bytes = (size_t)half0 * 16;
    const size_t budget = 226 * 1024 - kRcHeader;
    int R = (int)(budget / (kRcStages * half_bytes));
    if (R < 1) return false;
    if (R > kRcMaxR) R = kRcMaxR;
    if ((long long)R > nrows) R = (int)nrows;
    p.rows_per_stage = R;
    p.stages = kRcStages;
    p.smem = kRcHeader + (size_t)kRcStages * R * half_bytes;
    p.ntiles = (nrows + R - 1) / R;
    long long clusters = kSmCount / 2;
    if (clusters > p.ntiles) clusters = p.ntiles;
    if (clusters < 1) clusters = 1;
    p.grid = (int)(2 * clusters);
    *out = p;
    return true;
}

template <class D, int V>
static aweq_status rc_launch_one(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    auto kern = rowquant_cluster_kernel<D, V>;
    AWEQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
    // A persistent grid must be resident as a whole (a cluster that starts after the others doubles
    // the run time): ask once how many clusters of this shape the device holds at the same time.
    static std::mutex lock;
    static size_t asked_smem = 0;
    static int asked_resident = 0;
    int resident;
    {
        std::lock_guard<std::mutex> hold(lock);
        if (asked_smem != pl.smem) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(pl.grid); cfg.blockDim = dim3(kRcThreads); cfg.dynamicSmemBytes = pl.smem;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            int nc = 0;
            AWEQ_CUDA_OK(cudaOccupancyMaxActiveClusters(&nc, kern, &cfg));
            asked_resident = nc;
            asked_smem = pl.smem;
        }
        resident = asked_resident;
    }
    int grid = pl.grid;
    if (resident > 0 && grid > 2 * resident) grid = 2 * resident;
    cudaError_t e = launch_pdl_cluster(kern, dim3(grid), dim3(kRcThreads), pl.smem, stream, 2u, p);
    note_launch();
    if (e != cudaSuccess) return cuda_failed(e);
    return AWEQ_OK;
}

template <class D>
static aweq_status rc_launch(const RowQuantParams &p, const RowQuantPlan &pl, cudaStream_t stream)
{
    switch (pl.V) {
    case 5: return rc_launch_one<D, 5>(p, pl, stream);
    }
    return AWEQ_ERR_UNSUPPORTED;
}

aweq_status run_rowquant_cluster(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream)
{
    return dt == AWEQ_F16 ? rc_launch<F16>(p, pl, stream) : rc_launch<BF16>(p, pl, stream);
}

}  // namespace aweq
