// Host side of the row quantisers: which kernel takes a row width (plain loads; for step 6 beyond
// 36864 channels the cluster pair) and what the plan query reports for it.
#include "rowdirect_impl.cuh"

namespace aweq {

// widest row any of the row quantisers takes
constexpr long long kRowQuantMaxCols = 40960;

bool rowquant_supported(long long nrows, long long cols)
{
    return nrows >= 1 && cols >= 8 && cols <= kRowQuantMaxCols;
}

bool rowquant_describe(long long rows, long long cols, bool weights, long long plan[8])
{
    RowQuantPlan pl;
    int tw = 0, dv = 0;
    if (plan_rowdirect(cols, weights, &tw, &dv)) {
        // the plain-load kernel: no stages; teams take rows one by one
        const int teams = rd_threads(tw) / (tw * 32), per_sm = rd_ctas_per_sm(tw, dv, !weights);
        long long grid = (rows + teams - 1) / teams;
        if (grid > (long long)kSmCount * per_sm) grid = (long long)kSmCount * per_sm;
        plan[0] = grid < 1 ? 1 : grid; plan[1] = rd_threads(tw); plan[2] = (long long)sizeof(RdSmem); plan[3] = tw * 32;
        plan[4] = dv; plan[5] = 0; plan[6] = 0; plan[7] = 2;
        return true;
    }
    if (weights || !plan_rowquant_cluster(rows, cols, &pl)) return false;
    plan[0] = pl.grid; plan[1] = pl.NT; plan[2] = (long long)pl.smem; plan[3] = pl.team; plan[4] = pl.V;
    plan[5] = pl.rows_per_stage; plan[6] = pl.stages; plan[7] = 3;
    return true;
}

// weights == true: packed bit stream + optional eps.mu sums; false: one byte per code
aweq_status run_rowquant(const void *X, aweq_dtype dt, long long nrows, long long cols, long long ld,
                         const float *scale, const float *mu, int bits, bool weights, unsigned char *out,
                         float *step, int *zp, float *epsmu, const BiasIO &bias, aweq_dev_status *st,
                         cudaStream_t stream)
{
    RowQuantPlan pl = {};
    int tw = 0, dv = 0;
    const bool direct = plan_rowdirect(cols, weights, &tw, &dv);
    const bool pair = !direct && !weights && plan_rowquant_cluster(nrows, cols, &pl);
    if (!direct && !pair) return AWEQ_ERR_SHAPE;
    RowQuantParams p;
    p.X = reinterpret_cast<const uint16_t *>(X);
    p.nrows = nrows; p.ld = ld; p.nvec = (int)(cols / 8);
    p.scale = scale; p.mu = mu; p.out = out;
    p.out_pitch = weights ? cols * bits / 8 : cols;
    p.step = step; p.zp = zp; p.epsmu = epsmu; p.bits = bits; p.bias = bias;
    p.team = pl.team; p.rows_per_stage = pl.rows_per_stage; p.stages = pl.stages; p.ntiles = pl.ntiles;
    p.st = st;
    const int mode = !weights ? 0 : ((mu && epsmu) ? 1 : 2);
    if (direct) return run_rowdirect(p, tw, dv, mode, dt, stream);
    return run_rowquant_cluster(p, pl, dt, stream);
}

}  // namespace aweq
