// Host side of the row quantiser: how a row is split over threads, how many rows
// form a stage, and the dispatch to the fp16 / bf16 instantiations.
#include "rowdirect_impl.cuh"

namespace aweq {

// Everything that happens once per row (exchange of the extremes, Step, 1/Step, Z) is
// repeated by every warp of the row's team, and a thread's last vector may be padding, so
// the cost of a row is about (T / 32) * (V * c_vec + c_row) issue slots.  Pick the team
// size that minimises it with V <= kRqMaxV.
static void pick_team(int nvec, int *T_out, int *V_out)
{
    double best = 1e30;
    int bestT = 0, bestV = 0;
    for (int T = 32; T <= 512; T *= 2) {
        const int V = (nvec + T - 1) / T;
        if (V > kRqMaxV) continue;
        const double c_vec = V <= kRqScaleRegsMaxV ? 55.0 : 59.0;
        const double cost = (T / 32) * (V * c_vec + 90.0);
        if (cost < best) { best = cost; bestT = T; bestV = V; }
    }
    *T_out = bestT;
    *V_out = bestV;
}

bool plan_rowquant(long long nrows, long long cols, RowQuantPlan *out)
{
    const int nvec = (int)(cols / 8);
    int T = 0, V = 0;
    pick_team(nvec, &T, &V);
    if (T == 0) return false;
    RowQuantPlan p;
    p.team = T;
    p.V = V;
    p.NT = T == 512 ? 512 : 256;
    const int teams = p.NT / T;
    const size_t row_bytes = (size_t)nvec * 16;
    const size_t budget = (p.NT == 512 ? 200 * 1024 : 100 * 1024) - kRqHeader;
    // rows per stage: about 32 KB, a multiple of the number of teams
    int R = (int)(32768 / row_bytes);
    R = R / teams * teams;
    if (R < teams) R = teams;
    if ((long long)R > nrows) R = (int)((nrows + teams - 1) / teams * teams);
    if (R < 1) R = 1;
    int S = (int)(budget / ((size_t)R * row_bytes));
    while (S < 2 && R > 1) {
        R = (R + 1) / 2;
        S = (int)(budget / ((size_t)R * row_bytes));
    }
    if (S < 2) return false;          // the ring needs two stages
    if (S > kRqStagesMax) S = kRqStagesMax;
    p.rows_per_stage = R;
    p.stages = S;
    p.smem = kRqHeader + (size_t)S * R * row_bytes;
    p.ntiles = (nrows + R - 1) / R;
    const int per_sm = p.NT == 512 ? 1 : 2;
    long long g = (long long)kSmCount * per_sm;
    if (g > p.ntiles) g = p.ntiles;
    if (g < 1) g = 1;
    p.grid = (int)g;
    *out = p;
    return true;
}

bool rowquant_supported(long long nrows, long long cols)
{
    RowQuantPlan pl;
    return plan_rowquant(nrows, cols, &pl);
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
    const bool pair = !weights && plan_rowquant_cluster(rows, cols, &pl);
    const bool wide = !pair && !weights && plan_rowquant_wide(rows, cols, &pl);
    if (!pair && !wide && !plan_rowquant(rows, cols, &pl)) return false;
    plan[0] = pl.grid; plan[1] = pl.NT; plan[2] = (long long)pl.smem; plan[3] = pl.team; plan[4] = pl.V;
    plan[5] = pl.rows_per_stage; plan[6] = pl.stages; plan[7] = pair ? 3 : wide ? 1 : 0;
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
    const bool wide = !direct && !pair && !weights && plan_rowquant_wide(nrows, cols, &pl);
    if (!direct && !pair && !wide && !plan_rowquant(nrows, cols, &pl)) return AWEQ_ERR_SHAPE;
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
    if (pair) return run_rowquant_cluster(p, pl, dt, stream);
    if (wide) return run_rowquant_wide(p, pl, dt, stream);
    return dt == AWEQ_F16 ? rq_launch_f16(p, pl, mode, stream) : rq_launch_bf16(p, pl, mode, stream);
}

}  // namespace aweq
