// Host side of the direct (plain-load) row quantiser: which rows it takes and the dispatch
// to its instantiations.
#include "rowdirect_impl.cuh"
#include "kernels.h"

namespace aweq {

// Weight matrices always take this kernel: the smallest team (1, 2, 4 or 8 warps) whose threads
// hold the row in at most ten vectors each; beyond 20480 columns a whole CTA of 32 warps with at
// most five vectors per thread.  The per-token quantiser of step 6 takes it for rows of up to
// 36864 columns, with at most nine vectors per thread because a team has the loads of its next
// row in flight while it reduces and quantises the current one; teams of up to 16 warps (a CTA
// of 512 threads, one per SM).  With that it measured faster than the shared-memory-staged
// kernels it replaced at every width (36864 columns: 6.14 against 5.23 TB/s).
bool plan_rowdirect(long long cols, bool weights, int *team_warps, int *V)
{
    const int nvec = (int)(cols / 8);
    if (!weights) {
        // step 6: the smallest team (up to a CTA of 16 warps) that holds the row with at most nine vectors per thread
        for (int tw = 1; tw <= kRdActMaxTeamWarps; tw *= 2) {
            const int v = (nvec + tw * 32 - 1) / (tw * 32);
            if (v <= kRdActMaxV) {
                *team_warps = tw;
                *V = v;
                return true;
            }
        }
        return false;
    }
    for (int tw = 1; tw <= 8; tw *= 2) {
        const int v = (nvec + tw * 32 - 1) / (tw * 32);
        if (v <= kRqMaxV) {
            *team_warps = tw;
            *V = v;
            return true;
        }
    }
    const int v = (nvec + 1023) / 1024;
    if (v <= 5) {
        *team_warps = 32;
        *V = v;
        return true;
    }
    return false;
}

aweq_status run_rowdirect(const RowQuantParams &p, int team_warps, int V, int mode, aweq_dtype dt, cudaStream_t stream)
{
    return dt == AWEQ_F16 ? rd_launch_f16(p, team_warps, V, mode, stream) : rd_launch_bf16(p, team_warps, V, mode, stream);
}

}  // namespace aweq
