// Step 4 for groups of 128 input channels (the 4-bit / 3-bit, group-128 case): fold s into
// W (Eq. 3), Eq. 1-2 per group, pack, and the eps . E[x^] sums of Eq. 15, in one pass over W.
//
// A warp owns a window of 256 consecutive columns -- lane l holds the 16-byte vector of
// columns 8l .. 8l+7, lanes 0-15 are one group and lanes 16-31 the next -- and walks down the
// rows in batches of eight.  Because the window is fixed, the lane's eight factors s_j and
// E[x^]_j are loaded once and stay in registers.  Because a batch has 8 rows x 2 groups =
// 16 (Step, Z) pairs, lane o forms exactly one of them (row o / 2, group o % 2) instead of
// every lane repeating the scalar part of Eq. 2 for every row; the pairs come back to the
// lanes that need them by shuffle.  The eight loads of a batch are in flight together.
//
// eps . E[x^] of a row is a sum over all windows of the row.  A lane accumulates its eight
// columns, the eight row sums of a batch are reduced across the warp together (a butterfly
// that halves the number of live values at every stage: 9 shuffles for 8 rows, always in the
// same order), and every (window, row) partial goes to scratch memory.  A second small kernel
// adds the windows of a row in order and writes the sum and the corrected bias, so the
// result does not depend on scheduling.
#include "groupquant_impl.cuh"
#include "kernels.h"

namespace aweq {

// eight rows per batch; the scaled values are formed again in the second pass rather than kept
// (80 registers: two CTAs of this kernel fit on an SM beside a column-reduction CTA)
constexpr int kGqRows = 8;
constexpr bool kGqKeep = false;
constexpr int kGqOcc = 3;

size_t groupquant_ws_bytes(long long rows, long long cols)
{
    const long long nwin = (cols / 8 + 31) / 32;
    const long long prow = (rows + kGqRows - 1) / kGqRows * kGqRows;
    return (size_t)nwin * prow * sizeof(float);
}

bool groupquant_supported(int bits, int group) { return group == 128 && (bits == 4 || bits == 3 || bits == 8); }

template <class D, int BITS>
static aweq_status launch_gq(const GroupQuantParams &p, bool mu, float *epsmu, const BiasIO &bias, cudaStream_t stream)
{
    const long long items = p.nbatch * p.nwin;
    long long blocks = (items + kGqWarps - 1) / kGqWarps;
    const long long cap = (long long)kSmCount * kGqOcc * 8;      // a few waves; warps stride over the items beyond that
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (mu) {
        AWEQ_LAUNCH((groupquant_kernel<D, BITS, true, kGqRows, kGqKeep, kGqOcc>), dim3((unsigned)blocks), dim3(kGqWarps * 32), 0, stream, p);
        AWEQ_LAUNCH(groupquant_finalize_kernel, dim3((unsigned)((p.nrows + 255) / 256)), dim3(256), 0, stream,
                    (const float *)p.partial, p.nwin, p.prow, p.nrows, epsmu, bias);
    } else {
        AWEQ_LAUNCH((groupquant_kernel<D, BITS, false, kGqRows, kGqKeep, kGqOcc>), dim3((unsigned)blocks), dim3(kGqWarps * 32), 0, stream, p);
    }
    return AWEQ_OK;
}

aweq_status run_groupquant(const void *W, aweq_dtype dt, long long nrows, long long cols, long long ld,
                           const float *scale, const float *mu, int bits, unsigned char *out, float *step, int *zp,
                           float *epsmu, const BiasIO &bias, void *ws, cudaStream_t stream)
{
    GroupQuantParams p;
    p.W = reinterpret_cast<const uint16_t *>(W);
    p.nrows = nrows; p.ld = ld; p.nvec = (int)(cols / 8);
    p.nwin = (p.nvec + 31) / 32;
    p.nbatch = (nrows + kGqRows - 1) / kGqRows;
    p.scale = scale; p.mu = mu; p.out = out;
    p.out_pitch = cols * bits / 8;
    p.step = step; p.zp = zp; p.ngroups = (int)(cols / 128);
    p.partial = reinterpret_cast<float *>(ws);
    p.prow = p.nbatch * kGqRows;
    const bool has_mu = mu && epsmu;
#define AWEQ_GQ_GO(DT)                                                                  \
    switch (bits) {                                                                     \
    case 8: return launch_gq<DT, 8>(p, has_mu, epsmu, bias, stream);                    \
    case 4: return launch_gq<DT, 4>(p, has_mu, epsmu, bias, stream);                    \
    default: return launch_gq<DT, 3>(p, has_mu, epsmu, bias, stream);                   \
    }
    if (dt == AWEQ_F16) { AWEQ_GQ_GO(F16) }
    AWEQ_GQ_GO(BF16)
#undef AWEQ_GQ_GO
}

}  // namespace aweq
