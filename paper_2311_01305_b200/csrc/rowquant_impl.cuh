// What the row-wise Eq. 1-2 quantisers share: the kernel parameters and launch plans, the
// barriers of the shared-memory ring of the staged kernel (rowquant_cluster.cu: persistent
// CTAs pull tiles of rows through stages filled by 1-D bulk copies, completion on mbarriers,
// warp 0 issues the copies between its own work) and the code packing.
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


struct RqSmem {
    uint64_t full[kRqStagesMax];
    uint64_t empty[kRqStagesMax];
    int abort_flag;
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

// warp 0: wait (bounded) until the stage of tile `t` is free again, i.e. released by every warp
// after its previous use.  *timed_out is set when the wait gave up.
__device__ __forceinline__ bool rq_stage_free(RqSmem *sm, long long t, int S, bool *timed_out)
{
    const int s = (int)(t % S);
    const uint32_t use = (uint32_t)(t / S);
    if (use == 0) return true;
    bool ready = mbar_wait(&sm->empty[s], (use - 1) & 1);
    ready = __all_sync(0xffffffffu, ready);
    if (!ready) *timed_out = true;
    return ready;
}

// rows of step 6 beyond 36864 channels, each shared by a cluster of two CTAs (rowquant_cluster.cu)
bool plan_rowquant_cluster(long long nrows, long long cols, RowQuantPlan *out);
aweq_status run_rowquant_cluster(const RowQuantParams &p, const RowQuantPlan &pl, aweq_dtype dt, cudaStream_t stream);

}  // namespace aweq
