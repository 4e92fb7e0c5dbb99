// Steps 1 and 2: per-column min / max (/ sum) of a row-major 16-bit matrix.
//
// Step 1 (aweq_stats) reduces the calibration inputs X[N x C_in] to per-channel
// min, max and mean (Section 3.2: channel range = max - min; Section 3.3: E[x]
// is gathered in the same sweep).  Step 2 (aweq_wrange) reduces W[C_out x C_in]
// to per-input-channel min and max.  Both are one streaming read of the matrix
// and are bound by HBM bandwidth.
//
// Layout of the work: the columns are cut into slabs of at most 256 16-byte
// vectors (2048 columns; 320 or 384 vectors where that divides the row better)
// and the rows into splits; one CTA per SM owns one
// (slab, split) pair, so a thread owns one vector column for its whole life and
// keeps that column's eight running minima, maxima and sums in registers.
// A producer warp streams the CTA's rows through two shared-memory stages of
// 24 rows each (16 in the wider CTAs; up to 96 KB per stage) with 1-D bulk copies
// (TMA, completion on mbarriers); the consumer warps read the stages back conflict-free
// (consecutive lanes, consecutive 16-byte vectors).  Of the geometries timed
// on B200 (2-6 stages of 8-24 rows, one or two CTAs per SM) the base one was the
// fastest on both the 4096- and the 11008-column inputs.  min / max stay in packed 16-bit arithmetic (exact); sums
// are binary32 over eight rows at a time (one mixed-precision add per element)
// and are then added without rounding loss into a (hi, lo) pair of binary32
// values per column, which is widened to binary64 once at the end.  Each CTA writes one partial per column; a second small
// kernel reduces the partials over the splits in a fixed order, so results are
// bit-reproducible from run to run.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace aweq {

#ifndef AWEQ_COL_THREADS
#define AWEQ_COL_THREADS 256
#endif
#ifndef AWEQ_COL_ROWS
#define AWEQ_COL_ROWS 24
#endif
#ifndef AWEQ_COL_STAGES
#define AWEQ_COL_STAGES 2
#endif
#ifndef AWEQ_COL_CTAS_PER_SM
#define AWEQ_COL_CTAS_PER_SM 1
#endif
constexpr int kColThreads = AWEQ_COL_THREADS;   // consumer threads = vectors per slab of the base geometry
constexpr int kColRows = AWEQ_COL_ROWS;         // rows per stage of the base geometry
constexpr int kColStages = AWEQ_COL_STAGES;
constexpr int kColCtasPerSm = AWEQ_COL_CTAS_PER_SM;
constexpr int kColTargetCtas = kColCtasPerSm * kSmCount;
constexpr int kFlushRowsHost = 8;               // rows summed in binary32 before the error-free fold
// Geometries (consumer threads x rows per stage x stages), from sweeps on 1 GiB inputs at eight widths:
//   256 x 24 x 2   rows of one or two slabs (up to 4096 columns): few, tall stages      (4096: 7.04 TB/s)
//   256 x 16 x 3   rows of three or more slabs: a third stage pays once a CTA's copies are short
//                  (9216 columns 6.82 -> 7.11 TB/s, 11008 6.82 -> 7.09, 13824 6.96 -> 7.04, 36864 6.94 -> 6.91)
//   320 x 8 x 4, 384 x 8 x 3   where the wider CTA brings a row into one or two slabs that 256 threads
//                  cut into more (5120 columns = two slabs of 320: 6.72 -> 7.07; 3072 = one contiguous slab
//                  of 384: 6.39 -> 6.92-7.03)
constexpr int kColMaxThreads = 384;
constexpr int kColMaxStages = 4;

struct ColPlan {
    int nvec, nslab, slab_w, nsplit;
    int threads;         // consumer threads of a CTA: 256, 320 or 384
    int phases;          // thread groups that share a slab's columns and split a stage's rows
    int stage_rows;      // rows per stage
    int stages;          // stages of the ring: 2, 3 or 4
    long long rows_per_split;
};

// Consumer threads for a row of nvec vectors: 256, unless 320 or 384 threads bring the row into
// one or two slabs where 256 need more (the narrower of the two that does).  max_threads = 256 pins
// the base geometry (the built-in scratch of aweq_stats_static is sized for it).
static int pick_threads(int nvec, int max_threads)
{
    const int base_slabs = (nvec + kColThreads - 1) / kColThreads;
    if (base_slabs <= 1) return kColThreads;
    const int cand[2] = {320, kColMaxThreads};
    for (int c : cand) {
        if (c > max_threads) continue;
        const int nslab = (nvec + c - 1) / c;
        if (nslab <= 2 && nslab < base_slabs) return c;
    }
    return kColThreads;
}

// Row phases and stage height.  A slab of w vectors keeps only w of the consumer threads
// busy; when w <= 96 the idle threads take a second share of every stage's rows and write
// partials of their own (more than two phases multiply the partials the finalize kernel has
// to walk and were slower).  A stage holds as many rows as fit 96 KB (24 rows of a full slab):
// narrow matrices get taller stages, so that one bulk copy still moves ~96 KB -- but a split
// keeps at least a dozen stages, or filling and draining the two-stage ring shows.
// (Narrower slabs with more phases were tried instead of idle threads and were slower.)
static void pick_slabs(int nvec, long long rows_per_split, int threads, int *nslab_out, int *slab_w_out, int *phases_out,
                       int *stage_rows_out, int *stages_out)
{
    const int nslab = (nvec + threads - 1) / threads;
    const int w = (nvec + nslab - 1) / nslab;
    const int wpad = (w + 31) / 32 * 32;
    const int ph = wpad <= 96 ? 2 : 1;                         // from four warps per slab on, phases gained nothing
    const int unit = kFlushRowsHost * ph;                      // every phase gets whole eight-row groups
    const int stages = threads == 320 ? 4 : (threads == 384 || nslab >= 3) ? 3 : kColStages;
    const int full_rows = threads > kColThreads ? 8 : stages == 3 ? 16 : kColRows;
    int rows = ph == 1 ? full_rows : (int)((size_t)kColRows * kColThreads / w) / unit * unit;
    if (rows > 256) rows = 256 / unit * unit;
    if (rows_per_split > 0 && rows > rows_per_split / 12) rows = (int)(rows_per_split / 12) / unit * unit;
    if (rows < unit) rows = unit;
    *nslab_out = nslab;
    *slab_w_out = w;
    *phases_out = ph;
    *stage_rows_out = rows;
    *stages_out = stages;
}

ColPlan plan_colreduce(long long rows, long long cols, int max_threads = kColMaxThreads)
{
    ColPlan p;
    p.nvec = (int)(cols / 8);
    p.threads = pick_threads(p.nvec, max_threads);
    pick_slabs(p.nvec, 0, p.threads, &p.nslab, &p.slab_w, &p.phases, &p.stage_rows, &p.stages);
    int nsplit = kColTargetCtas / p.nslab;
    if (nsplit < 1) nsplit = 1;
    long long max_split = (rows + 7) / 8;
    if (max_split < 1) max_split = 1;
    if (nsplit > max_split) nsplit = (int)max_split;
    long long rps = (rows + nsplit - 1) / nsplit;
    rps = (rps + 7) / 8 * 8;            // whole eight-row groups; the last stage of a split may be partial
    if (rps < 8) rps = 8;
    p.rows_per_split = rps;
    pick_slabs(p.nvec, rps, p.threads, &p.nslab, &p.slab_w, &p.phases, &p.stage_rows, &p.stages);
    p.nsplit = (int)((rows + rps - 1) / rps);
    if (p.nsplit < 1) p.nsplit = 1;
    return p;
}

static size_t colreduce_ws_bytes_for(long long cols, int max_threads)
{
    // pmin, pmax: float[nsplit * phases][cols]; psum: double[nsplit * phases][cols].  Sized for the
    // largest number of row splits any row count can get, so that a buffer sized
    // for N rows also serves every call with fewer rows (streamed chunks).
    const int nvec = (int)(cols / 8);
    int nslab = 1, slab_w = 1, phases = 1, stage_rows = 8, stages = 2;
    pick_slabs(nvec > 0 ? nvec : 1, 0, pick_threads(nvec > 0 ? nvec : 1, max_threads), &nslab, &slab_w, &phases, &stage_rows,
               &stages);
    int max_split = kColTargetCtas / nslab;
    if (max_split < 1) max_split = 1;
    return (size_t)max_split * phases * (size_t)cols * 16 + 256;
}

size_t colreduce_ws_bytes(long long rows, long long cols)
{
    (void)rows;
    return colreduce_ws_bytes_for(cols, kColMaxThreads);
}

constexpr int kFlushRows = kFlushRowsHost;
static_assert(kColRows % kFlushRows == 0, "stage rows must be a multiple of the flush period");

// acc += widen(16-bit value): one mixed-precision add per element (exact widening,
// one binary32 rounding), no separate conversion
template <class D>
__device__ __forceinline__ void add_pair(float &a0, float &a1, uint32_t u);
template <>
__device__ __forceinline__ void add_pair<F16>(float &a0, float &a1, uint32_t u)
{
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\t"
        "add.rn.f32.f16 %0, l, %0;\n\tadd.rn.f32.f16 %1, h, %1;\n\t}"
        : "+f"(a0), "+f"(a1) : "r"(u));
}
template <>
__device__ __forceinline__ void add_pair<BF16>(float &a0, float &a1, uint32_t u)
{
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\t"
        "add.rn.f32.bf16 %0, l, %0;\n\tadd.rn.f32.bf16 %1, h, %1;\n\t}"
        : "+f"(a0), "+f"(a1) : "r"(u));
}

template <class D, bool WITH_SUM>
__device__ __forceinline__ void accumulate_vec(const uint4 &v, typename D::T2 (&mn)[4], typename D::T2 (&mx)[4],
                                               float (&acc)[8])
{
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        typename D::T2 h = D::from_bits(u[k]);
        mn[k] = __hmin2(mn[k], h);
        mx[k] = __hmax2(mx[k], h);
        if (WITH_SUM) add_pair<D>(acc[2 * k], acc[2 * k + 1], u[k]);
    }
}

// (hi, lo) += a without losing the rounding error of hi + a (Knuth's two-sum)
__device__ __forceinline__ void two_sum_into(float &hi, float &lo, float a)
{
    const float s = __fadd_rn(hi, a);
    const float bb = __fsub_rn(s, hi);
    const float e = __fadd_rn(__fsub_rn(hi, __fsub_rn(s, bb)), __fsub_rn(a, bb));
    lo = __fadd_rn(lo, e);
    hi = s;
}

// Up to four matrices with the same number of columns, reduced as if stacked on top of one
// another (the weight matrices that share a layer input: q / k / v, gate / up).  A stage never
// straddles two of them.
constexpr int kColMaxSegs = 4;
struct ColSegs {
    const uint16_t *base[kColMaxSegs];
    long long rows[kColMaxSegs];
    long long ld[kColMaxSegs];
    int n;
};

// the matrix that holds stacked row v, the row inside it, and the stacked index where it ends
__device__ __forceinline__ void seg_locate(const ColSegs &sg, long long v, int &m, long long &local, long long &end)
{
    long long start = 0;
    m = 0;
#pragma unroll
    for (int k = 0; k < kColMaxSegs - 1; ++k) {
        if (m == k && k + 1 < sg.n && v >= start + sg.rows[k]) {
            start += sg.rows[k];
            m = k + 1;
        }
    }
    local = v - start;
    end = start + sg.rows[m];
}

struct ColSmem {
    uint64_t full[kColMaxStages];
    uint64_t empty[kColMaxStages];
    int abort_flag;
};

template <class D, bool WITH_SUM, int NT, int STAGES>
__global__ void __launch_bounds__(NT + 32, kColCtasPerSm)
colreduce_kernel(const ColSegs segs, long long nrows, int nvec, int nslab, int slab_w,
                 int phases, int stage_rows, long long rows_per_split, long long cols, float *__restrict__ pmin,
                 float *__restrict__ pmax, double *__restrict__ psum, aweq_dev_status *st, long long rows_a,
                 long long rows_per_split_b, float *__restrict__ pmin_b, float *__restrict__ pmax_b)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    ColSmem *sm = reinterpret_cast<ColSmem *>(smem_raw);
    uint4 *stage_base = reinterpret_cast<uint4 *>(smem_raw + 128);

    const int slab = blockIdx.x % nslab;
    const int split = blockIdx.x / nslab;
    const int v0 = slab * slab_w;
    const int w = min(slab_w, nvec - v0);                 // vectors in this slab (> 0)
    // Two jobs share the launch and the ring: job A is the first rows_a rows of the stack (all of it
    // in an ordinary call), job B the rest -- the weight matrices fed by the input whose statistics
    // job A takes -- reduced to extremes of their own.  Every CTA takes its share of both, one after
    // the other, so the second job costs neither a launch nor a fill and drain of the ring.
    const long long job_r0[2] = {min(rows_a, (long long)split * rows_per_split),
                                 min(nrows, rows_a + (long long)split * rows_per_split_b)};
    const long long job_r1[2] = {min(rows_a, job_r0[0] + rows_per_split),
                                 min(nrows, job_r0[1] + rows_per_split_b)};
    const int njobs = rows_per_split_b > 0 ? 2 : 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // phase p of the consumer threads takes rows [p, p + 1) * stage_rows / phases of every stage;
    // a phase is a whole number of warps
    const int wpad = (slab_w + 31) / 32 * 32;
    const int active_warps = phases * wpad / 32;
    const size_t stage_vecs = (size_t)stage_rows * slab_w;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sm->full[s], 1);
            mbar_init(&sm->empty[s], active_warps);
        }
        sm->abort_flag = 0;
        mbar_init_fence();
    }
    pdl_begin();                 // everything above overlaps the tail of the previous kernel
    __syncthreads();

    if (warp == NT / 32) {
        // ---------------- producer warp
        bool ok = true;
        int t = 0;
        for (int job = 0; job < njobs && ok; ++job) {
        long long cur = job_r0[job];
        const long long r1 = job_r1[job];
        for (; cur < r1 && ok; ++t) {
            const int s = t % STAGES;
            const uint32_t use = t / STAGES;
            if (use > 0) {
                ok = mbar_wait(&sm->empty[s], (use - 1) & 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
            }
            int m;
            long long local, seg_end;
            seg_locate(segs, cur, m, local, seg_end);
            const long long ld = segs.ld[m];
            const uint16_t *X = segs.base[m];
            const int rows = (int)min((long long)stage_rows, min(r1, seg_end) - cur);
            const bool contiguous = (nslab == 1) && (ld == cols);
            uint4 *dst = stage_base + (size_t)s * stage_vecs;
            if (lane == 0) mbar_arrive_expect_tx(&sm->full[s], (uint32_t)rows * w * 16u);
            __syncwarp();
            if (contiguous) {
                if (lane == 0) bulk_g2s(dst, X + local * ld, (uint32_t)rows * w * 16u, &sm->full[s]);
            } else {
                for (int r = lane; r < rows; r += 32)
                    bulk_g2s(dst + (size_t)r * w, X + (local + r) * ld + (long long)v0 * 8, (uint32_t)w * 16u,
                             &sm->full[s]);
            }
            cur += rows;
        }
        }
        if (!ok && lane == 0) {
            atomicExch(&sm->abort_flag, 1);
            if (st) atomicAdd(&st->wait_timeout, 1ull);
        }
    } else if (warp < active_warps) {
        // ---------------- consumer warps: thread <-> one vector column
        const int phase = threadIdx.x / wpad;
        const int t_col = threadIdx.x - phase * wpad;
        const bool mine = t_col < w;
        const int rows_per_phase = stage_rows / phases;          // a multiple of kFlushRows
        bool ok = true;
        int t = 0;
        for (int job = 0; job < njobs && ok; ++job) {
        typename D::T2 mn[4], mx[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            mn[k] = D::from_bits(D::pos_inf2());
            mx[k] = D::from_bits(D::neg_inf2());
        }
        float sum_hi[8], sum_lo[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) sum_hi[k] = sum_lo[k] = 0.0f;
        long long cur = job_r0[job];
        const long long r1 = job_r1[job];
        for (; cur < r1; ++t) {
            const int s = t % STAGES;
            const uint32_t use = t / STAGES;
            ok = mbar_wait(&sm->full[s], use & 1);
            if (!ok || *reinterpret_cast<volatile int *>(&sm->abort_flag)) { ok = false; break; }
            int m;
            long long local, seg_end;
            seg_locate(segs, cur, m, local, seg_end);
            const int rows_in_stage = (int)min((long long)stage_rows, min(r1, seg_end) - cur);
            cur += rows_in_stage;
            const int rows = min(rows_in_stage, (phase + 1) * rows_per_phase);      // end of my share
            const uint4 *src = stage_base + (size_t)s * stage_vecs + t_col;
            if (mine) {
                // groups of kFlushRows rows: binary32 partial sums, then an error-free
                // addition into the (hi, lo) running sum
                for (int rb = phase * rows_per_phase; rb < rows; rb += kFlushRows) {
                    float acc32[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc32[k] = 0.0f;
                    if (rows - rb >= kFlushRows) {
                        uint4 v[kFlushRows];
#pragma unroll
                        for (int r = 0; r < kFlushRows; ++r) v[r] = src[(size_t)(rb + r) * w];
#pragma unroll
                        for (int r = 0; r < kFlushRows; ++r)
                            accumulate_vec<D, WITH_SUM>(v[r], mn, mx, acc32);
                    } else {
                        for (int r = rb; r < rows; ++r)
                            accumulate_vec<D, WITH_SUM>(src[(size_t)r * w], mn, mx, acc32);
                    }
                    if (WITH_SUM) {
#pragma unroll
                        for (int k = 0; k < 8; ++k) two_sum_into(sum_hi[k], sum_lo[k], acc32[k]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->empty[s]);
        }
        if (!ok) break;
        if (mine) {
            // this CTA's partial of the job (neutral values when its share of the job is empty)
            const size_t o = ((size_t)split * phases + phase) * (size_t)cols + (size_t)(v0 + t_col) * 8;
            float lo[8], hi[8];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float2 a = D::to_float2(mn[k]), b = D::to_float2(mx[k]);
                lo[2 * k] = a.x; lo[2 * k + 1] = a.y;
                hi[2 * k] = b.x; hi[2 * k + 1] = b.y;
            }
            float4 *qlo = reinterpret_cast<float4 *>((job == 0 ? pmin : pmin_b) + o);
            float4 *qhi = reinterpret_cast<float4 *>((job == 0 ? pmax : pmax_b) + o);
            qlo[0] = make_float4(lo[0], lo[1], lo[2], lo[3]);
            qlo[1] = make_float4(lo[4], lo[5], lo[6], lo[7]);
            qhi[0] = make_float4(hi[0], hi[1], hi[2], hi[3]);
            qhi[1] = make_float4(hi[4], hi[5], hi[6], hi[7]);
            if (WITH_SUM && job == 0) {
                double2 *qs = reinterpret_cast<double2 *>(psum + o);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    qs[k] = make_double2((double)sum_hi[2 * k] + (double)sum_lo[2 * k],
                                         (double)sum_hi[2 * k + 1] + (double)sum_lo[2 * k + 1]);
            }
        }
        }
        if (!ok && lane == 0) {
            atomicExch(&sm->abort_flag, 1);
            if (st) atomicAdd(&st->wait_timeout, 1ull);
        }
    }
    // Every copy that was issued has been waited for by the consumers unless a
    // wait timed out; in that case give outstanding copies a bounded chance to
    // land before the shared memory is released.
    __syncthreads();
    if (threadIdx.x == 0 && sm->abort_flag) {
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) { }
    }
}

// Reduce the per-split partials in a fixed order; merge with the running state
// when accumulating.  A block handles 32 columns with 32 threads each: thread
// (c, k) folds partials k, k+32, ... and the 32 results of a column are then
// combined in order of k, so the result does not depend on timing.
constexpr int kFinCols = 32, kFinLanes = 32;

template <bool WITH_SUM>
__device__ __forceinline__ void colreduce_finalize_block(unsigned block, const float *__restrict__ pmin,
                                                         const float *__restrict__ pmax, const double *__restrict__ psum,
                                                         int nsplit, long long cols, long long nrows, float *omin,
                                                         float *omax, float *omean, double *osum, const long long *count,
                                                         int accumulate, aweq_dev_status *st, float *negmin_max,
                                                         double *count_f64)
{
    __shared__ float slo[kFinLanes][kFinCols], shi[kFinLanes][kFinCols];
    __shared__ double ssum[WITH_SUM ? kFinLanes : 1][kFinCols];
    if (count_f64 && block == 0 && threadIdx.x == 0) *count_f64 = (double)nrows;
    const int c = threadIdx.x % kFinCols, k0 = threadIdx.x / kFinCols;
    const long long j = (long long)block * kFinCols + c;
    float lo = INFINITY, hi = -INFINITY;
    double sum = 0.0;
    if (j < cols) {
        for (int k = k0; k < nsplit; k += kFinLanes) {
            lo = fminf(lo, pmin[(size_t)k * cols + j]);
            hi = fmaxf(hi, pmax[(size_t)k * cols + j]);
            if (WITH_SUM) sum += psum[(size_t)k * cols + j];
        }
    }
    slo[k0][c] = lo;
    shi[k0][c] = hi;
    if (WITH_SUM) ssum[k0][c] = sum;
    __syncthreads();
    if (k0 != 0 || j >= cols) return;
    for (int k = 1; k < kFinLanes; ++k) {
        lo = fminf(lo, slo[k][c]);
        hi = fmaxf(hi, shi[k][c]);
        if (WITH_SUM) sum += ssum[k][c];
    }
    long long total = nrows;
    if (accumulate) {
        lo = fminf(lo, omin[j]);
        hi = fmaxf(hi, omax[j]);
        if (WITH_SUM) {
            sum += osum[j];
            total += count[0];
        }
    }
    omin[j] = lo;
    omax[j] = hi;
    if (negmin_max) {                       // exchange form: one MAX all-reduce merges both extremes
        negmin_max[j] = -lo;
        negmin_max[cols + j] = hi;
    }
    if (WITH_SUM) {
        if (osum) osum[j] = sum;
        omean[j] = total > 0 ? (float)(sum / (double)total) : 0.0f;
    }
    if (st) {
        bool bad = (nrows > 0 || accumulate) && !(isfinite(lo) && isfinite(hi) && isfinite(sum));
        if (bad) atomicAdd(&st->nonfinite, 1ull);
    }
}

template <bool WITH_SUM>
__global__ void __launch_bounds__(kFinCols * kFinLanes)
colreduce_finalize_kernel(const float *__restrict__ pmin, const float *__restrict__ pmax,
                          const double *__restrict__ psum, int nsplit, long long cols, long long nrows, float *omin,
                          float *omax, float *omean, double *osum, const long long *count, int accumulate,
                          aweq_dev_status *st, float *negmin_max, double *count_f64)
{
    pdl_begin();
    colreduce_finalize_block<WITH_SUM>(blockIdx.x, pmin, pmax, psum, nsplit, cols, nrows, omin, omax, omean, osum, count,
                                       accumulate, st, negmin_max, count_f64);
}

// Both jobs of a fused statistics + weight-range launch in one finalize launch: the first `blocks_a`
// blocks finish job A (with the sums), the others job B (extremes only).
struct FinalizeB {
    const float *pmin, *pmax;
    long long nrows;
    float *omin, *omax;
};
__global__ void __launch_bounds__(kFinCols * kFinLanes)
colreduce_finalize_pair_kernel(const float *__restrict__ pmin, const float *__restrict__ pmax,
                               const double *__restrict__ psum, int nsplit, long long cols, long long nrows, float *omin,
                               float *omax, float *omean, double *osum, aweq_dev_status *st, float *negmin_max,
                               double *count_f64, unsigned blocks_a, const FinalizeB b)
{
    pdl_begin();
    if (blockIdx.x < blocks_a)
        colreduce_finalize_block<true>(blockIdx.x, pmin, pmax, psum, nsplit, cols, nrows, omin, omax, omean, osum,
                                       (const long long *)nullptr, 0, st, negmin_max, count_f64);
    else
        colreduce_finalize_block<false>(blockIdx.x - blocks_a, b.pmin, b.pmax, (const double *)nullptr, nsplit, cols, b.nrows,
                                        b.omin, b.omax, (float *)nullptr, (double *)nullptr, (const long long *)nullptr, 0, st,
                                        (float *)nullptr, (double *)nullptr);
}

__global__ void bump_count_kernel(long long *count, long long nrows, int accumulate)
{
    pdl_begin();
    count[0] = (accumulate ? count[0] : 0) + nrows;
}

static size_t colreduce_smem_bytes(int slab_w, int stage_rows, int stages)
{
    return 128 + (size_t)stages * stage_rows * slab_w * 16;
}

// Scratch of a fused statistics + weight-range launch: the partials of both jobs.
size_t colreduce_fused_ws_bytes(long long rows, long long cols)
{
    const size_t one = colreduce_ws_bytes(rows, cols) - 256;          // 16 bytes per (split, column)
    return one + one / 2 + 256;                                       // + 8 for the second job's extremes
}

// rows_a: rows of job A (the first segments); segments beyond them are job B, reduced to omin_b / omax_b
// (no sums).  rows_a < 0: a single job over all segments.
template <class D, bool WITH_SUM>
static aweq_status launch_colreduce(const ColSegs &segs, long long cols, float *omin,
                                    float *omax, float *omean, double *osum, long long *count, int accumulate,
                                    void *ws, aweq_dev_status *st, cudaStream_t stream, float *negmin_max = nullptr,
                                    double *count_f64 = nullptr, long long rows_a = -1, float *omin_b = nullptr,
                                    float *omax_b = nullptr, int max_threads = kColMaxThreads)
{
    long long rows_all = 0;
    for (int k = 0; k < segs.n; ++k) rows_all += segs.rows[k];
    const long long rows = rows_a < 0 ? rows_all : rows_a;
    const long long rows_b = rows_all - rows;
    ColPlan p = plan_colreduce(rows, cols, max_threads);
    char *base = reinterpret_cast<char *>(ws);
    float *pmin = reinterpret_cast<float *>(base);
    const size_t nparts = (size_t)p.nsplit * p.phases;
    float *pmax = pmin + nparts * cols;
    double *psum = reinterpret_cast<double *>(base + nparts * cols * 8);
    float *pmin_b = reinterpret_cast<float *>(base + nparts * cols * 16);
    float *pmax_b = pmin_b + nparts * cols;
    long long rps_b = 0;
    if (rows_b > 0) {
        rps_b = (rows_b + p.nsplit - 1) / p.nsplit;
        rps_b = (rps_b + 7) / 8 * 8;
    }
    const size_t smem = colreduce_smem_bytes(p.slab_w, p.stage_rows, p.stages);
    auto kern = p.threads == 384   ? colreduce_kernel<D, WITH_SUM, 384, 3>
                : p.threads == 320 ? colreduce_kernel<D, WITH_SUM, 320, 4>
                : p.stages == 3    ? colreduce_kernel<D, WITH_SUM, kColThreads, 3>
                                   : colreduce_kernel<D, WITH_SUM, kColThreads, kColStages>;
    // set on every launch: the attribute belongs to the current device, which may change between calls
    AWEQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)colreduce_smem_bytes(kColThreads, kColRows, kColStages)));
    int nsplit_eff = rows > 0 ? (int)nparts : 0;
    if (rows > 0) {
        AWEQ_LAUNCH(kern, dim3(p.nslab * p.nsplit), dim3(p.threads + 32), smem, stream,
                    segs, rows_all, p.nvec, p.nslab, p.slab_w, p.phases, p.stage_rows, p.rows_per_split, cols, pmin, pmax,
                    psum, st, rows, rps_b, pmin_b, pmax_b);
    }
    const unsigned fin_blocks = (unsigned)((cols + kFinCols - 1) / kFinCols);
    if constexpr (WITH_SUM) {
        if (rows_b > 0 && !accumulate && !count) {
            const FinalizeB fb = {pmin_b, pmax_b, rows_b, omin_b, omax_b};
            AWEQ_LAUNCH(colreduce_finalize_pair_kernel, dim3(2 * fin_blocks), dim3(kFinCols * kFinLanes), 0, stream,
                        (const float *)pmin, (const float *)pmax, (const double *)psum, nsplit_eff, cols, rows, omin, omax,
                        omean, osum, st, negmin_max, count_f64, fin_blocks, fb);
            return AWEQ_OK;
        }
    }
    AWEQ_LAUNCH(colreduce_finalize_kernel<WITH_SUM>, dim3(fin_blocks),
                dim3(kFinCols * kFinLanes), 0, stream, (const float *)pmin, (const float *)pmax, (const double *)psum,
                nsplit_eff, cols, rows, omin, omax, omean, osum, (const long long *)count, accumulate, st, negmin_max,
                count_f64);
    if (rows_b > 0) {
        AWEQ_LAUNCH(colreduce_finalize_kernel<false>, dim3((unsigned)((cols + kFinCols - 1) / kFinCols)),
                    dim3(kFinCols * kFinLanes), 0, stream, (const float *)pmin_b, (const float *)pmax_b,
                    (const double *)nullptr, nsplit_eff, cols, rows_b, omin_b, omax_b, (float *)nullptr, (double *)nullptr,
                    (const long long *)nullptr, 0, st, (float *)nullptr, (double *)nullptr);
    }
    if (WITH_SUM && count) {
        AWEQ_LAUNCH(bump_count_kernel, dim3(1), dim3(1), 0, stream, count, rows, accumulate);
    }
    return AWEQ_OK;
}

void colreduce_describe(long long rows, long long cols, long long plan[8])
{
    const ColPlan p = plan_colreduce(rows, cols);
    plan[0] = (long long)p.nslab * p.nsplit;
    plan[1] = p.threads + 32;
    plan[2] = (long long)colreduce_smem_bytes(p.slab_w, p.stage_rows, p.stages);
    plan[3] = p.nslab;
    plan[4] = p.slab_w;
    plan[5] = p.nsplit;
    plan[6] = p.phases;
    plan[7] = p.stage_rows;
}

// Statistics of a token shard back from their exchange form (see run_stats): after the two
// all-reduces the buffers hold the extremes, sums and token count of all shards.
__global__ void stats_from_exchange_kernel(const float *__restrict__ negmin_max, const double *__restrict__ sum_count,
                                           long long cols, float *xmin, float *xmax, float *xmean)
{
    pdl_begin();
    const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    const double total = sum_count[cols];
    xmin[j] = -negmin_max[j];
    xmax[j] = negmin_max[cols + j];
    xmean[j] = total > 0.0 ? (float)(sum_count[j] / total) : 0.0f;
}

aweq_status run_stats_from_exchange(const float *negmin_max, const double *sum_count, long long C, float *xmin,
                                    float *xmax, float *xmean, cudaStream_t stream)
{
    AWEQ_LAUNCH(stats_from_exchange_kernel, dim3((unsigned)((C + 255) / 256)), dim3(256), 0, stream, negmin_max,
                sum_count, C, xmin, xmax, xmean);
    return AWEQ_OK;
}

// negmin_max / sum_count (both or neither): also leave the statistics in exchange form,
// negmin_max = float[2 C] = { -xmin, xmax }, sum_count = double[C + 1] = { column sums, N }.
aweq_status run_stats(const void *X, aweq_dtype dt, long long N, long long C, long long ld, float *xmin, float *xmax,
                      float *xmean, double *xsum, long long *count, int accumulate, void *ws, aweq_dev_status *st,
                      cudaStream_t stream, float *negmin_max, double *sum_count)
{
    if (negmin_max && sum_count) {
        xsum = sum_count;
        count = nullptr;
        accumulate = 0;
    }
    double *count_f64 = (negmin_max && sum_count) ? sum_count + C : nullptr;
    ColSegs segs = {};
    segs.base[0] = reinterpret_cast<const uint16_t *>(X);
    segs.rows[0] = N;
    segs.ld[0] = ld;
    segs.n = 1;
    if (dt == AWEQ_F16)
        return launch_colreduce<F16, true>(segs, C, xmin, xmax, xmean, xsum, count, accumulate, ws, st, stream,
                                           negmin_max, count_f64);
    return launch_colreduce<BF16, true>(segs, C, xmin, xmax, xmean, xsum, count, accumulate, ws, st, stream, negmin_max,
                                        count_f64);
}

// Steps 1 and 2 of one input in a single launch: the statistics of X and the common ranges of the (at
// most three) weight matrices it feeds, which have the same number of columns.
// Worth it while the matrices are small enough for a launch of their own to be dominated by the fill and
// drain of its ring (measured: the passes of the LLaMA-7B, LLaMA-13B and OPT-125M shapes gain 0.5-1.2 %;
// two 680 MB matrices reduce at 6.7 TB/s on their own and lose 0.5 % when folded into the sweep).
bool stats_wrange_fusable(long long N, long long C_in, const long long *C_out, int n_w)
{
    if (N <= 0 || n_w < 1 || n_w > kColMaxSegs - 1) return false;
    long long rows = 0;
    for (int k = 0; k < n_w; ++k) rows += C_out[k];
    return 2 * rows * C_in <= 400000000ll;
}

aweq_status run_stats_wrange(const void *X, aweq_dtype dt, long long N, long long C, long long ld, float *xmin,
                             float *xmax, float *xmean, const void *const *W, const long long *C_out,
                             const long long *ldw, int n_w, float *wmin, float *wmax, void *ws, aweq_dev_status *st,
                             cudaStream_t stream, float *negmin_max, double *sum_count)
{
    double *xsum = (negmin_max && sum_count) ? sum_count : nullptr;
    double *count_f64 = (negmin_max && sum_count) ? sum_count + C : nullptr;
    ColSegs segs = {};
    segs.base[0] = reinterpret_cast<const uint16_t *>(X);
    segs.rows[0] = N;
    segs.ld[0] = ld;
    for (int k = 0; k < n_w; ++k) {
        segs.base[1 + k] = reinterpret_cast<const uint16_t *>(W[k]);
        segs.rows[1 + k] = C_out[k];
        segs.ld[1 + k] = ldw[k];
    }
    segs.n = 1 + n_w;
    if (dt == AWEQ_F16)
        return launch_colreduce<F16, true>(segs, C, xmin, xmax, xmean, xsum, nullptr, 0, ws, st, stream, negmin_max,
                                           count_f64, N, wmin, wmax);
    return launch_colreduce<BF16, true>(segs, C, xmin, xmax, xmean, xsum, nullptr, 0, ws, st, stream, negmin_max,
                                        count_f64, N, wmin, wmax);
}

aweq_status run_wrange(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ld, float *wmin,
                       float *wmax, int accumulate, void *ws, aweq_dev_status *st, cudaStream_t stream)
{
    const void *Ws[1] = {W};
    return run_wrange_multi(Ws, &C_out, &ld, 1, dt, C_in, wmin, wmax, accumulate, ws, st, stream);
}

// The common range of several matrices with the same C_in: stacks of up to four go through one
// launch (one pipeline fill and one finalize instead of one per matrix).
aweq_status run_wrange_multi(const void *const *W, const long long *C_out, const long long *ld, int n, aweq_dtype dt,
                             long long C_in, float *wmin, float *wmax, int accumulate, void *ws, aweq_dev_status *st,
                             cudaStream_t stream)
{
    for (int i0 = 0; i0 < n; i0 += kColMaxSegs) {
        ColSegs segs = {};
        segs.n = n - i0 < kColMaxSegs ? n - i0 : kColMaxSegs;
        for (int k = 0; k < segs.n; ++k) {
            segs.base[k] = reinterpret_cast<const uint16_t *>(W[i0 + k]);
            segs.rows[k] = C_out[i0 + k];
            segs.ld[k] = ld[i0 + k];
        }
        const int acc = accumulate || i0 > 0;
        const aweq_status rc =
            dt == AWEQ_F16 ? launch_colreduce<F16, false>(segs, C_in, wmin, wmax, nullptr, nullptr, nullptr, acc, ws, st, stream)
                           : launch_colreduce<BF16, false>(segs, C_in, wmin, wmax, nullptr, nullptr, nullptr, acc, ws, st,
                                                           stream);
        if (rc != AWEQ_OK) return rc;
    }
    return AWEQ_OK;
}

}  // namespace aweq

// ------------------------------------------------------------------ statistics without caller scratch
// Scratch for aweq_stats_static: the per-split partials of one call.  It lives in
// the library image, so every GPU that loads the library holds these bytes until
// the process exits.  The partials need (row splits) x (row phases) x C_in x 16
// bytes; the number of row splits is at most 148 / ceil(C_in / 2048), and two row
// phases are only used up to 768 columns (148 x 2 x 768 x 16 bytes), so
// 148 x 2048 x 16 bytes cover every supported width.  The entry point compares the
// planner's own figure with the array size as well.
namespace aweq {
constexpr size_t kStaticScratchBytes = (size_t)kColTargetCtas * kColThreads * 8 * 16 + 256;
constexpr long long kStaticMaxCin = 16384;
constexpr int kMaxDevices = 64;
}  // namespace aweq
static __device__ __align__(256) unsigned char g_stats_static_scratch[aweq::kStaticScratchBytes];

namespace aweq {
// Device address of the scratch array on the current device.  The array's name is
// only a host-side handle in host code; the address a kernel can use comes from
// cudaGetSymbolAddress, asked once per device with that device current.
static aweq_status static_scratch_address(void **out)
{
    static std::mutex lock;
    static void *address[kMaxDevices] = {};
    int dev = -1;
    AWEQ_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return AWEQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> guard(lock);
    if (!address[dev]) {
        void *p = nullptr;
        AWEQ_CUDA_OK(cudaGetSymbolAddress(&p, g_stats_static_scratch));
        address[dev] = p;
    }
    *out = address[dev];
    return AWEQ_OK;
}
}  // namespace aweq

extern "C" aweq_status aweq_stats_static(const void *X, aweq_dtype dt, long long N, long long C_in, long long ldx,
                                         float *xmin, float *xmax, float *xmean, aweq_dev_status *st, void *stream)
{
    using namespace aweq;
    if (!X || !xmin || !xmax || !xmean) return AWEQ_ERR_NULL;
    if (dt != AWEQ_F16 && dt != AWEQ_BF16) return AWEQ_ERR_DTYPE;
    if (C_in <= 0 || (C_in % 8) != 0 || N <= 0 || N > (1ll << 40)) return AWEQ_ERR_SHAPE;
    if (C_in > kStaticMaxCin || colreduce_ws_bytes_for(C_in, kColThreads) > kStaticScratchBytes) return AWEQ_ERR_LIMIT;
    if (ldx < C_in || (ldx % 8) != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0) return AWEQ_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(xmin) & 15) != 0 || (reinterpret_cast<uintptr_t>(xmax) & 15) != 0)
        return AWEQ_ERR_ALIGN;
    void *scratch = nullptr;
    aweq_status rc = static_scratch_address(&scratch);
    if (rc != AWEQ_OK) return rc;
    // every partial the reduction reads is written by this call first, so the
    // contents left by an earlier call need no clearing
    // (the base geometry: the array is sized for its number of partials)
    ColSegs segs = {};
    segs.base[0] = reinterpret_cast<const uint16_t *>(X);
    segs.rows[0] = N;
    segs.ld[0] = ldx;
    segs.n = 1;
    cudaStream_t cs = (cudaStream_t)stream;
    if (dt == AWEQ_F16)
        return launch_colreduce<F16, true>(segs, C_in, xmin, xmax, xmean, nullptr, nullptr, 0, scratch, st, cs, nullptr, nullptr,
                                           -1, nullptr, nullptr, kColThreads);
    return launch_colreduce<BF16, true>(segs, C_in, xmin, xmax, xmean, nullptr, nullptr, 0, scratch, st, cs, nullptr, nullptr, -1,
                                        nullptr, nullptr, kColThreads);
}

