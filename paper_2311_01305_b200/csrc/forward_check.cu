// W8A8 forward check: the calibrated layer  y~ = dequant(Xq) dequant(Wq)^T + bias'  against
// the 16-bit layer  y = X W^T + bias  on the calibration inputs, reported as the mean output
// error per output channel (the quantity of Eq. 11, E[y~_j - y_j], which bias correction
// is built to remove) and as sums of squares (output MSE and signal power).
//
// Both products are dense contractions and run on the tensor cores (forward_gemm.cuh):
//   S[n,o] = sum_k Xq[n,k] Wq[o,k]            unsigned 8-bit x unsigned 8-bit -> int32
//   Y[n,o] = sum_k X[n,k] W[o,k]              fp16 / bf16 -> binary32
// The zero-points of Eq. 1 are folded in afterwards, in integers:
//   y~[n,o] = Step^x_n Step^w_o (S - Z^x_n cw_o - Z^w_o rx_n + K Z^x_n Z^w_o) + bias'_o
// with rx_n = sum_k Xq[n,k] and cw_o = sum_k Wq[o,k].  A sum of K products of 8-bit codes
// fits int32 for K <= 33025; wider layers are contracted in two K-halves that are added in
// 64-bit.  Tokens are processed in chunks so that the [chunk x C_out] intermediates stay
// a few hundred MB.
#include "common.cuh"
#include "kernels.h"

namespace aweq {

constexpr long long kFcChunk = 16384;          // tokens per chunk
constexpr int kFcRowBlock = 128;               // tokens per CTA of the comparison kernel
constexpr long long kFcSplitK = 32768;         // above this C_in the integer product is taken in two halves
constexpr size_t kFcScratch = 1 << 20;         // scratch of the GEMMs

static inline size_t up256(size_t b) { return (b + 255) & ~(size_t)255; }

struct FcLayout {
    long long chunk, nchunks, blocks_per_chunk, nblocks;
    size_t S, S2, Y, rx, cw, partial, scratch, total;
};

static FcLayout fc_layout(long long N, long long C_in, long long C_out)
{
    FcLayout L;
    L.chunk = N < kFcChunk ? N : kFcChunk;
    L.nchunks = (N + kFcChunk - 1) / kFcChunk;
    L.blocks_per_chunk = (L.chunk + kFcRowBlock - 1) / kFcRowBlock;
    L.nblocks = L.blocks_per_chunk;            // every chunk adds into the same slots
    size_t off = 0;
    L.S = off; off += up256((size_t)L.chunk * C_out * 4);
    L.S2 = off; off += C_in > kFcSplitK ? up256((size_t)L.chunk * C_out * 4) : 0;
    L.Y = off; off += up256((size_t)L.chunk * C_out * 4);
    L.rx = off; off += up256((size_t)N * 4);
    L.cw = off; off += up256((size_t)C_out * 4);
    L.partial = off; off += up256((size_t)L.nblocks * C_out * 3 * 8);
    L.scratch = off; off += kFcScratch;
    L.total = off;
    return L;
}

size_t forward_check_ws_bytes(long long N, long long C_in, long long C_out) { return fc_layout(N, C_in, C_out).total; }

// sum of the bytes of every row of a row-major u8 matrix (one warp per row)
__global__ void __launch_bounds__(256) fc_rowsum_kernel(const unsigned char *__restrict__ Q, long long rows,
                                                        long long cols, int *__restrict__ out)
{
    pdl_begin();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    const uint4 *p = reinterpret_cast<const uint4 *>(Q + row * cols);
    unsigned int acc = 0;
    for (long long i = lane; i < cols / 16; i += 32) {
        const uint4 v = __ldg(p + i);
        acc = __dp4a(v.x, 0x01010101u, acc);
        acc = __dp4a(v.y, 0x01010101u, acc);
        acc = __dp4a(v.z, 0x01010101u, acc);
        acc = __dp4a(v.w, 0x01010101u, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[row] = (int)acc;
}

// Comparison of one token chunk.  A CTA covers kFcRowBlock tokens x 128 output channels: a lane
// owns four adjacent channels (16-byte loads of S and Y), the eight warps take the tokens
// round-robin, and the per-warp sums are added in warp order through shared memory, so the
// result does not depend on scheduling.  The integer part is formed in binary64, where it is
// exact (every term is an integer below 2^53):
//   acc = S - Z^x cw_o + Z^w (K Z^x - rx_n)
// The CTA's sums of d = y~ - y, d^2 and y^2 go to partial[block][channel]; chunk after chunk
// adds into the same slots in stream order.
// Weight-only mode (WO): the GEMM already produced d = x (W~ / s - W) in Dm; no integer part.
template <class D, bool WO>
__global__ void __launch_bounds__(256, 2)
fc_compare_kernel(const int *__restrict__ S, const int *__restrict__ S2, const float *__restrict__ Dm,
                  const float *__restrict__ Y, long long rows,
                  long long C_out, long long K, const float *__restrict__ act_step, const int *__restrict__ act_zp,
                  const int *__restrict__ rx, const float *__restrict__ w_step, const int *__restrict__ w_zp,
                  const int *__restrict__ cw, const float *__restrict__ bias_q, const uint16_t *__restrict__ bias,
                  double *__restrict__ partial, int accumulate)
{
    pdl_begin();
    __shared__ double sh[8][3][128];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long o0 = (long long)blockIdx.x * 128 + lane * 4;
    const long long r0 = (long long)blockIdx.y * kFcRowBlock, r1 = min(rows, r0 + (long long)kFcRowBlock);
    double sw[4], zw[4], cwd[4], bq[4], b[4];
    double sd[4] = {0, 0, 0, 0}, sd2[4] = {0, 0, 0, 0}, sy2[4] = {0, 0, 0, 0};
    const bool live = o0 < C_out;                    // C_out is a multiple of 8: a lane's four channels are all in or all out
    if (live) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (!WO) {
                sw[c] = (double)w_step[o0 + c];
                zw[c] = (double)w_zp[o0 + c];
                cwd[c] = (double)cw[o0 + c];
            }
            b[c] = bias ? (double)D::one(bias[o0 + c]) : 0.0;
            bq[c] = bias_q ? (double)bias_q[o0 + c] : b[c];      // no corrected bias: the layer keeps its own
        }
#pragma unroll 2
        for (long long n = r0 + warp; n < r1; n += 8) {
            const float4 y4 = __ldg(reinterpret_cast<const float4 *>(Y + n * C_out + o0));
            const float yv[4] = {y4.x, y4.y, y4.z, y4.w};
            double sv[4] = {0.0, 0.0, 0.0, 0.0};     // the integer contraction, exact in binary64
            float dv[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            double zx = 0.0, u = 0.0, sx = 0.0;
            if (WO) {
                const float4 d4 = __ldg(reinterpret_cast<const float4 *>(Dm + n * C_out + o0));
                dv[0] = d4.x; dv[1] = d4.y; dv[2] = d4.z; dv[3] = d4.w;
            } else {
                const int4 s4 = __ldg(reinterpret_cast<const int4 *>(S + n * C_out + o0));
                sv[0] = (double)s4.x; sv[1] = (double)s4.y; sv[2] = (double)s4.z; sv[3] = (double)s4.w;
                if (S2) {                     // a K above 32768 comes as two halves (the branch is uniform)
                    const int4 t4 = __ldg(reinterpret_cast<const int4 *>(S2 + n * C_out + o0));
                    sv[0] += (double)t4.x; sv[1] += (double)t4.y; sv[2] += (double)t4.z; sv[3] += (double)t4.w;
                }
                zx = (double)act_zp[n];
                u = (double)K * zx - (double)rx[n];
                sx = (double)act_step[n];
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const double y = (double)yv[c] + b[c];
                double d;
                if (WO) {
                    d = (double)dv[c] + (bq[c] - b[c]);
                } else {
                    const double acc = sv[c] - zx * cwd[c] + zw[c] * u;
                    d = (sx * sw[c] * acc + bq[c]) - y;
                }
                sd[c] += d;
                sd2[c] += d * d;
                sy2[c] += y * y;
            }
        }
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        sh[warp][0][lane * 4 + c] = sd[c];
        sh[warp][1][lane * 4 + c] = sd2[c];
        sh[warp][2][lane * 4 + c] = sy2[c];
    }
    __syncthreads();
    // 384 (quantity, channel) sums, 256 threads
    for (int i = threadIdx.x; i < 384; i += 256) {
        const int q = i / 128, c = i % 128;
        const long long o = (long long)blockIdx.x * 128 + c;
        if (o >= C_out) continue;
        double a = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) a += sh[w][q][c];
        double *out = partial + ((long long)blockIdx.y * C_out + o) * 3 + q;
        *out = accumulate ? *out + a : a;
    }
}

__global__ void __launch_bounds__(256)
fc_finish_kernel(const double *__restrict__ partial, long long nblocks, long long C_out, long long N,
                 double *__restrict__ mean_err, double *__restrict__ col_sums, int write_mean)
{
    pdl_begin();
    const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= C_out) return;
    double sd = 0.0, sd2 = 0.0, sy2 = 0.0;
    for (long long k = 0; k < nblocks; ++k) {
        const double *p = partial + (k * C_out + o) * 3;
        sd += p[0];
        sd2 += p[1];
        sy2 += p[2];
    }
    if (write_mean) mean_err[o] = sd / (double)N;
    col_sums[o * 2] = sd2;
    col_sums[o * 2 + 1] = sy2;
}

// sums[0] = sum (y~ - y)^2, sums[1] = sum y^2, sums[2] = sum_o mean_err_o^2, sums[3] = N * C_out
__global__ void __launch_bounds__(256)
fc_total_kernel(const double *__restrict__ col_sums, const double *__restrict__ mean_err, long long C_out, long long N,
                double *__restrict__ sums)
{
    pdl_begin();
    __shared__ double sh[3][256];
    double a = 0.0, b = 0.0, c = 0.0;
    for (long long o = threadIdx.x; o < C_out; o += 256) {
        a += col_sums[o * 2];
        b += col_sums[o * 2 + 1];
        c += mean_err[o] * mean_err[o];
    }
    sh[0][threadIdx.x] = a;
    sh[1][threadIdx.x] = b;
    sh[2][threadIdx.x] = c;
    __syncthreads();
    for (int w = 128; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w)
            for (int q = 0; q < 3; ++q) sh[q][threadIdx.x] += sh[q][threadIdx.x + w];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        sums[0] = sh[0][0];
        sums[1] = sh[1][0];
        sums[2] = sh[2][0];
        sums[3] = (double)N * (double)C_out;
    }
}

aweq_status run_forward_check(const unsigned char *Xq, const float *act_step, const int *act_zp,
                              const unsigned char *Wq, const float *w_step, const int *w_zp, const float *bias_q,
                              const void *X, const void *W, aweq_dtype dt, const void *bias, long long N,
                              long long C_in, long long C_out, double *mean_err, double *sums, void *ws,
                              size_t ws_bytes, cudaStream_t stream)
{
    const FcLayout L = fc_layout(N, C_in, C_out);
    if (L.total > ws_bytes) return AWEQ_ERR_WORKSPACE;
    char *base = reinterpret_cast<char *>(ws);
    int *S = reinterpret_cast<int *>(base + L.S);
    const bool split = C_in > kFcSplitK;
    int *S2 = split ? reinterpret_cast<int *>(base + L.S2) : nullptr;
    float *Y = reinterpret_cast<float *>(base + L.Y);
    int *rx = reinterpret_cast<int *>(base + L.rx);
    int *cw = reinterpret_cast<int *>(base + L.cw);
    double *partial = reinterpret_cast<double *>(base + L.partial);
    void *scratch = base + L.scratch;
    // K-halves: the first one a multiple of 128 so that the second starts on a tile boundary
    const long long K0 = split ? (C_in / 2 + 127) / 128 * 128 : C_in;

    AWEQ_LAUNCH(fc_rowsum_kernel, dim3((unsigned)((N + 7) / 8)), dim3(256), 0, stream, Xq, N, C_in, rx);
    AWEQ_LAUNCH(fc_rowsum_kernel, dim3((unsigned)((C_out + 7) / 8)), dim3(256), 0, stream, Wq, C_out, C_in, cw);
    for (long long c = 0; c < L.nchunks; ++c) {
        const long long n0 = c * kFcChunk;
        const long long rows = (N - n0) < kFcChunk ? (N - n0) : kFcChunk;
        aweq_status rc = fc_gemm_u8(Xq + n0 * C_in, Wq, S, (int)rows, (int)C_out, (int)K0, C_in, scratch, kFcScratch, stream);
        if (rc != AWEQ_OK) return rc;
        if (split) {
            rc = fc_gemm_u8(Xq + n0 * C_in + K0, Wq + K0, S2, (int)rows, (int)C_out, (int)(C_in - K0), C_in, scratch,
                            kFcScratch, stream);
            if (rc != AWEQ_OK) return rc;
        }
        const uint16_t *Xc = reinterpret_cast<const uint16_t *>(X) + n0 * C_in;
        rc = (dt == AWEQ_F16 ? fc_gemm_f16 : fc_gemm_bf16)(Xc, W, Y, (int)rows, (int)C_out, (int)C_in, C_in, scratch,
                                                           kFcScratch, stream);
        if (rc != AWEQ_OK) return rc;
        // the grid always spans a full chunk's row blocks so that a short last chunk adds zeros, not garbage
        const dim3 grid((unsigned)((C_out + 127) / 128), (unsigned)L.blocks_per_chunk);
        if (dt == AWEQ_F16)
            AWEQ_LAUNCH((fc_compare_kernel<F16, false>), grid, dim3(256), 0, stream, (const int *)S, (const int *)S2,
                        (const float *)nullptr, (const float *)Y, rows, C_out, C_in, act_step + n0, act_zp + n0, (const int *)(rx + n0), w_step,
                        w_zp, (const int *)cw, bias_q, (const uint16_t *)bias, partial, (int)(c > 0));
        else
            AWEQ_LAUNCH((fc_compare_kernel<BF16, false>), grid, dim3(256), 0, stream, (const int *)S, (const int *)S2,
                        (const float *)nullptr, (const float *)Y, rows, C_out, C_in, act_step + n0, act_zp + n0, (const int *)(rx + n0), w_step,
                        w_zp, (const int *)cw, bias_q, (const uint16_t *)bias, partial, (int)(c > 0));
    }
    double *cs = reinterpret_cast<double *>(Y);        // Y is free now: two doubles per output channel
    AWEQ_LAUNCH(fc_finish_kernel, dim3((unsigned)((C_out + 255) / 256)), dim3(256), 0, stream, (const double *)partial,
                L.nblocks, C_out, N, mean_err, cs, 1);
    AWEQ_LAUNCH(fc_total_kernel, dim3(1), dim3(256), 0, stream, (const double *)cs, (const double *)mean_err, C_out, N, sums);
    return AWEQ_OK;
}

// ------------------------------------------------------------------ weight-only check
// dW[o, j] = Step (q - Z) * (1/s_j) - W[o, j]: what the quantised, equalised weights differ by
// from the original ones once the 1/s of the input is folded back (Eq. 3), so that x . dW is
// the output error of a weight-only layer.  One warp per output row.  dW goes to memory
// rounded to 16 bits for the GEMM (good enough for the sums of squares); the MEAN error is
// linear in x, E[x . dW] = E[x] . dW, and is taken here from the unrounded dW and the binary64
// column sums of X, so it is not limited by the 16-bit rounding:
//     mean_err[o] = (sum_j xsum[j] dW[o, j]) / N + (bias_q[o] - bias[o])
template <class D>
__global__ void __launch_bounds__(256)
fc_delta_kernel(const unsigned char *__restrict__ codes, const float *__restrict__ step, const int *__restrict__ zp,
                int bits, int gran, int group, const float *__restrict__ rinv, const uint16_t *__restrict__ W,
                long long C_out, long long C_in, uint16_t *__restrict__ dW, const double *__restrict__ xsum,
                long long N, const float *__restrict__ bias_q, const uint16_t *__restrict__ bias,
                double *__restrict__ mean_err)
{
    pdl_begin();
    const int lane = threadIdx.x & 31;
    const long long nvec = C_in / 8;
    for (long long o = (long long)blockIdx.x * 8 + (threadIdx.x >> 5); o < C_out; o += (long long)gridDim.x * 8) {
        double dot = 0.0;
        for (long long v = lane; v < nvec; v += 32) {
            const long long j0 = v * 8;
            const long long k = gran == AWEQ_PER_TENSOR ? 0 : (gran == AWEQ_PER_ROW ? o : o * (C_in / group) + j0 / group);
            const float st = __ldg(step + k);
            const int z = __ldg(zp + k);
            // eight codes = `bits` bytes of the row's little-endian bit stream
            const unsigned char *src = codes + o * (C_in * bits / 8) + v * bits;
            unsigned long long word = 0;
            for (int t = 0; t < bits; ++t) word |= (unsigned long long)src[t] << (8 * t);
            float w8[8], r8[8];
            widen8<D>(ldg_stream(W + o * C_in + j0), w8);
            if (rinv) load8(rinv + j0, r8);
            uint32_t outw[4];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
                uint32_t pair = 0;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int q = (int)((word >> ((e + h) * bits)) & ((1u << bits) - 1u));
                    float t = __fmul_rn(st, (float)((long long)q - (long long)z));
                    if (rinv) t = __fmul_rn(t, r8[e + h]);
                    const float dw = __fsub_rn(t, w8[e + h]);
                    dot += xsum[j0 + e + h] * (double)dw;
                    pair |= (uint32_t)D::encode(dw) << (16 * h);
                }
                outw[e / 2] = pair;
            }
            *reinterpret_cast<uint4 *>(dW + o * C_in + j0) = make_uint4(outw[0], outw[1], outw[2], outw[3]);
        }
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, w);
        if (lane == 0) {
            const double b = bias ? (double)D::one(bias[o]) : 0.0;
            const double bq = bias_q ? (double)bias_q[o] : b;
            mean_err[o] = dot / (double)N + (bq - b);
        }
    }
}

struct FcwLayout {
    long long chunk, nchunks, blocks_per_chunk;
    size_t dW, Dm, Y, partial, xsum, xtmp, colws, scratch, total;
};

static FcwLayout fcw_layout(long long N, long long C_in, long long C_out)
{
    FcwLayout L;
    L.chunk = N < kFcChunk ? N : kFcChunk;
    L.nchunks = (N + kFcChunk - 1) / kFcChunk;
    L.blocks_per_chunk = (L.chunk + kFcRowBlock - 1) / kFcRowBlock;
    size_t off = 0;
    L.dW = off; off += up256((size_t)C_out * C_in * 2);
    L.Dm = off; off += up256((size_t)L.chunk * C_out * 4);
    L.Y = off; off += up256((size_t)L.chunk * C_out * 4);
    L.partial = off; off += up256((size_t)L.blocks_per_chunk * C_out * 3 * 8);
    L.xsum = off; off += up256((size_t)C_in * 8);
    L.xtmp = off; off += up256((size_t)C_in * 4) * 3;                 // min, max, mean of the column sweep (unused)
    L.colws = off; off += up256(colreduce_ws_bytes(N, C_in));
    L.scratch = off; off += kFcScratch;
    L.total = off;
    return L;
}

size_t forward_check_weights_ws_bytes(long long N, long long C_in, long long C_out)
{
    return fcw_layout(N, C_in, C_out).total;
}

aweq_status run_forward_check_weights(const unsigned char *codes, const float *step, const int *zp, int bits, int gran,
                                      int group, const float *rinv, const float *bias_q, const void *X, const void *W,
                                      aweq_dtype dt, const void *bias, long long N, long long C_in, long long C_out,
                                      double *mean_err, double *sums, void *ws, size_t ws_bytes, cudaStream_t stream)
{
    const FcwLayout L = fcw_layout(N, C_in, C_out);
    if (L.total > ws_bytes) return AWEQ_ERR_WORKSPACE;
    char *base = reinterpret_cast<char *>(ws);
    uint16_t *dW = reinterpret_cast<uint16_t *>(base + L.dW);
    float *Dm = reinterpret_cast<float *>(base + L.Dm);
    float *Y = reinterpret_cast<float *>(base + L.Y);
    double *partial = reinterpret_cast<double *>(base + L.partial);
    void *scratch = base + L.scratch;
    // binary64 column sums of X (the step-1 sweep), for the mean error
    double *xsum = reinterpret_cast<double *>(base + L.xsum);
    float *xtmp = reinterpret_cast<float *>(base + L.xtmp);
    const size_t tstride = up256((size_t)C_in * 4) / 4;
    aweq_status rs = run_stats(X, dt, N, C_in, C_in, xtmp, xtmp + tstride, xtmp + 2 * tstride, xsum, nullptr, 0,
                               base + L.colws, nullptr, stream);
    if (rs != AWEQ_OK) return rs;
    long long blocks = (C_out + 7) / 8;
    if (blocks > (long long)kSmCount * 8) blocks = (long long)kSmCount * 8;
    if (dt == AWEQ_F16)
        AWEQ_LAUNCH(fc_delta_kernel<F16>, dim3((unsigned)blocks), dim3(256), 0, stream, codes, step, zp, bits, gran, group,
                    rinv, (const uint16_t *)W, C_out, C_in, dW, (const double *)xsum, N, bias_q, (const uint16_t *)bias,
                    mean_err);
    else
        AWEQ_LAUNCH(fc_delta_kernel<BF16>, dim3((unsigned)blocks), dim3(256), 0, stream, codes, step, zp, bits, gran,
                    group, rinv, (const uint16_t *)W, C_out, C_in, dW, (const double *)xsum, N, bias_q,
                    (const uint16_t *)bias, mean_err);
    auto gemm = dt == AWEQ_F16 ? fc_gemm_f16 : fc_gemm_bf16;
    for (long long c = 0; c < L.nchunks; ++c) {
        const long long n0 = c * kFcChunk;
        const long long rows = (N - n0) < kFcChunk ? (N - n0) : kFcChunk;
        const uint16_t *Xc = reinterpret_cast<const uint16_t *>(X) + n0 * C_in;
        aweq_status rc = gemm(Xc, dW, Dm, (int)rows, (int)C_out, (int)C_in, C_in, scratch, kFcScratch, stream);
        if (rc != AWEQ_OK) return rc;
        rc = gemm(Xc, W, Y, (int)rows, (int)C_out, (int)C_in, C_in, scratch, kFcScratch, stream);
        if (rc != AWEQ_OK) return rc;
        const dim3 grid((unsigned)((C_out + 127) / 128), (unsigned)L.blocks_per_chunk);
        if (dt == AWEQ_F16)
            AWEQ_LAUNCH((fc_compare_kernel<F16, true>), grid, dim3(256), 0, stream, (const int *)nullptr,
                        (const int *)nullptr, (const float *)Dm, (const float *)Y, rows, C_out, C_in,
                        (const float *)nullptr, (const int *)nullptr, (const int *)nullptr, (const float *)nullptr,
                        (const int *)nullptr, (const int *)nullptr, bias_q, (const uint16_t *)bias, partial, (int)(c > 0));
        else
            AWEQ_LAUNCH((fc_compare_kernel<BF16, true>), grid, dim3(256), 0, stream, (const int *)nullptr,
                        (const int *)nullptr, (const float *)Dm, (const float *)Y, rows, C_out, C_in,
                        (const float *)nullptr, (const int *)nullptr, (const int *)nullptr, (const float *)nullptr,
                        (const int *)nullptr, (const int *)nullptr, bias_q, (const uint16_t *)bias, partial, (int)(c > 0));
    }
    double *cs = reinterpret_cast<double *>(Y);        // Y is free now: two doubles per output channel
    AWEQ_LAUNCH(fc_finish_kernel, dim3((unsigned)((C_out + 255) / 256)), dim3(256), 0, stream, (const double *)partial,
                L.blocks_per_chunk, C_out, N, mean_err, cs, 0);
    AWEQ_LAUNCH(fc_total_kernel, dim3(1), dim3(256), 0, stream, (const double *)cs, (const double *)mean_err, C_out, N, sums);
    return AWEQ_OK;
}

}  // namespace aweq
