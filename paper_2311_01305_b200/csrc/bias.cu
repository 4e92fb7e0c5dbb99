// Step 5: statistical bias correction (Eq. 11-15).  The expected output error
// of the quantised layer, eps . E[x^] with eps = W~ - W^, is subtracted from the
// layer's bias.  The fused route takes the row sums that step 4 produced while
// it had the weights in registers; the standalone route recomputes them from
// the stored codes (a bandwidth-bound GEMV over W and the packed codes).
#include "common.cuh"

namespace aweq {

__global__ void bias_apply_kernel(const float *__restrict__ epsmu, const uint16_t *__restrict__ bias_in,
                                  uint16_t *__restrict__ bias_out, float *__restrict__ bias_out_f32, int bias_bf16,
                                  long long C_out)
{
    pdl_begin();
    const long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= C_out) return;
    write_bias(o, epsmu[o], bias_in, bias_out, bias_out_f32, bias_bf16);
}

__device__ __forceinline__ int fetch_code(const unsigned char *row, long long i, int bits, long long pitch)
{
    const long long bit = i * bits;
    const long long b0 = bit >> 3;
    uint32_t w = row[b0];
    if (b0 + 1 < pitch) w |= (uint32_t)row[b0 + 1] << 8;
    return (int)((w >> (bit & 7)) & ((1u << bits) - 1u));
}

// one warp per output row; lane-strided over the input channels
template <class D>
__global__ void __launch_bounds__(256)
bias_gemv_kernel(const uint16_t *__restrict__ W, long long C_out, long long C_in, long long ld,
                 const float *__restrict__ s, const unsigned char *__restrict__ codes,
                 const float *__restrict__ step, const int *__restrict__ zp, const float *__restrict__ mu_hat,
                 int bits, int gran, int group, const uint16_t *__restrict__ bias_in, uint16_t *__restrict__ bias_out,
                 float *__restrict__ bias_out_f32, int bias_bf16)
{
    pdl_begin();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= C_out) return;
    const long long pitch = C_in * bits / 8;
    const unsigned char *crow = codes + row * pitch;
    const long long ngroups = gran == AWEQ_PER_GROUP ? C_in / group : 1;
    float acc = 0.0f;
    for (long long j = lane; j < C_in; j += 32) {
        const long long k = gran == AWEQ_PER_TENSOR ? 0 : (gran == AWEQ_PER_ROW ? row : row * ngroups + j / group);
        const float w = D::one(W[row * ld + j]);
        const float wh = s ? __fmul_rn(w, s[j]) : w;
        const int q = fetch_code(crow, j, bits, pitch);
        const float rq = (float)((long long)q - (long long)zp[k]);
        const float eps = __fmaf_rn(step[k], rq, -wh);
        acc = __fmaf_rn(eps, mu_hat[j], acc);
    }
    acc = warp_sum(acc);
    if (lane == 0) write_bias(row, acc, bias_in, bias_out, bias_out_f32, bias_bf16);
}

aweq_status run_bias_apply(const float *epsmu, const void *bias_in, void *bias_out, float *bias_out_f32,
                           aweq_dtype bias_dt, long long C_out, cudaStream_t stream)
{
    const int t = 256;
    const unsigned g = (unsigned)((C_out + t - 1) / t);
    AWEQ_LAUNCH(bias_apply_kernel, dim3(g), dim3(t), 0, stream, epsmu, (const uint16_t *)bias_in, (uint16_t *)bias_out,
                bias_out_f32, (int)(bias_dt == AWEQ_BF16), C_out);
    return AWEQ_OK;
}

aweq_status run_bias_gemv(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ld,
                          const float *s, const unsigned char *codes, const float *step, const int *zp,
                          const float *mu_hat, int bits, int gran, int group, const void *bias_in, void *bias_out,
                          float *bias_out_f32, aweq_dtype bias_dt, cudaStream_t stream)
{
    const unsigned g = (unsigned)((C_out + 7) / 8);
    if (dt == AWEQ_F16)
        AWEQ_LAUNCH(bias_gemv_kernel<F16>, dim3(g), dim3(256), 0, stream, (const uint16_t *)W, C_out, C_in, ld, s, codes,
                    step, zp, mu_hat, bits, gran, group, (const uint16_t *)bias_in, (uint16_t *)bias_out, bias_out_f32,
                    (int)(bias_dt == AWEQ_BF16));
    else
        AWEQ_LAUNCH(bias_gemv_kernel<BF16>, dim3(g), dim3(256), 0, stream, (const uint16_t *)W, C_out, C_in, ld, s, codes,
                    step, zp, mu_hat, bits, gran, group, (const uint16_t *)bias_in, (uint16_t *)bias_out, bias_out_f32,
                    (int)(bias_dt == AWEQ_BF16));
    return AWEQ_OK;
}

}  // namespace aweq
