// Internal launch functions behind the C ABI (one per kernel family).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#include "../../include/aweq.h"
#include "common.cuh"

namespace aweq {

size_t colreduce_ws_bytes(long long rows, long long cols);
void colreduce_describe(long long rows, long long cols, long long plan[8]);
bool rowquant_describe(long long rows, long long cols, bool weights, long long plan[8]);

aweq_status run_stats(const void *X, aweq_dtype dt, long long N, long long C, long long ld, float *xmin, float *xmax,
                      float *xmean, double *xsum, long long *count, int accumulate, void *ws, aweq_dev_status *st,
                      cudaStream_t stream, float *negmin_max = nullptr, double *sum_count = nullptr);
// steps 1 and 2 of one input in one launch (n_w <= 3 matrices); ws: colreduce_fused_ws_bytes
size_t colreduce_fused_ws_bytes(long long rows, long long cols);
bool stats_wrange_fusable(long long N, long long C_in, const long long *C_out, int n_w);
aweq_status run_stats_wrange(const void *X, aweq_dtype dt, long long N, long long C, long long ld, float *xmin,
                             float *xmax, float *xmean, const void *const *W, const long long *C_out,
                             const long long *ldw, int n_w, float *wmin, float *wmax, void *ws, aweq_dev_status *st,
                             cudaStream_t stream, float *negmin_max = nullptr, double *sum_count = nullptr);
aweq_status run_stats_from_exchange(const float *negmin_max, const double *sum_count, long long C, float *xmin,
                                    float *xmax, float *xmean, cudaStream_t stream);
aweq_status run_wrange(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ld, float *wmin,
                       float *wmax, int accumulate, void *ws, aweq_dev_status *st, cudaStream_t stream);
aweq_status run_wrange_multi(const void *const *W, const long long *C_out, const long long *ld, int n, aweq_dtype dt,
                             long long C_in, float *wmin, float *wmax, int accumulate, void *ws, aweq_dev_status *st,
                             cudaStream_t stream);
aweq_status run_factors(const float *xmin, const float *xmax, const float *xmean, const float *wmin,
                        const float *wmax, long long C, float *s, float *rinv, float *mu_hat, float *pX, float *pW,
                        double *scalars, aweq_dev_status *st, cudaStream_t stream, int criterion = 0);
bool rowquant_supported(long long nrows, long long cols);
aweq_status run_rowquant(const void *X, aweq_dtype dt, long long nrows, long long cols, long long ld,
                         const float *scale, const float *mu, int bits, bool weights, unsigned char *out,
                         float *step, int *zp, float *epsmu, const BiasIO &bias, aweq_dev_status *st,
                         cudaStream_t stream);
aweq_status run_warpquant(const void *X, aweq_dtype dt, long long nrows, long long cols, long long ld,
                          const float *scale, const float *mu, int bits, bool weights, int group,
                          const float *lo_hi, unsigned char *out, float *step, int *zp, float *epsmu,
                          const BiasIO &bias, aweq_dev_status *st, cudaStream_t stream);
// group-128 quantiser with column windows (3, 4 or 8 bits); ws: groupquant_ws_bytes
bool groupquant_supported(int bits, int group);
size_t groupquant_ws_bytes(long long rows, long long cols);
aweq_status run_groupquant(const void *W, aweq_dtype dt, long long nrows, long long cols, long long ld,
                           const float *scale, const float *mu, int bits, unsigned char *out, float *step, int *zp,
                           float *epsmu, const BiasIO &bias, void *ws, cudaStream_t stream);
aweq_status run_scaled_tensor_range(const float *cmin, const float *cmax, const float *scale, long long C,
                                    float *lo_hi, cudaStream_t stream);
aweq_status run_bias_apply(const float *epsmu, const void *bias_in, void *bias_out, float *bias_out_f32,
                           aweq_dtype bias_dt, long long C_out, cudaStream_t stream);
aweq_status run_bias_gemv(const void *W, aweq_dtype dt, long long C_out, long long C_in, long long ld,
                          const float *s, const unsigned char *codes, const float *step, const int *zp,
                          const float *mu_hat, int bits, int gran, int group, const void *bias_in, void *bias_out,
                          float *bias_out_f32, aweq_dtype bias_dt, cudaStream_t stream);

aweq_status run_fold_scale(const void *P, aweq_dtype dt, long long rows, long long cols, long long ld,
                           const float *rinv, void *out, long long ld_out, cudaStream_t stream);

aweq_status run_relabel_signed(const unsigned char *codes, long long n, signed char *out, const int *zp, long long nz,
                               int *zp_out, cudaStream_t stream);

// forward check (tensor-core GEMMs + comparison)
size_t forward_check_ws_bytes(long long N, long long C_in, long long C_out);
aweq_status run_forward_check(const unsigned char *Xq, const float *act_step, const int *act_zp,
                              const unsigned char *Wq, const float *w_step, const int *w_zp, const float *bias_q,
                              const void *X, const void *W, aweq_dtype dt, const void *bias, long long N,
                              long long C_in, long long C_out, double *mean_err, double *sums, void *ws,
                              size_t ws_bytes, cudaStream_t stream);
size_t forward_check_weights_ws_bytes(long long N, long long C_in, long long C_out);
aweq_status run_forward_check_weights(const unsigned char *codes, const float *step, const int *zp, int bits, int gran,
                                      int group, const float *rinv, const float *bias_q, const void *X, const void *W,
                                      aweq_dtype dt, const void *bias, long long N, long long C_in, long long C_out,
                                      double *mean_err, double *sums, void *ws, size_t ws_bytes, cudaStream_t stream);
// C[M x N] = A[M x K] B[N x K]^T on the tensor cores; A and B have ld elements per row
aweq_status fc_gemm_u8(const void *A, const void *B, void *C, int M, int N, int K, long long ld, void *scratch,
                       size_t scratch_bytes, cudaStream_t stream);
aweq_status fc_gemm_f16(const void *A, const void *B, void *C, int M, int N, int K, long long ld, void *scratch,
                        size_t scratch_bytes, cudaStream_t stream);
aweq_status fc_gemm_bf16(const void *A, const void *B, void *C, int M, int N, int K, long long ld, void *scratch,
                         size_t scratch_bytes, cudaStream_t stream);

}  // namespace aweq
