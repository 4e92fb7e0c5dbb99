// fp16 -> binary32 instantiation of the forward-check GEMM.
#include "forward_gemm.cuh"

namespace aweq {
#ifndef AWEQ_NO_CUTLASS
aweq_status fc_gemm_f16(const void *A, const void *B, void *C, int M, int N, int K, long long ld, void *scratch,
        size_t scratch_bytes, cudaStream_t stream)
{
    using G = FcGemm<cutlass::half_t, cutlass::half_t, float, float, 8, Shape<_256, _256, _64>, Shape<_2, _1, _1>>;
    return G::run(reinterpret_cast<const cutlass::half_t *>(A), reinterpret_cast<const cutlass::half_t *>(B), reinterpret_cast<float *>(C), M, N,
                  K, ld, scratch, scratch_bytes, stream);
}
#else
aweq_status fc_gemm_f16(const void *, const void *, void *, int, int, int, long long, void *, size_t, cudaStream_t)
{
    return AWEQ_ERR_UNSUPPORTED;
}
#endif
}  // namespace aweq
