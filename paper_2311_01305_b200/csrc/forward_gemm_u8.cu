// unsigned 8-bit x unsigned 8-bit -> int32 instantiation of the forward-check GEMM.
#include "forward_gemm.cuh"

namespace aweq {
#ifndef AWEQ_NO_CUTLASS
aweq_status fc_gemm_u8(const void *A, const void *B, void *C, int M, int N, int K, long long ld, void *scratch,
        size_t scratch_bytes, cudaStream_t stream)
{
    using G = FcGemm<uint8_t, uint8_t, int32_t, int32_t, 16, Shape<_256, _256, _128>, Shape<_2, _1, _1>>;
    return G::run(reinterpret_cast<const uint8_t *>(A), reinterpret_cast<const uint8_t *>(B), reinterpret_cast<int32_t *>(C), M, N,
                  K, ld, scratch, scratch_bytes, stream);
}
#else
aweq_status fc_gemm_u8(const void *, const void *, void *, int, int, int, long long, void *, size_t, cudaStream_t)
{
    return AWEQ_ERR_UNSUPPORTED;
}
#endif
}  // namespace aweq
