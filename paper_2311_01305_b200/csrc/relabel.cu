// Signed relabelling of 8-bit codes.  Eq. 1 produces unsigned codes q in [0, 255] with a
// zero-point Z; integer GEMM paths that take signed 8-bit operands want q' = q - 128 in
// [-128, 127] with Z' = Z - 128, which de-quantises to the same values: Step (q' - Z') = Step (q - Z).
// Subtracting 128 modulo 256 is flipping the top bit of every byte.
#include "common.cuh"
#include "kernels.h"

namespace aweq {

__global__ void __launch_bounds__(256) relabel_kernel(const unsigned char *__restrict__ codes, long long n,
                                                      unsigned char *__restrict__ out, const int *__restrict__ zp,
                                                      long long nz, int *__restrict__ zp_out)
{
    pdl_begin();
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long stride = (long long)gridDim.x * blockDim.x;
    const bool vec = ((reinterpret_cast<uintptr_t>(codes) | reinterpret_cast<uintptr_t>(out)) & 15) == 0;
    const long long nv = vec ? n / 16 : 0;
    for (long long i = tid; i < nv; i += stride) {
        uint4 v = ldg_stream(codes + i * 16);
        v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
        *reinterpret_cast<uint4 *>(out + i * 16) = v;
    }
    for (long long i = nv * 16 + tid; i < n; i += stride) out[i] = codes[i] ^ 0x80u;
    if (zp && zp_out)
        for (long long k = tid; k < nz; k += stride) {
            int z;
            asm("sub.sat.s32 %0, %1, 128;" : "=r"(z) : "r"(zp[k]));      // zero-points saturate like everywhere else
            zp_out[k] = z;
        }
}

aweq_status run_relabel_signed(const unsigned char *codes, long long n, signed char *out, const int *zp, long long nz,
                               int *zp_out, cudaStream_t stream)
{
    long long work = n / 16 > nz ? n / 16 : nz;
    long long blocks = (work + 255) / 256;
    if (blocks > (long long)kSmCount * 16) blocks = (long long)kSmCount * 16;
    if (blocks < 1) blocks = 1;
    AWEQ_LAUNCH(relabel_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, codes, n,
                reinterpret_cast<unsigned char *>(out), zp, nz, zp_out);
    return AWEQ_OK;
}

}  // namespace aweq
