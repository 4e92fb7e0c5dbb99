// Folding diag(s)^-1 into whatever produces a layer input (Section 3.1, the text after
// Eq. 3: the division of the activations by s is fused into the previous block, so the
// equalised model runs the same operations as the original one).  The producer is either a
// normalisation layer -- its per-channel gain and shift are scaled by 1/s_j -- or a linear
// layer whose output channel j is this input's channel j -- row j of its weight matrix and
// element j of its bias are scaled by 1/s_j.  Both are "scale row r of a 16-bit matrix by
// rinv[r]" (a vector is a matrix with one column):
//     out[r, c] = round16( float(P[r, c]) * rinv[r] )       binary32 product, then one
//                                                            round-to-nearest-even to 16 bits
#include "common.cuh"
#include "kernels.h"

namespace aweq {

// rows of eight-element vectors; one vector per thread, grid-stride
template <class D>
__global__ void __launch_bounds__(256) fold_vec_kernel(const uint16_t *__restrict__ P, long long rows, int nvec,
                                                       long long ld, const float *__restrict__ rinv,
                                                       uint16_t *__restrict__ out, long long ld_out)
{
    pdl_begin();
    const long long total = rows * nvec;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / nvec;
        const int v = (int)(i - r * nvec);
        const float k = __ldg(rinv + r);
        float f[8];
        widen8<D>(ldg_stream(P + r * ld + v * 8), f);
        uint4 o;
        o.x = (uint32_t)D::encode(f[0] * k) | ((uint32_t)D::encode(f[1] * k) << 16);
        o.y = (uint32_t)D::encode(f[2] * k) | ((uint32_t)D::encode(f[3] * k) << 16);
        o.z = (uint32_t)D::encode(f[4] * k) | ((uint32_t)D::encode(f[5] * k) << 16);
        o.w = (uint32_t)D::encode(f[6] * k) | ((uint32_t)D::encode(f[7] * k) << 16);
        *reinterpret_cast<uint4 *>(out + r * ld_out + v * 8) = o;
    }
}

// any shape (vectors, odd widths): one element per thread
template <class D>
__global__ void __launch_bounds__(256) fold_elem_kernel(const uint16_t *__restrict__ P, long long rows, long long cols,
                                                        long long ld, const float *__restrict__ rinv,
                                                        uint16_t *__restrict__ out, long long ld_out)
{
    pdl_begin();
    const long long total = rows * cols;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / cols, c = i - r * cols;
        out[r * ld_out + c] = D::encode(D::one(P[r * ld + c]) * __ldg(rinv + r));
    }
}

aweq_status run_fold_scale(const void *P, aweq_dtype dt, long long rows, long long cols, long long ld,
                           const float *rinv, void *out, long long ld_out, cudaStream_t stream)
{
    const uint16_t *src = reinterpret_cast<const uint16_t *>(P);
    uint16_t *dst = reinterpret_cast<uint16_t *>(out);
    const bool vec = cols % 8 == 0 && ld % 8 == 0 && ld_out % 8 == 0 && (reinterpret_cast<uintptr_t>(P) & 15) == 0 &&
                     (reinterpret_cast<uintptr_t>(out) & 15) == 0;
    const long long work = vec ? rows * (cols / 8) : rows * cols;
    long long blocks = (work + 255) / 256;
    const long long cap = (long long)kSmCount * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (vec) {
        if (dt == AWEQ_F16)
            AWEQ_LAUNCH(fold_vec_kernel<F16>, dim3((unsigned)blocks), dim3(256), 0, stream, src, rows, (int)(cols / 8), ld,
                        rinv, dst, ld_out);
        else
            AWEQ_LAUNCH(fold_vec_kernel<BF16>, dim3((unsigned)blocks), dim3(256), 0, stream, src, rows, (int)(cols / 8),
                        ld, rinv, dst, ld_out);
    } else {
        if (dt == AWEQ_F16)
            AWEQ_LAUNCH(fold_elem_kernel<F16>, dim3((unsigned)blocks), dim3(256), 0, stream, src, rows, cols, ld, rinv,
                        dst, ld_out);
        else
            AWEQ_LAUNCH(fold_elem_kernel<BF16>, dim3((unsigned)blocks), dim3(256), 0, stream, src, rows, cols, ld, rinv,
                        dst, ld_out);
    }
    return AWEQ_OK;
}

}  // namespace aweq
