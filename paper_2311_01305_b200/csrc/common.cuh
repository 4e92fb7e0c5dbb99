// Shared device helpers of the AWEQ kernels (sm_100a only): 16-bit type
// traits, mbarrier / bulk-copy (TMA) wrappers with bounded waits, warp
// reductions and the scalar pieces of the Eq. 1-2 quantiser.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/aweq.h"

namespace aweq {

constexpr int kSmCount = 148;              // B200
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // a wait longer than 2 s is reported, not spun on

// ------------------------------------------------------------------ host side
void note_launch();                        // bumps the launch counter
aweq_status cuda_failed(cudaError_t e);    // records the error text, returns AWEQ_ERR_CUDA

#define AWEQ_CUDA_OK(expr)                                   \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) return ::aweq::cuda_failed(e__); \
    } while (0)

#define AWEQ_LAUNCH_CHECK()                                  \
    do {                                                     \
        ::aweq::note_launch();                               \
        cudaError_t e__ = cudaGetLastError();                \
        if (e__ != cudaSuccess) return ::aweq::cuda_failed(e__); \
    } while (0)

#define AWEQ_LAUNCH(...)                                     \
    do {                                                     \
        cudaError_t e__ = ::aweq::launch_pdl(__VA_ARGS__);   \
        ::aweq::note_launch();                               \
        if (e__ != cudaSuccess) return ::aweq::cuda_failed(e__); \
    } while (0)

// ------------------------------------------------------------------ programmatic dependent launch
// Every kernel of the library is launched with programmatic stream serialisation: the next
// kernel of the stream may be scheduled while this one drains, and waits (pdl_wait, first
// statement that touches global memory) until everything before it has completed and is
// visible.  That removes most of the launch gap between the many short kernels of a pass.
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
// the same launch for a kernel whose CTAs form clusters of `cluster` along x
template <class... KArgs, class... Args>
inline cudaError_t launch_pdl_cluster(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                      unsigned cluster, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}
__device__ __forceinline__ void pdl_begin()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------ 16-bit traits
struct F16 {
    using T2 = __half2;
    static __device__ __forceinline__ T2 from_bits(uint32_t u) { return *reinterpret_cast<T2 *>(&u); }
    static __device__ __forceinline__ uint32_t pos_inf2() { return 0x7C007C00u; }
    static __device__ __forceinline__ uint32_t neg_inf2() { return 0xFC00FC00u; }
    // fp16 -> binary32 as "x + (-0)" with the mixed-precision add of sm_100 (exact, signed zeros
    // included): it issues on the FMA pipe, whereas cvt.f32.f16 goes through the conversion unit,
    // which the row quantisers saturated (16 conversions per 16 bytes of input)
    static __device__ __forceinline__ float2 to_float2(T2 v)
    {
        float2 r;
        asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\t"
            "add.rn.f32.f16 %0, l, 0f80000000;\n\tadd.rn.f32.f16 %1, h, 0f80000000;\n\t}"
            : "=f"(r.x), "=f"(r.y) : "r"(*reinterpret_cast<const uint32_t *>(&v)));
        return r;
    }
    static __device__ __forceinline__ float one(uint16_t b) { return __half2float(__ushort_as_half(b)); }
    static __device__ __forceinline__ uint16_t encode(float f) { return __half_as_ushort(__float2half_rn(f)); }
};
struct BF16 {
    using T2 = __nv_bfloat162;
    static __device__ __forceinline__ T2 from_bits(uint32_t u) { return *reinterpret_cast<T2 *>(&u); }
    static __device__ __forceinline__ uint32_t pos_inf2() { return 0x7F807F80u; }
    static __device__ __forceinline__ uint32_t neg_inf2() { return 0xFF80FF80u; }
    static __device__ __forceinline__ float2 to_float2(T2 v)
    {
        uint32_t u = *reinterpret_cast<uint32_t *>(&v);    // bf16 is the upper half of a binary32
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
    }
    static __device__ __forceinline__ float one(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
    static __device__ __forceinline__ uint16_t encode(float f) { return __bfloat16_as_ushort(__float2bfloat16_rn(f)); }
};

// widen the 8 elements of a 16-byte vector
template <class D>
__device__ __forceinline__ void widen8(const uint4 &v, float (&f)[8])
{
    float2 a = D::to_float2(D::from_bits(v.x)), b = D::to_float2(D::from_bits(v.y));
    float2 c = D::to_float2(D::from_bits(v.z)), d = D::to_float2(D::from_bits(v.w));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

// ------------------------------------------------------------------ loads
__device__ __forceinline__ uint4 ldg_stream(const void *p)   // read-once data: bypass L1 allocation
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ldg_f4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ void load8(const float *p, float (&f)[8])
{
    float4 a = ldg_f4(p), b = ldg_f4(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

// ------------------------------------------------------------------ mbarrier + bulk copy
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Wait for a phase of the barrier; gives up after kWaitLimitNs and returns false.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > kWaitLimitNs) return false;
    }
}
// 1-D bulk copy global -> this CTA's shared memory, completion on an mbarrier.
// Both addresses 16-byte aligned, bytes a multiple of 16.  The copy lands in this CTA only.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// ------------------------------------------------------------------ thread-block clusters
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in the CTA `rank` of this cluster
__device__ __forceinline__ uint32_t cluster_map(const void *p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_store_f2(uint32_t remote, float a, float b)
{
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(remote), "f"(a), "f"(b) : "memory");
}
// arrive on an mbarrier of another CTA of the cluster; releases this thread's earlier stores to it
__device__ __forceinline__ void cluster_mbar_arrive(uint32_t remote_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
}
// bounded wait on a local mbarrier that CTAs of the cluster arrive on
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;      // the clock is read only when the wait is a real one
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (global_ns() - t0 > kWaitLimitNs) return false;
    }
}
// every CTA of the cluster has arrived (and none has left) -- only at points that every CTA reaches
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void named_bar_sync(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// barrier over `threads` threads that also ANDs a predicate (all arrive, all get the same answer)
__device__ __forceinline__ bool named_bar_and(int id, int threads, bool pred)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"(id), "r"(threads), "r"((uint32_t)pred) : "memory");
    return r != 0;
}

// three-input min / max (one instruction on sm_100)
__device__ __forceinline__ float fmin3(float a, float b, float c)
{
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// ------------------------------------------------------------------ warp reductions
__device__ __forceinline__ float redux_min(float v, uint32_t mask)
{
    float r;
    asm volatile("redux.sync.min.f32 %0, %1, %2;" : "=f"(r) : "f"(v), "r"(mask));
    return r;
}
__device__ __forceinline__ float redux_max(float v, uint32_t mask)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, %2;" : "=f"(r) : "f"(v), "r"(mask));
    return r;
}
__device__ __forceinline__ float warp_sum(float v)      // fixed butterfly order: reproducible
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ------------------------------------------------------------------ Eq. 15, last step
struct BiasIO {
    const uint16_t *in;      // 16-bit bias of the layer, or NULL (no bias)
    uint16_t *out;           // corrected bias, 16-bit (may be NULL)
    float *out_f32;          // corrected bias, binary32 (may be NULL)
    int bf16;                // 16-bit type of in / out
};
// bias'[o] = bias[o] - delta, written as binary32 and / or in the 16-bit bias type
__device__ __forceinline__ void write_bias(long long o, float delta, const uint16_t *bias_in, uint16_t *bias_out,
                                           float *bias_out_f32, int bias_bf16)
{
    float b = 0.0f;
    if (bias_in) b = bias_bf16 ? BF16::one(bias_in[o]) : F16::one(bias_in[o]);
    const float c = __fsub_rn(b, delta);
    if (bias_out_f32) bias_out_f32[o] = c;
    if (bias_out) bias_out[o] = bias_bf16 ? BF16::encode(c) : F16::encode(c);
}


// ------------------------------------------------------------------ Eq. 1-2, scalar part
// (Step, 1/Step, Z) of a vector with extremes lo, hi; all IEEE binary32, no FMA.
struct QParams {
    float step, inv;
    int zp;
    bool fast;      // |Z| small enough for the add-magic rounding path
};
__device__ __forceinline__ QParams make_qparams(float lo, float hi, int qmax)
{
    QParams p;
    float st = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
    if (!(st > 0.0f)) st = (lo != 0.0f) ? fabsf(lo) : 1.0f;      // constant vector
    p.step = st;
    p.inv = __frcp_rn(st);                                       // correctly rounded 1 / Step
    const float z = __fmul_rn(lo, p.inv);
    int zi;
    asm("cvt.rni.sat.s32.f32 %0, %1;" : "=r"(zi) : "f"(-z));    // saturating; NaN -> 0
    p.zp = zi;
    // |lo / Step| < 4e6 keeps every clamped value below 2^22, where adding 1.5 * 2^23 rounds
    // exactly like rint; an infinite 1 / Step makes z infinite or NaN and fails the test.  An
    // infinite Step (an infinite element in the vector) has 1 / Step = 0 and z = 0: it must
    // take the literal path too, where Inf * 0 = NaN becomes code Z as the definition says
    p.fast = fabsf(z) < 4.0e6f && st <= 3.0e38f;
    return p;
}
// exact reference form of one code: clamp(rint(fl(v*inv)) + Z, 0, qmax) with saturating int32
__device__ __forceinline__ int code_generic(float v, float inv, int zp, int qmax)
{
    int t, q;
    asm("cvt.rni.sat.s32.f32 %0, %1;" : "=r"(t) : "f"(__fmul_rn(v, inv)));
    asm("add.sat.s32 %0, %1, %2;" : "=r"(q) : "r"(t), "r"(zp));
    return min(max(q, 0), qmax);
}
// flags travelling with a (Step, inv, Z) triple
constexpr int kQFast = 1;       // add-constant rounding is valid
constexpr int kQNoClamp = 2;    // the upper clamp cannot fire

__device__ __forceinline__ int qflags(const QParams &q, float hi, int qmax)
{
    int top;
    asm("cvt.rni.sat.s32.f32 %0, %1;" : "=r"(top) : "f"(__fmul_rn(hi, q.inv)));
    // with q.fast both terms are below 2^22 in magnitude: no overflow
    return q.fast ? (kQFast | ((top + q.zp <= qmax) ? kQNoClamp : 0)) : 0;
}

constexpr float kMagic = 12582912.0f;            // 1.5 * 2^23: adding it rounds to an integer, ties to even
constexpr int kMagicBits = 0x4B400000;

}  // namespace aweq
