// Tensor-core GEMM of the forward check: the CUTLASS sm_100 collectives (tcgen05.mma with
// TMEM accumulators, TMA-fed shared-memory stages) instantiated for one operand type per
// translation unit.  C[M x N] = A[M x K] B[N x K]^T, both operands K-contiguous.
// The instantiations use 256 x 256 output tiles computed by CTA pairs (cta_group::2, cluster
// 2 x 1): each CTA of a pair stages half of the A and half of the B tile, so no operand is
// loaded twice and every TMA copy has a single destination CTA.  Of the tile shapes tried on layer-sized
// problems this one was the fastest for both operand types.
#pragma once
#include "common.cuh"
#include "kernels.h"

#ifndef AWEQ_NO_CUTLASS
#include "cutlass/cutlass.h"
#include "cute/tensor.hpp"
#include "cutlass/epilogue/collective/collective_builder.hpp"
#include "cutlass/gemm/collective/collective_builder.hpp"
#include "cutlass/gemm/device/gemm_universal_adapter.h"
#include "cutlass/gemm/kernel/gemm_universal.hpp"
#include "cutlass/util/packed_stride.hpp"

namespace aweq {
using namespace cute;


template <class EA, class EB, class EC, class EAcc, int AlignAB, class Tile, class Cluster = Shape<_1, _1, _1>>
struct FcGemm {
    using LayoutA = cutlass::layout::RowMajor;       // [M x K], K contiguous
    using LayoutB = cutlass::layout::ColumnMajor;    // [N x K] stored row-major = K contiguous
    using LayoutC = cutlass::layout::RowMajor;
    static constexpr int AlignC = 128 / cutlass::sizeof_bits<EC>::value;
    using Epi = typename cutlass::epilogue::collective::CollectiveBuilder<
        cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, Tile, Cluster,
        cutlass::epilogue::collective::EpilogueTileAuto, EAcc, EAcc, EC, LayoutC, AlignC, EC, LayoutC, AlignC,
        cutlass::epilogue::collective::EpilogueScheduleAuto>::CollectiveOp;
    using Main = typename cutlass::gemm::collective::CollectiveBuilder<
        cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, EA, LayoutA, AlignAB, EB, LayoutB, AlignAB, EAcc, Tile,
        Cluster,
        cutlass::gemm::collective::StageCountAutoCarveout<static_cast<int>(sizeof(typename Epi::SharedStorage))>,
        cutlass::gemm::collective::KernelScheduleAuto>::CollectiveOp;
    using Kernel = cutlass::gemm::kernel::GemmUniversal<Shape<int, int, int, int>, Main, Epi>;
    using Gemm = cutlass::gemm::device::GemmUniversalAdapter<Kernel>;

    // ld: elements between consecutive rows of A and of B (>= K: a K-slice of wider matrices)
    static aweq_status run(const EA *A, const EB *B, EC *C, int M, int N, int K, long long ld, void *scratch,
                           size_t scratch_bytes, cudaStream_t stream)
    {
        auto sA = cutlass::make_cute_packed_stride(typename Gemm::GemmKernel::StrideA{}, make_shape(M, (int)ld, 1));
        auto sB = cutlass::make_cute_packed_stride(typename Gemm::GemmKernel::StrideB{}, make_shape(N, (int)ld, 1));
        auto sC = cutlass::make_cute_packed_stride(typename Gemm::GemmKernel::StrideC{}, make_shape(M, N, 1));
        typename Gemm::Arguments args{cutlass::gemm::GemmUniversalMode::kGemm,
                                      {M, N, K, 1},
                                      {A, sA, B, sB},
                                      {{EAcc(1), EAcc(0)}, C, sC, C, sC}};
        Gemm gemm;
        if (gemm.can_implement(args) != cutlass::Status::kSuccess) return AWEQ_ERR_UNSUPPORTED;
        if (Gemm::get_workspace_size(args) > scratch_bytes) return AWEQ_ERR_WORKSPACE;
        if (gemm.initialize(args, scratch, stream) != cutlass::Status::kSuccess) return AWEQ_ERR_CUDA;
        if (gemm.run(stream) != cutlass::Status::kSuccess) return AWEQ_ERR_CUDA;
        note_launch();
        return AWEQ_OK;
    }
};

}  // namespace aweq
#endif
