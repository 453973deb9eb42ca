// tcgen05 (5th-generation tensor core) GEMM for the row-split first dense
// layer: bf16 operands staged by TMA, fp32 accumulators in tensor memory,
// built from the CUTLASS / CuTe sm100 collective templates (the header tree
// ships with the Python environment; nothing of it is copied here).  One
// translation unit per operand layout, each exporting one plain function:
//
//   rc = f(M, N, K, L, A, B, C, D, beta, workspace, workspace_bytes, stream)
//        D[l][M][N] (fp32, row-major) = A_l * B_l + beta * C[l]   for l < L,
//        where the K extent of A and B is cut into L consecutive pieces of K each (a batched
//        GEMM over packed operands: with L > 1 this is a split-K product whose L partial
//        results the caller adds up; L = 1 is the plain product)
//   rc: 0 ok; 1 shape / alignment not supported by the TMA path (caller falls
//       back to the CUDA-core kernel); 2 workspace too small; 3, 4 CUTLASS error.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#if defined(DES_TC_GEMM_DECL_ONLY)
/* prototypes only */
#elif !defined(DES_NO_CUTLASS)
#include "cutlass/cutlass.h"
#include "cute/tensor.hpp"
#include "cutlass/gemm/device/gemm_universal_adapter.h"
#include "cutlass/gemm/kernel/gemm_universal.hpp"
#include "cutlass/gemm/collective/collective_builder.hpp"
#include "cutlass/epilogue/collective/collective_builder.hpp"
#include "cutlass/util/packed_stride.hpp"

// LayoutA: RowMajor = K contiguous, ColumnMajor = M contiguous.
// LayoutB: ColumnMajor = K contiguous, RowMajor = N contiguous.
#define DES_DEFINE_TC_GEMM(NAME, LayoutA, LayoutB)                                                                    \
  struct NAME {                                                                                                       \
    using ElementA = cutlass::bfloat16_t;                                                                             \
    using ElementB = cutlass::bfloat16_t;                                                                             \
    using ElementC = float;                                                                                           \
    using LayoutC = cutlass::layout::RowMajor;                                                                        \
    using ElementAccumulator = float;                                                                                 \
    using ArchTag = cutlass::arch::Sm100;                                                                             \
    using OperatorClass = cutlass::arch::OpClassTensorOp;                                                             \
    using MmaTileShape = cute::Shape<cute::_128, cute::_128, cute::_64>;                                              \
    using ClusterShape = cute::Shape<cute::_1, cute::_1, cute::_1>; /* one CTA per tile, plain (non-cluster) TMA loads */        \
    using CollectiveEpilogue = cutlass::epilogue::collective::CollectiveBuilder<                                      \
        ArchTag, OperatorClass, MmaTileShape, ClusterShape, cutlass::epilogue::collective::EpilogueTileAuto,          \
        ElementAccumulator, ElementAccumulator, ElementC, LayoutC, 4, ElementC, LayoutC, 4,                           \
        cutlass::epilogue::collective::EpilogueScheduleAuto>::CollectiveOp;                                           \
    using CollectiveMainloop = cutlass::gemm::collective::CollectiveBuilder<                                          \
        ArchTag, OperatorClass, ElementA, LayoutA, 8, ElementB, LayoutB, 8, ElementAccumulator, MmaTileShape,         \
        ClusterShape,                                                                                                 \
        cutlass::gemm::collective::StageCountAutoCarveout<static_cast<int>(sizeof(CollectiveEpilogue::SharedStorage))>, \
        cutlass::gemm::collective::KernelScheduleAuto>::CollectiveOp;                                                 \
    using GemmKernel = cutlass::gemm::kernel::GemmUniversal<cute::Shape<int, int, int, int>, CollectiveMainloop,      \
                                                            CollectiveEpilogue, void>;                                \
    using Gemm = cutlass::gemm::device::GemmUniversalAdapter<GemmKernel>;                                             \
    using StrideA = Gemm::GemmKernel::StrideA;                                                                        \
    using StrideB = Gemm::GemmKernel::StrideB;                                                                        \
    using StrideC = Gemm::GemmKernel::StrideC;                                                                        \
    using StrideD = Gemm::GemmKernel::StrideD;                                                                        \
    static int run(int M, int N, int K, int L, const void* A, const void* B, const float* C, float* D, float beta,    \
                   void* workspace, size_t ws_bytes, cudaStream_t stream) {                                           \
      StrideA sa = cutlass::make_cute_packed_stride(StrideA{}, cute::make_shape(M, K, L));                            \
      StrideB sb = cutlass::make_cute_packed_stride(StrideB{}, cute::make_shape(N, K, L));                            \
      StrideC sc = cutlass::make_cute_packed_stride(StrideC{}, cute::make_shape(M, N, L));                            \
      StrideD sd = cutlass::make_cute_packed_stride(StrideD{}, cute::make_shape(M, N, L));                            \
      Gemm::Arguments args{cutlass::gemm::GemmUniversalMode::kGemm,                                                   \
                           {M, N, K, L},                                                                              \
                           {(const ElementA*)A, sa, (const ElementB*)B, sb},                                          \
                           {{1.0f, beta}, C, sc, D, sd}};                                                             \
      Gemm gemm;                                                                                                      \
      if (gemm.can_implement(args) != cutlass::Status::kSuccess) return 1;                                            \
      if (Gemm::get_workspace_size(args) > ws_bytes) return 2;                                                        \
      if (gemm.initialize(args, workspace, stream) != cutlass::Status::kSuccess) return 3;                            \
      if (gemm.run(stream) != cutlass::Status::kSuccess) return 4;                                                    \
      return 0;                                                                                                       \
    }                                                                                                                 \
  };
#define DES_TC_GEMM_BODY(NAME) return NAME::run(M, N, K, L, A, B, C, D, beta, ws, ws_bytes, stream);
#else
#define DES_DEFINE_TC_GEMM(NAME, LayoutA, LayoutB)
#define DES_TC_GEMM_BODY(NAME) return 1;   /* built without the CUTLASS headers: CUDA-core fallback only */
#endif

// Z = V W: A = pooled bf16 [B][F*k] (K contiguous), B = W1 bf16 [F*k][H] (N contiguous)
int des_tc_gemm_fwd(int M, int N, int K, int L, const void* A, const void* B, const float* C, float* D, float beta, void* ws,
                    size_t ws_bytes, cudaStream_t stream);
// gE = gZ W1^T: A = gZ bf16 [B][H] (K contiguous), B = W1 bf16 [F*k][H] read as (N = F*k, K = H), K contiguous
int des_tc_gemm_dgrad(int M, int N, int K, int L, const void* A, const void* B, const float* C, float* D, float beta, void* ws,
                      size_t ws_bytes, cudaStream_t stream);
// gW1 = V^T gZ: A = pooled bf16 [B][F*k] read as (M = F*k, K = B), M contiguous; B = gZ bf16 [B][H] (N contiguous);
// L > 1 cuts the batch into L pieces (K = B / L samples each) whose partial products the caller adds
int des_tc_gemm_wgrad(int M, int N, int K, int L, const void* A, const void* B, const float* C, float* D, float beta, void* ws,
                      size_t ws_bytes, cudaStream_t stream);
