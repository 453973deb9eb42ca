// tcgen05 GEMM, operand layout "fwd" (see des_tc_gemm.cuh).
#include "des_tc_gemm.cuh"
DES_DEFINE_TC_GEMM(TcGemm_fwd, cutlass::layout::RowMajor, cutlass::layout::RowMajor)
int des_tc_gemm_fwd(int M, int N, int K, int L, const void* A, const void* B, const float* C, float* D, float beta, void* ws,
                   size_t ws_bytes, cudaStream_t stream) {
  DES_TC_GEMM_BODY(TcGemm_fwd)
}
