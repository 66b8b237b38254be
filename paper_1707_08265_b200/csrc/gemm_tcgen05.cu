// InnerProduct contraction C[M,N] = A[M,K] * B[N,K]^T (bf16 operands, fp32 accumulate).
#include <cuda_runtime.h>

#include "plan.h"

namespace dragon {

int launch_gemm_bf16(const void* A, const void* B, void* C, int c_dtype, int M, int N, int K, int* status, cudaStream_t st) {
  (void)A; (void)B; (void)C; (void)c_dtype; (void)M; (void)N; (void)K; (void)status; (void)st;
  set_error("InnerProduct: the tensor-core contraction is not built into this library yet");
  return DRAGON_ERR_UNSUPPORTED;
}

}  // namespace dragon
