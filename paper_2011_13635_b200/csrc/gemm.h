// Dense contraction with the step's fused epilogue; see mslt_gemm_desc in mslt.h.
//   D[z][m][n] = epilogue(alpha * sum_k A[z](m,k) * B[z](n,k))
// dtype 0: fp32 CUDA-core kernel (gemm_simt.cu); dtype 1: bf16 tcgen05 kernel (gemm_tc.cu).
#pragma once
#include <cuda_runtime.h>

#include "../../include/mslt.h"

namespace mslt {

// Enqueues the contraction on `st`.  `status` is a device word that a tensor-core kernel ORs an
// error bit into when one of its bounded waits runs out.  Returns 0, or a negative mslt_status
// with a message in `err` (at least 256 bytes).
int gemm_launch(const mslt_gemm_desc& d, int* status, cudaStream_t st, char* err);

int gemm_simt_launch(const mslt_gemm_desc& d, cudaStream_t st, char* err);
int gemm_tc_launch(const mslt_gemm_desc& d, int* status, cudaStream_t st, char* err);

// Test hook: the next tensor-core launch gets a producer that issues no copies and a wait limit of
// about 20 ms, so that its first wait runs out and the give-up path is exercised.
void gemm_tc_starve_next(int on);

// Kernels launched by the GEMM front end since the library was loaded (for launch accounting).
int64_t gemm_launches();

}  // namespace mslt
