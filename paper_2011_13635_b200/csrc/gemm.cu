// Front end of the dense contraction: validates the descriptor and picks the kernel.
// dtype 0 runs on the CUDA cores in fp32; dtype 1 on the tcgen05 tensor cores.
#include <stdio.h>
#include <stdlib.h>

#include <atomic>

#include "gemm.h"

namespace mslt {

static std::atomic<int64_t> g_launches{0};
int64_t gemm_launches() { return g_launches.load(); }

int gemm_launch(const mslt_gemm_desc& d, int* status, cudaStream_t st, char* err) {
  if ((d.a_rs != 1 && d.a_ks != 1) || (d.b_rs != 1 && d.b_ks != 1)) {
    snprintf(err, 256, "gemm: each operand needs one unit stride");
    return MSLT_ERR_ARG;
  }
  int rc;
  if (d.dtype == 1) {
    // MSLT_BF16_CUDA_CORES=1 routes bf16 products to the CUDA-core kernel: a debugging aid for
    // telling a tensor-core kernel fault from an orchestration fault, never a silent fallback.
    static const bool cuda_cores = getenv("MSLT_BF16_CUDA_CORES") && atoi(getenv("MSLT_BF16_CUDA_CORES")) == 1;
    rc = cuda_cores ? gemm_simt_launch(d, st, err) : gemm_tc_launch(d, status, st, err);
  } else if (d.dtype == 0) {
    rc = gemm_simt_launch(d, st, err);
  } else {
    snprintf(err, 256, "gemm: unknown dtype %d", d.dtype);
    return MSLT_ERR_ARG;
  }
  if (rc == 0) g_launches.fetch_add(1);
  return rc;
}

}  // namespace mslt
