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
// Measurement hook: 0 = automatic tiling, 1 = one CTA per tile, 2 = CTA pairs wherever possible.
void gemm_tc_set_variant(int variant);

// Fused attention forward (attn_tc.cu) for bf16, head width 64 and at most 512 keys per row:
//   probs[b,h,i,:] = softmax over valid keys j < seq_lens[b] of scale * q_i . k_j,  ctx = probs * v.
// qkv is the fused projection [B*S, 3*A*d] (queries, keys, values; head h in columns h*d..);
// probs ([B, A, S, S], may be null: not written) and ctx ([B*S, A*d]) are outputs.  `status` as for
// gemm_launch.  Returns 0 or a negative mslt_status with a message in `err`.
int attn_fwd_launch(const void* qkv, void* probs, void* ctx, const int* seq_lens, int B, int S, int A, int d,
                    float scale, int* status, cudaStream_t st, char* err);
// Its backward: dqkv ([B*S, 3*A*d], queries | keys | values like qkv) from the saved probabilities
// and the gradient of the context dctx ([B*S, A*d]); S a multiple of 8.
//   dV = P^T dC,  dP = dC V^T,  dS = P o (dP - rowsum(dP o P)) * scale,  dQ = dS K,  dK = dS^T Q
int attn_bwd_launch(const void* qkv, const void* probs, const void* dctx, void* dqkv, int B, int S, int A, int d,
                    float scale, int* status, cudaStream_t st, char* err);
long long attn_launches();
// Test hook like gemm_tc_starve_next, for the next attention launch (forward or backward).
void attn_starve_next(int on);

// Kernels launched by the GEMM front end since the library was loaded (for launch accounting).
int64_t gemm_launches();

}  // namespace mslt
