// CUDA-core contraction for the fp32 path (and for any element type as a plain-ALU kernel):
// 64x64 output tile per block, 16-deep k slices in shared memory, 4x4 outputs per thread,
// fp32 accumulation in k order.  Operands are addressed by (row stride, k stride), so forward,
// input-gradient and weight-gradient products and the batched attention products all run here
// without transposed copies.  TF32 tensor cores are not used: the fp32 path is held to 1e-4.
#include <stdio.h>

#include "common.cuh"
#include "gemm.h"

namespace mslt {

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(mslt_gemm_desc d) {
  __shared__ float As[16][64 + 4];
  __shared__ float Bs[16][64 + 4];
  const int z = blockIdx.z;
  const int zo = z / d.hdiv, zi = z % d.hdiv;
  const T* A = (const T*)d.A + zo * d.a_bo + zi * d.a_bi;
  const T* B = (const T*)d.B + zo * d.b_bo + zi * d.b_bi;
  const int64_t doff = zo * d.d_bo + zi * d.d_bi;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < d.K; k0 += 16) {
#pragma unroll
    for (int i = 0; i < 4; i++) {
      const int idx = tid + i * 256;
      int r, k;
      if (d.a_ks == 1) { k = idx & 15; r = idx >> 4; } else { r = idx & 63; k = idx >> 6; }
      float v = 0.f;
      if (m0 + r < d.M && k0 + k < d.K) v = to_f<T>(A[(int64_t)(m0 + r) * d.a_rs + (int64_t)(k0 + k) * d.a_ks]);
      As[k][r] = v;
      if (d.b_ks == 1) { k = idx & 15; r = idx >> 4; } else { r = idx & 63; k = idx >> 6; }
      v = 0.f;
      if (n0 + r < d.N && k0 + k < d.K) v = to_f<T>(B[(int64_t)(n0 + r) * d.b_rs + (int64_t)(k0 + k) * d.b_ks]);
      Bs[k][r] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; k++) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; i++) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; j++) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; i++) {
    const int m = m0 + ty * 4 + i;
    if (m >= d.M) continue;
#pragma unroll
    for (int j = 0; j < 4; j++) {
      const int n = n0 + tx * 4 + j;
      if (n >= d.N) continue;
      const int64_t o = doff + (int64_t)m * d.ldd + n;
      float v = d.alpha * acc[i][j];
      if (d.bias) v += d.bias[n];
      if (d.act == 1) {
        if (d.aux) ((T*)d.aux)[o] = from_f<T>(v);
        v = gelu_f(v);
      } else if (d.act == 2) {
        v *= gelu_grad_f(to_f<T>(((const T*)d.aux)[o]));
      }
      if (d.residual) v += to_f<T>(((const T*)d.residual)[o]);
      if (d.d_fp32) {
        float* D = (float*)d.D;
        if (d.accumulate) atomicAdd(D + o, v); else D[o] = v;
      } else {
        ((T*)d.D)[o] = from_f<T>(v);
      }
    }
  }
}

int gemm_simt_launch(const mslt_gemm_desc& d, cudaStream_t st, char* err) {
  if (d.act == 3) {
    snprintf(err, 256, "gemm: the softmax epilogue exists only in the tensor-core kernel");
    return MSLT_ERR_ARG;
  }
  dim3 grid((d.N + 63) / 64, (d.M + 63) / 64, d.batch);
  if (grid.y > 65535 || grid.z > 65535) {
    snprintf(err, 256, "gemm: grid too large for the CUDA-core kernel");
    return MSLT_ERR_SIZE;
  }
  if (d.dtype == 1) gemm_simt_kernel<bf16><<<grid, 256, 0, st>>>(d);
  else gemm_simt_kernel<float><<<grid, 256, 0, st>>>(d);
  return 0;
}

}  // namespace mslt
