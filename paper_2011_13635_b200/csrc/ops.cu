// Single-kernel entry points of the C ABI, for per-kernel tests and profiling.
#include <stdarg.h>
#include <stdio.h>

#include <mutex>

#include "../../include/mslt.h"
#include "common.cuh"
#include "gemm.h"
#include "kernels.h"

using namespace mslt;

namespace mslt {
void set_last_error(const char* msg);  // defined with the C ABI (mslt.cu)
}

namespace {

int op_fail(int code, const char* fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof(buf), fmt, ap);
  va_end(ap);
  set_last_error(buf);
  return code;
}

// labels >= V are treated as "ignore" after raising the status bit; counts the valid rows
__global__ void count_labels_kernel(const int* __restrict__ labels, int R, int V, int* __restrict__ rowlabel,
                                    int* __restrict__ n_valid, float* __restrict__ inv_n) {
  __shared__ int cnt;
  if (threadIdx.x == 0) cnt = 0;
  __syncthreads();
  int local = 0;
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const int lab = labels[r];
    const bool ok = lab >= 0 && lab < V;
    rowlabel[r] = ok ? lab : -1;
    local += ok ? 1 : 0;
  }
  if (local) atomicAdd(&cnt, local);
  __syncthreads();
  if (threadIdx.x == 0) {
    *n_valid = cnt;
    *inv_n = cnt > 0 ? 1.0f / (float)cnt : 0.f;
  }
}

size_t ce_scratch_bytes(int R) { return ((size_t)R * 8 + 8 + 255) / 256 * 256; }

int check_ce_args(int dtype, const float* logits, int64_t ldl, const int32_t* labels, int R, int V,
                  const void* dlogits, int64_t ldd, const float* loss) {
  if (!logits || !labels || !loss) return op_fail(MSLT_ERR_ARG, "cross_entropy: null pointer");
  if (dtype != 0 && dtype != 1) return op_fail(MSLT_ERR_ARG, "cross_entropy: dtype must be 0 or 1");
  if (R < 1 || V < 1) return op_fail(MSLT_ERR_ARG, "cross_entropy: bad shape");
  if (ldl % 8 || ldl < (V + 7) / 8 * 8)
    return op_fail(MSLT_ERR_ARG, "cross_entropy: ldl must be a multiple of 8 and cover V rounded up to 8");
  if (dlogits && (ldd % 8 || ldd > ldl || ldd < V))
    return op_fail(MSLT_ERR_ARG, "cross_entropy: ldd must be a multiple of 8 with V <= ldd <= ldl");
  if (((uintptr_t)logits | (uintptr_t)dlogits) & 15)
    return op_fail(MSLT_ERR_ARG, "cross_entropy: buffers must be 16-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
    return op_fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  return 0;
}

// scratch: [R] float nll, [R] int row label, then n_valid (int) and 1/n_valid (float)
int run_ce(int dtype, const float* logits, int64_t ldl, const int32_t* labels, int R, int V, void* dlogits,
           int64_t ldd, float* loss, void* scratch, cudaStream_t st) {
  float* nll = (float*)scratch;
  int* rowlabel = (int*)scratch + R;
  int* n_valid = (int*)scratch + 2 * (size_t)R;
  float* inv_n = (float*)scratch + 2 * (size_t)R + 1;
  count_labels_kernel<<<1, 256, 0, st>>>(labels, R, V, rowlabel, n_valid, inv_n);
  launch_cross_entropy(dtype == 1, logits, ldl, rowlabel, inv_n, dlogits, ldd, nll, R, V, st);
  launch_loss_reduce(nll, R, inv_n, loss, st);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return op_fail(MSLT_ERR_CUDA, "cross_entropy: %s", cudaGetErrorString(e));
  return 0;
}

int finish_op(const char* what, cudaStream_t st, int sync) {
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess && sync) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return op_fail(MSLT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
  return 0;
}

int check_rows(const char* what, int dtype, int rows, int width, int width_mult, int width_max) {
  if (dtype != 0 && dtype != 1) return op_fail(MSLT_ERR_ARG, "%s: dtype must be 0 or 1", what);
  if (rows < 1) return op_fail(MSLT_ERR_ARG, "%s: rows must be >= 1", what);
  if (width < 1 || width % width_mult || width > width_max)
    return op_fail(MSLT_ERR_ARG, "%s: row length must be a multiple of %d and <= %d", what, width_mult, width_max);
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
    return op_fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  return 0;
}

// ---- allocation-free variant ------------------------------------------------------------------
// Scratch for mslt_op_cross_entropy_noalloc lives in the library image, so the call needs no
// cudaMalloc.  Every GPU that loads the library holds these bytes until the process exits.
constexpr int kNoAllocMaxRows = 16384;
constexpr size_t kNoAllocBytes = ((size_t)kNoAllocMaxRows * 8 + 8 + 255) / 256 * 256;
static __device__ __align__(256) unsigned char g_ce_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
void* g_ce_scratch_ptr[kMaxDevices];  // device address of g_ce_scratch, per device ordinal
std::mutex g_ce_mu;

// In host code `g_ce_scratch` is only a handle; the address a kernel can use must be asked for,
// once per device, while that device is current.
int noalloc_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return op_fail(MSLT_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return op_fail(MSLT_ERR_CUDA, "device ordinal %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_ce_mu);
  if (!g_ce_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_ce_scratch);
    if (e != cudaSuccess || !p)
      return op_fail(MSLT_ERR_CUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
    g_ce_scratch_ptr[dev] = p;
  }
  *out = g_ce_scratch_ptr[dev];
  return 0;
}

}  // namespace

extern "C" {

int mslt_op_cross_entropy_noalloc(int32_t dtype, const float* d_logits, int64_t ldl,
                                  const int32_t* d_labels, int32_t R, int32_t V, void* d_dlogits,
                                  int64_t ldd, float* d_loss, void* cuda_stream) {
  int rc = check_ce_args(dtype, d_logits, ldl, d_labels, R, V, d_dlogits, ldd, d_loss);
  if (rc) return rc;
  if (R > kNoAllocMaxRows)
    return op_fail(MSLT_ERR_SIZE, "cross_entropy_noalloc: R = %d exceeds the built-in scratch (%d rows); "
                   "use mslt_op_cross_entropy with caller scratch", R, kNoAllocMaxRows);
  void* scratch = nullptr;
  rc = noalloc_scratch(&scratch);
  if (rc) return rc;
  // nothing in the scratch has to start at zero: every word the kernels read is written earlier in
  // the same call (row labels and the count first, then the per-row terms)
  return run_ce(dtype, d_logits, ldl, d_labels, R, V, d_dlogits, ldd, d_loss, scratch,
                (cudaStream_t)cuda_stream);
}


size_t mslt_op_cross_entropy_scratch_bytes(int32_t R) { return R > 0 ? ce_scratch_bytes(R) : 0; }

int mslt_op_cross_entropy(int32_t dtype, const float* d_logits, int64_t ldl, const int32_t* d_labels,
                          int32_t R, int32_t V, void* d_dlogits, int64_t ldd, float* d_loss,
                          void* d_scratch, size_t scratch_bytes, void* cuda_stream) {
  int rc = check_ce_args(dtype, d_logits, ldl, d_labels, R, V, d_dlogits, ldd, d_loss);
  if (rc) return rc;
  if (!d_scratch || scratch_bytes < ce_scratch_bytes(R) || ((uintptr_t)d_scratch & 15))
    return op_fail(MSLT_ERR_SIZE, "cross_entropy: scratch must be 16-byte aligned and hold %zu bytes",
                   ce_scratch_bytes(R));
  return run_ce(dtype, d_logits, ldl, d_labels, R, V, d_dlogits, ldd, d_loss, d_scratch,
                (cudaStream_t)cuda_stream);
}

}  // extern "C"

extern "C" {

int mslt_op_layernorm(int32_t dtype, const void* d_z, const float* d_gamma, const float* d_beta, void* d_y,
                      float* d_stats, int32_t rows, int32_t H, float eps, void* cuda_stream, int32_t sync) {
  if (!d_z || !d_gamma || !d_beta || !d_y) return op_fail(MSLT_ERR_ARG, "layernorm: null pointer");
  int rc = check_rows("layernorm", dtype, rows, H, 8, 1024);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  launch_ln_fwd(dtype == 1, d_z, d_gamma, d_beta, d_y, d_stats, rows, H, eps, st);
  return finish_op("layernorm", st, sync);
}

int mslt_op_layernorm_bwd(int32_t dtype, const void* d_dy, const void* d_z, const float* d_stats,
                          const float* d_gamma, void* d_dz, float* d_dgamma, float* d_dbeta, float* d_dbias,
                          int32_t rows, int32_t H, void* cuda_stream, int32_t sync) {
  if (!d_dy || !d_z || !d_stats || !d_gamma || !d_dz || !d_dgamma || !d_dbeta)
    return op_fail(MSLT_ERR_ARG, "layernorm_bwd: null pointer");
  int rc = check_rows("layernorm_bwd", dtype, rows, H, 8, 1024);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  launch_ln_bwd(dtype == 1, d_dy, d_z, d_stats, d_gamma, d_dz, d_dgamma, d_dbeta, d_dbias, rows, H, st);
  return finish_op("layernorm_bwd", st, sync);
}

int mslt_op_attention(const void* d_qkv, void* d_probs, void* d_ctx, const int32_t* d_seq_lens, int32_t B,
                      int32_t S, int32_t heads, float scale, int32_t* d_status, void* cuda_stream,
                      int32_t sync) {
  if (!d_qkv || !d_ctx || !d_status) return op_fail(MSLT_ERR_ARG, "attention: null pointer");
  if (((uintptr_t)d_qkv | (uintptr_t)d_ctx | (uintptr_t)d_probs) & 15)
    return op_fail(MSLT_ERR_ARG, "attention: buffers must be 16-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return op_fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char err[256] = "";
  int rc = attn_fwd_launch(d_qkv, d_probs, d_ctx, d_seq_lens, B, S, heads, 64, scale, d_status, st, err);
  if (rc) return op_fail(rc, "%s", err);
  if (sync) {
    rc = finish_op("attention", st, 1);
    if (rc) return rc;
    int h = 0;
    if (cudaMemcpy(&h, d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess)
      return op_fail(MSLT_ERR_CUDA, "attention: reading the status word failed");
    if (h & 1) return op_fail(MSLT_ERR_DEVICE, "attention: a bounded wait ran out on the device");
    return 0;
  }
  return finish_op("attention", st, 0);
}

int mslt_op_attention_bwd(const void* d_qkv, const void* d_probs, const void* d_dctx, void* d_dqkv, int32_t B,
                          int32_t S, int32_t heads, float scale, int32_t* d_status, void* cuda_stream,
                          int32_t sync) {
  if (!d_qkv || !d_probs || !d_dctx || !d_dqkv || !d_status)
    return op_fail(MSLT_ERR_ARG, "attention_bwd: null pointer");
  if (((uintptr_t)d_qkv | (uintptr_t)d_probs | (uintptr_t)d_dctx | (uintptr_t)d_dqkv) & 15)
    return op_fail(MSLT_ERR_ARG, "attention_bwd: buffers must be 16-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1)
    return op_fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  char err[256] = "";
  int rc = attn_bwd_launch(d_qkv, d_probs, d_dctx, d_dqkv, B, S, heads, 64, scale, d_status, st, err);
  if (rc) return op_fail(rc, "%s", err);
  if (sync) {
    rc = finish_op("attention_bwd", st, 1);
    if (rc) return rc;
    int h = 0;
    if (cudaMemcpy(&h, d_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess)
      return op_fail(MSLT_ERR_CUDA, "attention_bwd: reading the status word failed");
    if (h & 1) return op_fail(MSLT_ERR_DEVICE, "attention_bwd: a bounded wait ran out on the device");
    return 0;
  }
  return finish_op("attention_bwd", st, 0);
}

int mslt_op_softmax(int32_t dtype, const void* d_scores, void* d_probs, const int32_t* d_seq_lens,
                    int32_t rows, int32_t S, int32_t rows_per_seq, float scale, void* cuda_stream,
                    int32_t sync) {
  if (!d_scores || !d_probs) return op_fail(MSLT_ERR_ARG, "softmax: null pointer");
  int rc = check_rows("softmax", dtype, rows, S, 8, 512);
  if (rc) return rc;
  if (rows_per_seq < 1) return op_fail(MSLT_ERR_ARG, "softmax: rows_per_seq must be >= 1");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  launch_softmax_fwd(dtype == 1, d_scores, d_probs, d_seq_lens, rows, S, rows_per_seq, scale, st);
  return finish_op("softmax", st, sync);
}

int mslt_op_softmax_bwd(int32_t dtype, void* d_dp, const void* d_probs, int32_t rows, int32_t S, float scale,
                        void* cuda_stream, int32_t sync) {
  if (!d_dp || !d_probs) return op_fail(MSLT_ERR_ARG, "softmax_bwd: null pointer");
  int rc = check_rows("softmax_bwd", dtype, rows, S, 8, 512);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  launch_softmax_bwd(dtype == 1, d_dp, d_probs, rows, S, scale, st);
  return finish_op("softmax_bwd", st, sync);
}

int mslt_op_colsum(int32_t dtype, const void* d_x, int64_t ld, int32_t rows, int32_t N, float* d_out,
                   void* cuda_stream, int32_t sync) {
  if (!d_x || !d_out) return op_fail(MSLT_ERR_ARG, "colsum: null pointer");
  int rc = check_rows("colsum", dtype, rows, N, 8, 1 << 30);
  if (rc) return rc;
  if (ld < N || ld % 8) return op_fail(MSLT_ERR_ARG, "colsum: ld must be a multiple of 8 and >= N");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  launch_colsum(dtype == 1, d_x, ld, rows, N, d_out, st);
  return finish_op("colsum", st, sync);
}

}  // extern "C"
