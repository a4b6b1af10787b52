// Host-side launchers of the fused memory-bound kernels (kernels.cu).
// `bf` selects the activation type: true = bf16, false = float.  All pointers are device
// pointers; every launcher only enqueues work on `st`.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mslt {

struct AdamChunk {
  int64_t offset;  // element offset into the parameter arena (multiple of 4)
  int32_t count;   // elements in this chunk (multiple of 4)
  float decay;     // 1 for matrices and tables, 0 for vectors
  int32_t tensor;  // index of the tensor the chunk belongs to (LAMB sums its norms per tensor)
  int32_t pad_;
};
struct AdamHyper {
  float lr, beta1, beta2, eps, weight_decay;
  float omb1, omb2;  // 1 - beta, formed in double on the host
  float bc1, bc2;    // bias corrections 1 / (1 - beta^t), or 1: filled on the device
};

void launch_ln_fwd(bool bf, const void* z, const float* gamma, const float* beta, void* y,
                   float* stats, int rows, int H, float eps, cudaStream_t st);
// segments / type: segment ids and the two-row segment table, or null (no segment term)
void launch_embed_ln(bool bf, const int* tokens, const int* segments, const void* word, const void* pos,
                     const void* type, const float* gamma, const float* beta, void* y, void* zstash,
                     float* stats, int rows, int S, int H, int V, float eps, int* status, cudaStream_t st);
void launch_ln_bwd(bool bf, const void* dy, const void* z, const float* stats, const float* gamma,
                   void* dz, float* dgamma, float* dbeta, float* dbias, int rows, int H, cudaStream_t st);
void launch_softmax_fwd(bool bf, const void* sc, void* p, const int* seq_lens, int rows, int S,
                        int rows_per_seq, float scale, cudaStream_t st);
void launch_softmax_bwd(bool bf, void* dp, const void* p, int rows, int S, float scale,
                        cudaStream_t st);
void launch_slots_prepare(const int* positions, const int* labels, const int* seq_lens, int B,
                          int S, int P, int V, int* rowsrc, int* rowlabel, int* n_valid,
                          float* inv_n, int* status, cudaStream_t st);
void launch_gather_rows(bool bf, const void* x, const int* rowsrc, void* out, int R, int H,
                        cudaStream_t st);
void launch_scatter_rows(bool bf, const void* d, const int* rowsrc, void* dx, int B, int P, int H,
                         cudaStream_t st);
// logits fp32 [R, ldl]; dlogits (activation type) [R, ldd] or null; ldl >= ldd, both multiples of 8
void launch_cross_entropy(bool bf, const float* logits, int64_t ldl, const int* rowlabel,
                          const float* inv_n, void* dlogits, int64_t ldd, float* nll, int R, int V,
                          cudaStream_t st);
void launch_loss_reduce(const float* nll, int R, const float* inv_n, float* loss, cudaStream_t st);
// out[n] += sum over rows; N a multiple of the 16-byte vector width, out has room for N floats
void launch_colsum(bool bf, const void* x, int64_t ld, int rows, int N, float* out,
                   cudaStream_t st);
// The embedding gradients without hot-row atomics and with run-to-run identical bits: counting sort
// of the rows by token id, one block per token id, batch sum per position.  Needs H / (16 bytes of
// activation) <= 1024 column threads and V <= 262144.  Scratch: counts [ceil(T/256) * V], total [V],
// start [V], rank [T], order [T], blocksum [1024], hot [2 + 3 * 2048] (ints), partial [2048 * H] (floats);
// needs T <= 65536 and H / (16-byte vector) <= 256.  Nine launches.
void launch_embed_grad_sorted(bool bf, const void* dz, const int* tokens, float* dword, float* dpos, int B, int S,
                              int H, int V, int* counts, int* total, int* start, int* rank, int* order,
                              int* blocksum, int* hot, float* partial, cudaStream_t st);
// t_dev: step count in device memory (incremented here); bc_dev: two floats that receive the bias
// corrections of this step
void launch_adam(const AdamChunk* chunks, int n_chunks, float* w, const float* g, float* m, float* v,
                 void* wb, const AdamHyper& h, int* t_dev, float* bc_dev, int bias_correction,
                 cudaStream_t st);
// LAMB on the same chunk table: the Adam direction r = m_hat / (sqrt(v_hat) + eps) + decay * w is
// scaled per tensor by ||w|| / ||r|| (1 when either norm is 0).  Two kernels: the first updates m and
// v and sums w^2 and r^2 of every tensor into norms[2 * tensor] / [2 * tensor + 1] (zeroed here);
// the second forms r again from the new moments and applies the step.  n_tensors: entries of norms.
void launch_lamb(const AdamChunk* chunks, int n_chunks, float* w, const float* g, float* m, float* v,
                 void* wb, const AdamHyper& h, int* t_dev, float* bc_dev, int bias_correction,
                 float* norms, int n_tensors, cudaStream_t st);
// d[i] *= gelu'(u[i]); n a multiple of the vector width
// Next-sentence-prediction head.  prepare: rowsrc[b] = b * S (first tokens) and inv_n = 1 / (number of
// labels in {0, 1}, or *total_valid when given).  head: two-way classifier on the pooled rows, loss
// added to *loss, gradients of the classifier added to dwn [2,H] / dbn [2], and dup [B,H] = gradient
// at the pooler's pre-activation (tanh derivative included).
void launch_nsp_prepare(const int* labels, int B, int S, int* rowsrc, float* inv_n, const int* total_valid,
                        cudaStream_t st);
void launch_nsp_head(bool bf, const void* pooled, const float* wn, const float* bn, const int* labels,
                     const float* inv_n, void* dup, float* dwn, float* dbn, float* loss, int B, int H,
                     cudaStream_t st);
void launch_tanh(bool bf, const void* x, void* y, int64_t n, cudaStream_t st);
// dtype[seg[t], :] += dz[t, :] for the two-row segment table
void launch_type_grad(bool bf, const void* dz, const int* segments, float* dtype, int rows, int H,
                      cudaStream_t st);
// data-parallel steps: the loss normaliser becomes 1 / *total_valid (0 when that count is 0)
void launch_override_inv_n(const int* total_valid, float* inv_n, cudaStream_t st);
void launch_dgelu(bool bf, void* d, const void* u, int64_t n, cudaStream_t st);
void launch_f32_to_bf16(const float* src, void* dst, int64_t n, cudaStream_t st);

}  // namespace mslt
