/*
 * mslt.h - C ABI of the per-stage training step of multi-stage layerwise
 * training (MSLT) for BERT on one NVIDIA B200 (sm_100a).
 *
 * The procedure (paper, Section 3.1 last paragraph, Section 3.2 and Fig. 1):
 * the encoder stack grows by a group of layers per stage; in each stage the
 * bottom layers, trained earlier, only run forward to feed the top layers,
 * while the newly added top layers and the output layer run forward and
 * backward and are the only parameters updated.  The word-embedding matrix
 * is shared by the input and the output layer and moves only while every
 * layer is trainable (first stage, joint retraining).
 *
 * General rules
 *  - Every function returns 0 on success or a negative mslt_status; nothing
 *    throws or aborts across this boundary.  mslt_last_error() gives a
 *    message for the last failure on the calling thread.
 *  - The library allocates no device memory.  The caller owns the parameter
 *    block and the workspace (sizes from mslt_query_bytes) and the CUDA
 *    stream; they must outlive the context.  All work is enqueued on that
 *    stream.  Pointers marked "device" must be device addresses on the
 *    context's GPU; pointers marked "host" are ordinary host memory.
 *  - Index tensors are int32, row-major.  Weight matrices are [out, in]
 *    row-major, so the tied decoder is the [vocab, hidden] embedding table.
 *  - There is no CPU fallback: without a CUDA device every compute call fails
 *    with MSLT_ERR_CUDA.
 */
#ifndef MSLT_H_
#define MSLT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mslt_ctx mslt_ctx; /* opaque; host state owned by the library */

typedef enum {
  MSLT_OK = 0,
  MSLT_ERR_ARG = -1,    /* invalid argument (null pointer, bad shape, unknown name)   */
  MSLT_ERR_SIZE = -2,   /* shape exceeds what the context was created for             */
  MSLT_ERR_STATE = -3,  /* call not valid in this state (k > L, arena full, ...)      */
  MSLT_ERR_CUDA = -4,   /* a CUDA call failed, or no usable device                    */
  MSLT_ERR_DEVICE = -5  /* a kernel reported an error: a bounded wait ran out, or an  */
                        /* index (token id, MLM position or label) was out of range   */
} mslt_status;

/* Architecture and capacity.  BERT encoder: post-LayerNorm, erf GELU, head dim = hidden/heads. */
typedef struct {
  int32_t hidden;      /* H; multiple of 64, <= 1024                                  */
  int32_t heads;       /* A; H % A == 0; dtype 1 needs H / A == 64                     */
  int32_t ffn;         /* F; multiple of 64                                            */
  int32_t vocab;       /* V                                                            */
  int32_t max_pos;     /* rows of the position table, >= max_seq                       */
  int32_t init_layers; /* encoder layers present after mslt_create (stage 1 depth)     */
  int32_t max_layers;  /* capacity of the layer arena (final depth N)                  */
  int32_t max_batch;   /* largest B of any later call                                  */
  int32_t max_seq;     /* largest S; multiple of 8, <= 512                             */
  int32_t max_pred;    /* largest P (MLM slots per sequence)                           */
  int32_t dtype;       /* 0: fp32 everywhere; 1: bf16 weights/activations, fp32 master */
                       /*    weights, gradients and Adam state                         */
  float ln_eps;        /* LayerNorm epsilon (BERT: 1e-12)                              */
  int32_t max_trainable; /* most top layers that will ever be trainable at once; 0 = max_layers.  Only */
                       /* trainable layers keep their activations for the backward pass (Section    */
                       /* 3.2: the bottom layers run forward only), so the workspace holds this many  */
                       /* saved-activation slots: BERT-Base 9 + 3 needs 3 of them, not 12             */
  int32_t share_group; /* grouped parameter sharing (Section 3.3, the paper's change to ALBERT): encoder  */
                       /* layers l with the same l / share_group use ONE parameter block, their weight   */
                       /* gradients add up, and stages add and train whole groups.  0 or 1: every layer  */
                       /* has its own parameters.  init_layers, max_layers and every k / top_k below     */
                       /* must be multiples of it; tensors are named by block: "layer.<block>.<name>"    */
  int32_t nsp;         /* 1: the network also has BERT's second objective (Section 4.1, "the same MLM    */
                       /* and NSP objectives"): a segment table "emb.type" [2,H] added to the embeddings  */
                       /* (trained with them), a tanh pooler "head.pooler.*" on the first token and a    */
                       /* two-way classifier "head.nsp.*" (part of the output layer, always trained);    */
                       /* see mslt_step_nsp.  0: MLM only, these tensors do not exist                    */
} mslt_arch;

/*
 * Optimizer of the trainable parameters.  Adam with decoupled weight decay (decay on matrices and
 * tables only), or, with lamb = 1, LAMB, the optimizer of the paper's experiments (Section 4.1,
 * learning rate 0.00088): the same direction r = m_hat / (sqrt(v_hat) + eps) + decay * w, scaled
 * for every tensor by its trust ratio ||w|| / ||r|| (Euclidean norms over the tensor; 1 when
 * either norm is 0), w <- w - lr * ratio * r.
 */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t bias_correction; /* 1: divide m, v by (1 - beta^t)                           */
  int32_t lamb;            /* 0: Adam; 1: LAMB                                         */
} mslt_opt;

/*
 * Bytes of device memory the caller must provide for this architecture: the parameter block
 * (master weights, gradients, optimizer state and bf16 copies of every layer up to max_layers: the
 * stack grows in place when layers are added, Section 3.2) and the workspace (two activation
 * buffers for the forward-only bottom layers, saved activations for max_trainable top layers, the
 * output layer's buffers).
 */
int mslt_query_bytes(const mslt_arch* arch, size_t* param_bytes, size_t* workspace_bytes);

/*
 * Creates a context with init_layers encoder layers, all trainable (in the first
 * stage every parameter is trained, Section 3.2); if max_trainable is smaller than
 * init_layers, the top max_trainable layers are trainable instead.  dev_params / dev_workspace:
 * device, at least the queried sizes, 256-byte aligned; the library zeroes
 * both.  Parameters are left at zero: set them with mslt_set_param.
 * cuda_stream: a cudaStream_t (NULL = the default stream).  *out: host.
 */
int mslt_create(const mslt_arch* arch, void* dev_params, size_t param_bytes, void* dev_workspace,
                size_t workspace_bytes, void* cuda_stream, mslt_ctx** out);

/* Frees host state only; device memory stays with the caller. */
int mslt_destroy(mslt_ctx* ctx);

/*
 * Stacks k new layers on top (Section 3.2: new layers start as copies of the
 * top k layers of the previous stage's model): layer L+i <- layer L-k+i, for
 * master weights and compute copies alike.  Needs 1 <= k <= L and
 * L + k <= max_layers (else MSLT_ERR_STATE).  The number of trainable top
 * layers is kept; the optimizer state (m, v, step count) is zeroed.
 */
int mslt_add_layers(mslt_ctx* ctx, int32_t k);

/*
 * Moves the frozen/trainable boundary (Section 3.2): layers [L-top_k, L) and
 * the output layer (MLM transform, its LayerNorm, decoder bias) are trained;
 * top_k == L also trains the embeddings (word table shared with the decoder,
 * position table, embedding LayerNorm).  0 <= top_k <= L (MSLT_ERR_STATE otherwise) and
 * top_k <= max_trainable (MSLT_ERR_SIZE otherwise).  Zeroes the optimizer state.
 */
int mslt_set_trainable(mslt_ctx* ctx, int32_t top_k);

/*
 * Hyper-parameters used from the next step on.  The paper trains with a warm-up of the learning
 * rate over the first 10 000 steps of a stage and a smaller rate in the final joint retraining
 * (Sections 4.2, 5.2): such schedules are the caller's, who sets the rate before each step.
 */
int mslt_set_optimizer(mslt_ctx* ctx, const mslt_opt* opt);

/*
 * One training step (Section 3.1/3.2, Fig. 1): forward-only pass through the
 * frozen layers keeping nothing but the boundary activation; forward with
 * saved activations and backward through the trainable layers and the MLM
 * head; mean cross-entropy over the valid slots; Adam on the trainable
 * parameters only.  Frozen parameters are never written.
 *   d_tokens        device [B,S]   token ids in [0, vocab)
 *   d_seq_lens      device [B] or NULL (= all S); key j of sequence b is valid iff j < len, len >= 1
 *   d_mlm_positions device [B,P]   position in [0, len) or -1 for an empty slot
 *   d_mlm_labels    device [B,P]   label in [0, vocab) or -1 to ignore the slot
 *   loss_out        host float or NULL.  Non-NULL: the stream is synchronised and the loss
 *                   and the device status word are read back (an out-of-range index or a
 *                   kernel wait that ran out gives MSLT_ERR_DEVICE).  NULL: nothing is
 *                   synchronised; use mslt_read_loss later.  In this form the call only enqueues
 *                   kernels and memsets on the context's stream (the Adam step count lives in
 *                   device memory), so after one ordinary step it may be captured into a CUDA
 *                   graph by the caller and replayed on the same buffers.
 */
int mslt_step(mslt_ctx* ctx, const int32_t* d_tokens, const int32_t* d_seq_lens,
              const int32_t* d_mlm_positions, const int32_t* d_mlm_labels, int32_t B, int32_t S,
              int32_t P, float* loss_out);

/*
 * mslt_step with both BERT objectives (needs arch.nsp = 1): loss = MLM loss + NSP loss, where the
 * NSP loss is the mean two-way cross-entropy, over the sequences whose label is 0 or 1, of the
 * classifier on tanh(pooler(first token's final hidden state)).
 *   d_segment_ids  device [B,S] values in {0, 1}, or NULL (all 0): row of "emb.type" added to every
 *                  token's embedding before the embedding LayerNorm
 *   d_nsp_labels   device [B] in {0, 1}, other values = sequence ignored; NULL = no NSP term at all
 *                  (the NSP parameters then get zero gradients)
 * Everything else as mslt_step, which on an nsp context runs with segment 0 everywhere and no NSP
 * term.  loss_out receives the sum of the two losses.
 */
int mslt_step_nsp(mslt_ctx* ctx, const int32_t* d_tokens, const int32_t* d_seq_lens,
                  const int32_t* d_segment_ids, const int32_t* d_mlm_positions,
                  const int32_t* d_mlm_labels, const int32_t* d_nsp_labels, int32_t B, int32_t S,
                  int32_t P, float* loss_out);

/*
 * The same step in two halves, for data-parallel training (Section 3.1, last paragraph, and Section
 * 4.1: every worker takes a share of the batch, and only the gradients of the trainable top layers
 * and the output layer are exchanged; those of the bottom layers are neither computed nor
 * communicated).  mslt_step_backward runs forward, loss and backward and leaves the gradients of
 * the trainable parameters in the gradient arena; the caller sums them over the workers;
 * mslt_step_apply then runs the optimizer.  Between the two calls only the gradient buckets may be
 * touched (no mslt_step, mslt_set_trainable or mslt_add_layers: MSLT_ERR_STATE).
 *   d_total_valid  device int32 or NULL: number of valid MLM slots over ALL workers' batches.  With
 *                  it the loss and the gradients are divided by that count, so that the SUM over
 *                  workers of the returned losses and of the gradients is exactly the mean loss of
 *                  the concatenated batch and its gradient.  NULL: this batch's own count.
 * Other arguments as for mslt_step.
 */
int mslt_step_backward(mslt_ctx* ctx, const int32_t* d_tokens, const int32_t* d_seq_lens,
                       const int32_t* d_mlm_positions, const int32_t* d_mlm_labels, int32_t B, int32_t S,
                       int32_t P, const int32_t* d_total_valid, float* loss_out);
int mslt_step_apply(mslt_ctx* ctx);

/*
 * Gradient buckets: the trainable gradients as a few contiguous fp32 device ranges, numbered in
 * the order in which mslt_step_backward completes them: 0 the output layer, 1..top_k the trainable
 * layers from the top down, then the embeddings when every layer is trainable.  The frozen layers
 * have no bucket: that is the communication the method saves.
 */
int mslt_num_grad_buckets(const mslt_ctx* ctx);
int mslt_grad_bucket(mslt_ctx* ctx, int32_t index, float** d_ptr, int64_t* count);
/*
 * Overlap of the exchange with the rest of the backward pass: if a hook is set, mslt_step_backward
 * calls fn(user, bucket) on the host as soon as the kernels that complete that bucket have been
 * enqueued; comm_stream (a cudaStream_t) has been made to wait for them, so a reduction enqueued on
 * it by the hook runs while the layers below are still in their backward pass.  mslt_step_apply
 * makes the context's stream wait for everything enqueued on comm_stream.  fn = NULL clears it.
 */
typedef void (*mslt_bucket_fn)(void* user, int32_t bucket);
int mslt_set_bucket_hook(mslt_ctx* ctx, void* comm_stream, mslt_bucket_fn fn, void* user);

/* Synchronises the stream and returns the loss of the last mslt_step (host pointer). */
int mslt_read_loss(mslt_ctx* ctx, float* loss_out);

/*
 * Forward only, nothing saved at any layer, no update: the pass that the bottom layers of a stage
 * take part in (Section 3.2, "only participate in forward computation"), here through the whole
 * stack and optionally through the output layer, e.g. for evaluation between stages.
 *   d_hidden_out  device [B,S,H] in the compute dtype (float or bf16), or NULL
 *   d_mlm_positions device [B,P] or NULL; d_logits_out device [B*P, vocab] fp32 or NULL
 *   (rows of empty slots are computed from a zero feature row).
 * Synchronises the stream before returning.
 */
int mslt_forward(mslt_ctx* ctx, const int32_t* d_tokens, const int32_t* d_seq_lens, int32_t B,
                 int32_t S, void* d_hidden_out, const int32_t* d_mlm_positions, int32_t P,
                 float* d_logits_out);

/* Inspection.  Tensor names: "emb.word", "emb.pos", "emb.ln.gamma", "layer.3.ffn1.weight",
 * "head.transform.bias", "head.decoder.bias", ...  All buffers below are host memory. */
int mslt_num_layers(const mslt_ctx* ctx);
int mslt_num_trainable(const mslt_ctx* ctx);
int mslt_num_tensors(const mslt_ctx* ctx); /* tensors of the layers present now */
int mslt_tensor_info(const mslt_ctx* ctx, int32_t index, const char** name, int32_t* rank,
                     int64_t shape[2], int32_t* trainable);
/* fp32 master values; n must equal the tensor's element count. */
int mslt_get_param(mslt_ctx* ctx, const char* name, float* host_dst, size_t n);
/* Writes the master value and, for dtype 1, its bf16 rounding (nearest even). */
int mslt_set_param(mslt_ctx* ctx, const char* name, const float* host_src, size_t n);
/* Raw bits of the copy the kernels read (bf16 for matrices at dtype 1, else fp32), for bit-exact checks. */
int mslt_get_param_raw(mslt_ctx* ctx, const char* name, void* host_dst, size_t bytes);
/* fp32 gradient of a trainable tensor as left by the last mslt_step. */
int mslt_get_grad(mslt_ctx* ctx, const char* name, float* host_dst, size_t n);
/* Adam moments of a trainable tensor (which = 0: m, 1: v). */
int mslt_get_opt_state(mslt_ctx* ctx, const char* name, int32_t which, float* host_dst, size_t n);
/* Number of kernels the library has launched on this context since creation. */
int64_t mslt_launch_count(const mslt_ctx* ctx);
/* Milliseconds of the phases of the last mslt_step when timing is on (mslt_set_timing(ctx,1)):
 * [0] frozen forward, [1] trainable forward, [2] head forward+backward, [3] encoder backward,
 * [4] Adam.  Turning timing on adds event records and one synchronisation per step. */
int mslt_set_timing(mslt_ctx* ctx, int32_t on);
int mslt_get_timings(mslt_ctx* ctx, float* host_ms, int32_t n);
/* Timing level 2 (mslt_set_timing(ctx, 2)) also brackets every kernel launch of a step with an
 * event pair.  This call returns and clears what has been accumulated since the last call, as
 * 10 x 3 host doubles: per kernel class {launches, work, milliseconds}, where work is
 * floating-point operations (2*M*N*K*batch) for the two contraction classes and algorithmic
 * bytes for the others.  Classes, in order: linear-layer products, batched attention products,
 * LayerNorm forward (incl. embedding), LayerNorm backward, softmax forward, softmax backward,
 * column sums, cross-entropy, Adam, other. */
int mslt_get_kernel_profile(mslt_ctx* ctx, double* host_out, int32_t n);
/* Message for the last error on this thread (ctx may be NULL). */
const char* mslt_last_error(const mslt_ctx* ctx);

/*
 * One dense contraction with the step's fused epilogue, exposed for per-kernel tests and
 * profiling:  D[z][m][n] = epilogue( alpha * sum_k A[z](m,k) * B[z](n,k) ).
 * It is the kernel behind every linear layer and attention product of the step (forward:
 * both operands k-contiguous; input-gradient and weight-gradient products: operands with
 * the m / n index contiguous).  dtype 0 runs the fp32 CUDA-core kernel, dtype 1 the bf16
 * tcgen05 tensor-core kernel with fp32 accumulation in tensor memory.
 * All pointers are device pointers; strides are in elements.
 */
typedef struct {
  int32_t dtype;            /* 0: A, B fp32; 1: A, B bf16                                   */
  int32_t M, N, K, batch;   /* batch >= 1; z in [0, batch)                                  */
  int32_t hdiv;             /* z splits as (z / hdiv, z % hdiv) for the two batch strides   */
  const void* A;            /* element (z,m,k) at A + (z/hdiv)*a_bo + (z%hdiv)*a_bi + m*a_rs + k*a_ks */
  int64_t a_rs, a_ks, a_bo, a_bi; /* one of a_rs, a_ks must be 1                            */
  const void* B;            /* element (z,n,k) likewise                                     */
  int64_t b_rs, b_ks, b_bo, b_bi;
  void* D;                  /* element (z,m,n) at D + (z/hdiv)*d_bo + (z%hdiv)*d_bi + m*ldd + n */
  int64_t ldd, d_bo, d_bi;
  int32_t d_fp32;           /* 1: D is fp32 (else the A/B dtype)                            */
  int32_t accumulate;       /* 1 (needs d_fp32): D += result (atomic adds; order not fixed) */
  float alpha;
  const float* bias;        /* [N] fp32 added after alpha, or NULL                          */
  int32_t act;              /* 0 none; 1 GELU(erf); 2 multiply by GELU'(aux); 3 masked       */
                            /* softmax over each row (dtype 1 only, N <= 128, bf16 output;    */
                            /* bias, aux and residual are not applied)                        */
  void* aux;                /* D's layout and A/B dtype. act 1: receives the pre-activation */
                            /* (may be NULL); act 2: holds the pre-activation               */
  const void* residual;     /* D's layout, A/B dtype, added last; or NULL                   */
  int32_t split_k;          /* 0 = automatic; > 1 needs d_fp32 and accumulate               */
  const int32_t* seq_lens;  /* act 3: device [batch / hdiv]; key n of batch z is valid iff    */
                            /* n < seq_lens[z / hdiv]; NULL = all N                           */
} mslt_gemm_desc;

/* Runs one contraction on `cuda_stream` and synchronises it.  d_status: device int32 word,
 * zeroed by the caller, that receives a non-zero code if a kernel wait ran out (then the
 * call returns MSLT_ERR_DEVICE). */
int mslt_op_gemm(const mslt_gemm_desc* desc, void* cuda_stream, int32_t* d_status);
/* The same contraction, only enqueued: no synchronisation and no read of the status word, which
 * the caller inspects after synchronising the stream itself. */
int mslt_op_gemm_enqueue(const mslt_gemm_desc* desc, void* cuda_stream, int32_t* d_status);

/*
 * Test hook for the failure path.  Every wait inside the tensor-core kernel is bounded; when one
 * runs out the CTA sets bit 0 of the status word, drains, frees its tensor memory and returns, and
 * the host call reports MSLT_ERR_DEVICE.  After mslt_debug_starve_next_gemm(1) the NEXT dtype-1
 * contraction (and only that one) runs with a producer that issues no copies and a wait limit of
 * about 20 ms, so this path can be exercised without faulting or hanging the GPU; its output is
 * garbage.  The context and the device stay usable.
 */
int mslt_debug_starve_next_gemm(int32_t on);
/* The same hook for the fused attention kernels: the NEXT mslt_op_attention / mslt_op_attention_bwd
 * call (or attention launch inside a step) runs with an idle producer and a 20 ms wait limit. */
int mslt_debug_starve_next_attention(int32_t on);

/*
 * Environment switches read once per process, for debugging and A/B measurements only (they
 * change speed, not results beyond rounding): MSLT_BF16_CUDA_CORES=1 sends dtype-1 contractions
 * to the plain CUDA-core kernel; MSLT_UNFUSED_ATTENTION=1 runs attention as batched contractions
 * with a separate softmax instead of the fused kernels.
 */

/*
 * Measurement hook: how the dtype-1 contraction kernel tiles its output from now on, process
 * wide.  0 (the default): the library chooses; 1: one CTA per 128 x BN tile; 2: a pair of CTAs per
 * 256 x 256 tile wherever the shape allows it.  Adding 4 to any of these makes the bf16 epilogues
 * store their rows from registers instead of through shared memory and the copy engine.  Results
 * are identical up to summation order; only the speed differs.  Used by the micro-benchmarks to
 * compare the forms on one shape.
 */
int mslt_debug_set_gemm_variant(int32_t variant);

/*
 * Memory-safety check for tests: every buffer the library carves out of the workspace is followed
 * by a 256-byte guard band that no kernel may write and that is zero from mslt_create on.  Counts
 * the guard bands that are no longer zero (*bad_out, host; 0 = no stray write).  Synchronises. */
int mslt_debug_check_guards(mslt_ctx* ctx, int32_t* bad_out);

/*
 * The loss kernel alone (MLM objective, Section 4.1; mean over the valid slots as in the step):
 * for every row r of fp32 logits [R, ldl] with label in [0, V): nll = logsumexp - logit[label];
 * *d_loss = sum nll / n_valid; d_dlogits (may be NULL) [R, ldd] receives
 * (softmax - onehot) / n_valid in the dtype's activation type (0: float, 1: bf16), zero rows for
 * labels < 0 or >= V, zero in columns V..ldd.  ldl, ldd multiples of 8, V <= ldd <= ldl.
 * d_scratch: device memory of mslt_op_cross_entropy_scratch_bytes(R) bytes, 16-byte aligned,
 * used for per-row terms; contents on entry do not matter.  All pointers are device pointers.
 * Synchronises the stream before returning.
 */
size_t mslt_op_cross_entropy_scratch_bytes(int32_t R);
int mslt_op_cross_entropy(int32_t dtype, const float* d_logits, int64_t ldl, const int32_t* d_labels,
                          int32_t R, int32_t V, void* d_dlogits, int64_t ldd, float* d_loss,
                          void* d_scratch, size_t scratch_bytes, void* cuda_stream);

/*
 * The fused memory-bound kernels of the step one at a time, for per-kernel tests and bandwidth
 * measurements.  dtype 0: rows of float, dtype 1: rows of bf16; statistics, gains, biases and
 * column sums are fp32.  All pointers are device pointers, rows are contiguous (row length a
 * multiple of 8; rows 16-byte aligned).  sync != 0 synchronises the stream before returning.
 *
 * LayerNorm of the encoder (post-LN BERT, Section 4.1): y = gamma * (z - mean) / sqrt(var + eps) +
 * beta over rows of H <= 1024 elements, biased variance; d_stats (may be NULL) receives
 * {mean, 1/sqrt(var + eps)} per row.  The backward call takes those statistics and returns dz and
 * ADDS the column sums dgamma += sum dy * xhat, dbeta += sum dy (the caller zeroes them); with
 * d_dbias != NULL it also ADDS dbias += sum dz, the bias gradient of the linear layer whose output
 * (plus residual) was normalised, which saves a separate pass over dz.
 */
int mslt_op_layernorm(int32_t dtype, const void* d_z, const float* d_gamma, const float* d_beta, void* d_y,
                      float* d_stats, int32_t rows, int32_t H, float eps, void* cuda_stream, int32_t sync);
int mslt_op_layernorm_bwd(int32_t dtype, const void* d_dy, const void* d_z, const float* d_stats,
                          const float* d_gamma, void* d_dz, float* d_dgamma, float* d_dbeta, float* d_dbias,
                          int32_t rows, int32_t H, void* cuda_stream, int32_t sync);
/* Scaled masked softmax of attention over rows of S <= 512 scores: row r belongs to sequence
 * r / rows_per_seq; key j is valid iff j < d_seq_lens[sequence] (NULL: all valid); masked
 * probabilities are exactly 0.  May run in place.  The backward call overwrites dp with
 * p * (dp - sum_j dp * p) * scale. */
int mslt_op_softmax(int32_t dtype, const void* d_scores, void* d_probs, const int32_t* d_seq_lens,
                    int32_t rows, int32_t S, int32_t rows_per_seq, float scale, void* cuda_stream,
                    int32_t sync);
int mslt_op_softmax_bwd(int32_t dtype, void* d_dp, const void* d_probs, int32_t rows, int32_t S, float scale,
                        void* cuda_stream, int32_t sync);
/* Bias gradient: d_out[n] += sum over rows of x[row, n] (leading dimension ld, N a multiple of 8;
 * fp32 atomic adds, order not fixed). */
int mslt_op_colsum(int32_t dtype, const void* d_x, int64_t ld, int32_t rows, int32_t N, float* d_out,
                   void* cuda_stream, int32_t sync);

/* Attention of one encoder layer in a single kernel (the paper defers the encoder to BERT,
 * Section 4.1: scaled dot-product attention with a key-padding mask), bf16 only, head width 64,
 * 1 <= S <= 512 (rows of more than 128 keys run a two-pass form of the kernel):  probs[b,h,i,:] = softmax over the valid keys j < d_seq_lens[b] (NULL: all S) of
 * scale * q_i . k_j, masked probabilities exactly 0;  ctx[b,i,h,:] = sum_j probs[b,h,i,j] v_j with
 * probs rounded to bf16 first.  d_qkv: device, [B*S, 3*heads*64] row-major, columns = queries |
 * keys | values, head h in columns h*64.. of each; d_probs: device, [B, heads, S, S] or NULL (not
 * written); d_ctx: device, [B*S, heads*64].  All buffers 16-byte aligned and caller-owned.
 * d_status: device int32 that receives bit 0 if a bounded wait ran out (returned as
 * MSLT_ERR_DEVICE when sync != 0).  Other shapes are rejected with MSLT_ERR_ARG. */
int mslt_op_attention(const void* d_qkv, void* d_probs, void* d_ctx, const int32_t* d_seq_lens, int32_t B,
                      int32_t S, int32_t heads, float scale, int32_t* d_status, void* cuda_stream,
                      int32_t sync);

/* Backward of mslt_op_attention in a single kernel (reverse-mode gradient of the same definition):
 * with P the probabilities the forward call wrote and dC = d_dctx,
 *   dV = P^T dC,  dP = dC V^T,  dS = P o (dP - rowsum(dP o P)) * scale,  dQ = dS K,  dK = dS^T Q,
 * written to d_dqkv in d_qkv's layout.  bf16, head width 64, S a multiple of 8 in [8, 128].
 * d_qkv, d_probs ([B, heads, S, S]), d_dctx ([B*S, heads*64]) are inputs, d_dqkv ([B*S, 3*heads*64])
 * is the output; all device, 16-byte aligned, caller-owned.  d_status and sync as above. */
int mslt_op_attention_bwd(const void* d_qkv, const void* d_probs, const void* d_dctx, void* d_dqkv, int32_t B,
                          int32_t S, int32_t heads, float scale, int32_t* d_status, void* cuda_stream,
                          int32_t sync);

/*
 * mslt_op_cross_entropy without any device allocation by anybody.  (The paper has no counterpart
 * of this call; it exists for the integration below.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plugin inside a host
 * application that hands out a fixed memory budget up front, a callback running while another
 * component owns the allocator lock, a real-time loop that must not touch the driver's
 * allocator, or a process whose memory pool is already sized to the last byte.  Such callers can
 * pass inputs and outputs they already own but cannot produce a scratch buffer.
 *
 * What it does: the same kernels and the same results as mslt_op_cross_entropy, with the per-row
 * scratch taken from a fixed array inside the library image instead of from the caller.  The
 * array holds 16384 rows (about 128 KB) and every GPU that loads the library keeps it until the
 * process exits.  R > 16384 is refused with MSLT_ERR_SIZE; use the caller-scratch call then.
 *
 * The call itself, and everything under it, calls no cudaMalloc, cudaFree or allocating library
 * routine.  The first call on each device looks up the array's device address (the device must be
 * current, as for any call here) and may make the driver load the library's image onto that
 * device; make that first call outside any stream capture.  Later calls take no device memory at
 * all.
 * All calls on one GPU share the one array, which keeps whatever the last call left in it; each
 * call overwrites what it reads, so nothing needs clearing, but two calls that overlap in time on
 * the same GPU (different streams or threads) race on it and give undefined results: serialise
 * them.  Arguments, layout rules and error codes are those of mslt_op_cross_entropy.
 */
int mslt_op_cross_entropy_noalloc(int32_t dtype, const float* d_logits, int64_t ldl,
                                  const int32_t* d_labels, int32_t R, int32_t V, void* d_dlogits,
                                  int64_t ldd, float* d_loss, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MSLT_H_ */
