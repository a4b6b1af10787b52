// Host orchestration and C ABI of the MSLT stage step (paper, Section 3.1-3.2, Fig. 1):
// forward-only pass through the frozen bottom layers that keeps only the boundary activation,
// forward with saved activations and backward through the trainable top layers and the MLM
// head, Adam on the trainable slice.  Every arithmetic step runs in a CUDA kernel (gemm_*.cu,
// kernels.cu); this file holds the parameter arena, the workspace plan and the launch order.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <utility>
#include <unordered_map>
#include <vector>

#include "../../include/mslt.h"
#include "gemm.h"
#include "kernels.h"

using namespace mslt;

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

}  // namespace

namespace mslt {
void set_last_error(const char* msg) { snprintf(g_err, sizeof(g_err), "%s", msg); }
}  // namespace mslt

namespace {

#define CUDA_TRY(x)                                                                  \
  do {                                                                               \
    cudaError_t e_ = (x);                                                            \
    if (e_ != cudaSuccess)                                                           \
      return fail(MSLT_ERR_CUDA, "%s failed: %s", #x, cudaGetErrorString(e_));        \
  } while (0)

inline int64_t pad_to(int64_t n, int64_t a) { return (n + a - 1) / a * a; }

struct Tensor {
  std::string name;
  int rank;
  int64_t shape[2];
  int64_t count;   // elements
  int64_t padded;  // elements reserved (multiple of 64)
  int64_t offset;  // element offset in every arena
  int layer;       // >= 0 parameter block of encoder layers (= layer index without sharing), -1 embeddings, -2 head
};

// Saved activations of one encoder layer (also the scratch of a frozen layer).
struct LayerBuf {
  char *qkv, *p, *c, *z1, *y, *u, *g, *z2, *xout;
  float *st1, *st2;
};

struct Workspace {
  size_t bytes = 0;
  std::vector<size_t> guards;  // byte offsets of the 256-byte guard bands that follow every buffer
  int* scalars;  // [0] status, [1] n_valid, [2] inv_n (float), [3] loss (float), [4] Adam step count,
                 // [5], [6] Adam bias corrections (float)
  int *rowsrc, *rowlabel;
  float* norms;  // LAMB: sums of w^2 and r^2 per tensor
  AdamChunk* chunks;
  int64_t max_chunks;
  char *xa, *xb;
  LayerBuf scratch;
  std::vector<LayerBuf> layer;
  char* z0;
  float* st0;
  char *hm, *ut, *gt, *tm, *dlogits, *dtm, *dgt, *dhm;
  int *es_counts, *es_total, *es_start, *es_rank, *es_order, *es_blocksum, *es_hot;
  float* es_partial;  // embedding backward: rows sorted by token id
  int* nsp_rowsrc;                          // NSP head: first-token row of every sequence
  char *cls, *up, *pooled, *dup, *dcls;     // [B,H] each
  float *hst, *logits, *nll, *dtm32;
  char *dxa, *dxb, *dz2, *dg, *dy, *dz1, *dc, *dp, *dqkv;
};

}  // namespace

struct mslt_ctx {
  mslt_arch a;
  mslt_opt opt;
  cudaStream_t st;
  bool bf;
  int esz;  // bytes per activation element
  int L, top_k;
  int64_t t_step;
  int64_t n_elems;  // elements per arena
  float *master, *grad, *m, *v;
  char* wb;  // bf16 compute copy (dtype 1) or null
  std::vector<Tensor> tensors;  // all max_layers layers
  std::unordered_map<std::string, int> by_name;
  int64_t emb_off, emb_cnt, layer0_off, layer_cnt, layer_mat_cnt, head_off, head_cnt;
  Workspace ws;
  int n_chunks;
  int64_t launches;
  int Vp;
  bool timing;
  cudaEvent_t ev[6];
  float phase_ms[5];
  bool have_events;
  // per-contraction profiling (timing level 2): one event pair per GEMM launch of a step
  int profile;
  std::vector<cudaEvent_t> pev;
  struct PRec { int cls; double flops; };
  std::vector<PRec> prec;
  double prof[10][3];  // per kernel class: launches, work (flops or bytes), ms
  // data-parallel hook: called on the host each time the kernels that finish a gradient bucket have
  // been enqueued (the communication stream already waits for them)
  cudaStream_t comm;
  mslt_bucket_fn bucket_fn;
  void* bucket_user;
  std::vector<cudaEvent_t> bev;
  cudaEvent_t comm_done;
  bool pending_update;  // mslt_step_backward ran, mslt_step_apply has not yet
};

namespace {

// order of the tensors inside one layer block: matrices first, then vectors
const char* kLayerNames[12] = {"qkv.weight", "out.weight", "ffn1.weight", "ffn2.weight",
                               "qkv.bias",   "out.bias",   "ln1.gamma",   "ln1.beta",
                               "ffn1.bias",  "ffn2.bias",  "ln2.gamma",   "ln2.beta"};

int check_arch(const mslt_arch* a) {
  if (!a) return fail(MSLT_ERR_ARG, "arch is null");
  if (a->hidden <= 0 || a->hidden % 64 || a->hidden > 1024)
    return fail(MSLT_ERR_ARG, "hidden must be a multiple of 64 and <= 1024");
  if (a->heads <= 0 || a->hidden % a->heads) return fail(MSLT_ERR_ARG, "hidden %% heads != 0");
  if ((a->hidden / a->heads) % 8) return fail(MSLT_ERR_ARG, "head dim must be a multiple of 8");
  if (a->dtype == 1 && a->hidden / a->heads != 64)
    return fail(MSLT_ERR_ARG, "dtype 1 (bf16 tensor-core path) needs head dim 64");
  if (a->dtype != 0 && a->dtype != 1) return fail(MSLT_ERR_ARG, "dtype must be 0 or 1");
  if (a->ffn <= 0 || a->ffn % 64) return fail(MSLT_ERR_ARG, "ffn must be a multiple of 64");
  if (a->vocab < 2 || a->vocab > 262144) return fail(MSLT_ERR_ARG, "vocab must lie in [2, 262144]");
  if (a->init_layers < 1 || a->max_layers < a->init_layers)
    return fail(MSLT_ERR_ARG, "need 1 <= init_layers <= max_layers");
  if (a->max_batch < 1 || a->max_pred < 1) return fail(MSLT_ERR_ARG, "bad batch/pred capacity");
  if (a->max_seq < 8 || a->max_seq % 8 || a->max_seq > 512)
    return fail(MSLT_ERR_ARG, "max_seq must be a multiple of 8 in [8, 512]");
  if (a->max_pos < a->max_seq) return fail(MSLT_ERR_ARG, "max_pos < max_seq");
  if ((int64_t)a->max_batch * a->max_seq > 65536)
    return fail(MSLT_ERR_ARG, "max_batch * max_seq must not exceed 65536 tokens");
  if (!(a->ln_eps >= 0.f)) return fail(MSLT_ERR_ARG, "ln_eps must be >= 0");
  if (a->max_trainable < 0 || a->max_trainable > a->max_layers)
    return fail(MSLT_ERR_ARG, "need 0 <= max_trainable <= max_layers");
  if (a->share_group < 0) return fail(MSLT_ERR_ARG, "share_group must be >= 0");
  if (a->nsp != 0 && a->nsp != 1) return fail(MSLT_ERR_ARG, "nsp must be 0 or 1");
  if (a->share_group > 1 && (a->init_layers % a->share_group || a->max_layers % a->share_group ||
                             a->max_trainable % a->share_group))
    return fail(MSLT_ERR_ARG, "init_layers, max_layers and max_trainable must be multiples of share_group");
  return 0;
}

// tensors before the first encoder block and after the last
int n_emb_tensors(const mslt_arch& a) { return a.nsp ? 5 : 4; }
int n_head_tensors(const mslt_arch& a) { return a.nsp ? 9 : 5; }
// layers per shared parameter block (Section 3.3); layer l reads block l / group
int group_of(const mslt_arch& a) { return a.share_group > 1 ? a.share_group : 1; }

void build_tensor_table(const mslt_arch& a, std::vector<Tensor>& out, int64_t& total) {
  const int64_t H = a.hidden, F = a.ffn, V = a.vocab;
  int64_t off = 0;
  auto add = [&](const std::string& n, int rank, int64_t s0, int64_t s1, int layer) {
    Tensor t;
    t.name = n; t.rank = rank; t.shape[0] = s0; t.shape[1] = s1;
    t.count = rank == 2 ? s0 * s1 : s0;
    t.padded = pad_to(t.count, 64);
    t.offset = off; t.layer = layer;
    off += t.padded;
    out.push_back(t);
  };
  add("emb.word", 2, V, H, -1);
  add("emb.pos", 2, a.max_pos, H, -1);
  add("emb.ln.gamma", 1, H, 0, -1);
  add("emb.ln.beta", 1, H, 0, -1);
  if (a.nsp) add("emb.type", 2, 2, H, -1);  // segment table, part of the embeddings
  for (int l = 0; l < a.max_layers / group_of(a); l++) {  // one block per group of layers
    const std::string p = "layer." + std::to_string(l) + ".";
    const int64_t rows[12] = {3 * H, H, F, H, 3 * H, H, H, H, F, H, H, H};
    const int64_t cols[4] = {H, H, H, F};
    for (int i = 0; i < 12; i++) add(p + kLayerNames[i], i < 4 ? 2 : 1, rows[i], i < 4 ? cols[i] : 0, l);
  }
  add("head.transform.weight", 2, H, H, -2);
  add("head.transform.bias", 1, H, 0, -2);
  add("head.ln.gamma", 1, H, 0, -2);
  add("head.ln.beta", 1, H, 0, -2);
  add("head.decoder.bias", 1, V, 0, -2);
  if (a.nsp) {  // next-sentence-prediction head, part of the output layer
    add("head.pooler.weight", 2, H, H, -2);
    add("head.pooler.bias", 1, H, 0, -2);
    add("head.nsp.weight", 2, 2, H, -2);
    add("head.nsp.bias", 1, 2, 0, -2);
  }
  total = off;
}

constexpr int64_t kAdamChunk = 8192;

// saved-activation slots: one per layer that may be trainable at the same time
int trainable_slots(const mslt_arch& a) { return a.max_trainable > 0 ? a.max_trainable : a.max_layers; }

// Lays out the workspace; with base == nullptr only the size is computed.
void plan_workspace(const mslt_arch& a, const std::vector<Tensor>& tensors, char* base,
                    Workspace& w) {
  size_t off = 0;
  // every buffer is followed by a 256-byte guard band that no kernel may touch (it stays zero
  // from creation on; mslt_debug_check_guards looks for stray writes)
  w.guards.clear();
  auto take = [&](size_t bytes) -> char* {
    char* p = base ? base + off : nullptr;
    off += (bytes + 255) / 256 * 256;
    w.guards.push_back(off);
    off += 256;
    return p;
  };
  const int64_t E = a.dtype == 1 ? 2 : 4;
  const int64_t H = a.hidden, F = a.ffn, A = a.heads;
  const int64_t T = (int64_t)a.max_batch * a.max_seq, R = (int64_t)a.max_batch * a.max_pred;
  const int64_t Vp = pad_to(a.vocab, 8);
  const int64_t P2 = (int64_t)a.max_batch * A * a.max_seq * a.max_seq;
  w.scalars = (int*)take(256);
  w.rowsrc = (int*)take(R * 4);
  w.rowlabel = (int*)take(R * 4);
  w.max_chunks = 0;
  for (const Tensor& t : tensors) w.max_chunks += (t.padded + kAdamChunk - 1) / kAdamChunk;
  w.chunks = (AdamChunk*)take(w.max_chunks * sizeof(AdamChunk));
  w.norms = (float*)take(tensors.size() * 2 * sizeof(float));
  w.xa = take(T * H * E);
  w.xb = take(T * H * E);
  auto take_layer = [&](LayerBuf& b) {
    b.qkv = take(T * 3 * H * E); b.p = take(P2 * E); b.c = take(T * H * E);
    b.z1 = take(T * H * E); b.y = take(T * H * E); b.u = take(T * F * E);
    b.g = take(T * F * E); b.z2 = take(T * H * E); b.xout = take(T * H * E);
    b.st1 = (float*)take(T * 2 * 4); b.st2 = (float*)take(T * 2 * 4);
  };
  take_layer(w.scratch);
  // Only the trainable top layers save activations (the bottom layers run forward only and share
  // the scratch slot above): trainable layer l of a step uses slot l - (L - top_k).
  w.layer.resize(trainable_slots(a));
  for (int l = 0; l < trainable_slots(a); l++) take_layer(w.layer[l]);
  w.z0 = take(T * H * E);
  w.es_counts = (int*)take(((T + 255) / 256) * (int64_t)a.vocab * 4);
  w.es_total = (int*)take((int64_t)a.vocab * 4);
  w.es_start = (int*)take((int64_t)a.vocab * 4);
  w.es_rank = (int*)take(T * 4);
  w.es_order = (int*)take(T * 4);
  w.es_blocksum = (int*)take(1024 * 4);
  w.es_hot = (int*)take((2 + 3 * 2048) * 4);
  w.es_partial = (float*)take(2048 * H * 4);
  w.st0 = (float*)take(T * 2 * 4);
  w.hm = take(R * H * E); w.ut = take(R * H * E); w.gt = take(R * H * E); w.tm = take(R * H * E);
  w.hst = (float*)take(R * 2 * 4);
  w.logits = (float*)take(R * Vp * 4);
  w.dlogits = take(R * Vp * E);
  w.nll = (float*)take(R * 4);
  w.dtm = take(R * H * E); w.dgt = take(R * H * E); w.dhm = take(R * H * E);
  w.dtm32 = (float*)take(R * H * 4);
  if (a.nsp) {
    const int64_t Bm = a.max_batch;
    w.nsp_rowsrc = (int*)take(Bm * 4);
    w.cls = take(Bm * H * E); w.up = take(Bm * H * E); w.pooled = take(Bm * H * E);
    w.dup = take(Bm * H * E); w.dcls = take(Bm * H * E);
  }
  w.dxa = take(T * H * E); w.dxb = take(T * H * E); w.dz2 = take(T * H * E);
  w.dg = take(T * F * E); w.dy = take(T * H * E); w.dz1 = take(T * H * E);
  w.dc = take(T * H * E); w.dp = take(P2 * E); w.dqkv = take(T * 3 * H * E);
  w.bytes = off;
}

size_t param_bytes_for(const mslt_arch& a, int64_t n) {
  return (size_t)n * (a.dtype == 1 ? 18 : 16);
}

// ---- small accessors ------------------------------------------------------------------------
const Tensor* find(const mslt_ctx* c, const char* name) {
  auto it = c->by_name.find(name);
  if (it == c->by_name.end()) return nullptr;
  const Tensor* t = &c->tensors[it->second];
  if (t->layer >= c->L / group_of(c->a)) return nullptr;
  return t;
}
bool is_trainable(const mslt_ctx* c, const Tensor& t) {
  if (t.layer == -2) return true;
  if (t.layer == -1) return c->top_k == c->L;
  const int g = group_of(c->a);
  return t.layer >= (c->L - c->top_k) / g && t.layer < c->L / g;
}
int64_t toff(const mslt_ctx* c, int layer, const char* n) {
  if (layer >= 0) {
    for (int i = 0; i < 12; i++)
      if (strcmp(n, kLayerNames[i]) == 0) return c->tensors[n_emb_tensors(c->a) + 12 * (layer / group_of(c->a)) + i].offset;
  }
  return c->tensors[c->by_name.at(n)].offset;
}
// the copy the kernels read: bf16 for matrices at dtype 1, fp32 master otherwise
const void* Wc(const mslt_ctx* c, int64_t off) {
  return c->bf ? (const void*)(c->wb + off * 2) : (const void*)(c->master + off);
}
const float* Wv(const mslt_ctx* c, int64_t off) { return c->master + off; }
float* G(const mslt_ctx* c, int64_t off) { return c->grad + off; }

int rebuild_chunks(mslt_ctx* c) {
  std::vector<AdamChunk> h;
  for (size_t ti = 0; ti < c->tensors.size(); ti++) {
    const Tensor& t = c->tensors[ti];
    if (t.layer >= c->L / group_of(c->a) || !is_trainable(c, t)) continue;
    for (int64_t o = 0; o < t.padded; o += kAdamChunk) {
      AdamChunk ch;
      ch.offset = t.offset + o;
      ch.count = (int32_t)std::min<int64_t>(kAdamChunk, t.padded - o);
      ch.decay = t.rank == 2 ? 1.f : 0.f;
      ch.tensor = (int32_t)ti;
      ch.pad_ = 0;
      h.push_back(ch);
    }
  }
  c->n_chunks = (int)h.size();
  CUDA_TRY(cudaStreamSynchronize(c->st));
  if (!h.empty())
  {
    // In-stream copy, then wait: a plain cudaMemcpy from pageable memory may return while its DMA is
    // still in flight, and a non-blocking stream does not wait for it.
    CUDA_TRY(cudaMemcpyAsync(c->ws.chunks, h.data(), h.size() * sizeof(AdamChunk), cudaMemcpyHostToDevice, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
  }
  return 0;
}

int reset_optimizer(mslt_ctx* c) {
  c->t_step = 0;
  CUDA_TRY(cudaMemsetAsync(c->ws.scalars + 4, 0, 12, c->st));
  CUDA_TRY(cudaMemsetAsync(c->m, 0, c->n_elems * 4, c->st));
  CUDA_TRY(cudaMemsetAsync(c->v, 0, c->n_elems * 4, c->st));
  return rebuild_chunks(c);
}

// ---- GEMM helpers ------------------------------------------------------------------------------
struct Lin {  // a plain 2-D contraction
  mslt_gemm_desc d;
  Lin(const mslt_ctx* c, int M, int N, int K) {
    memset(&d, 0, sizeof(d));
    d.dtype = c->bf ? 1 : 0;
    d.M = M; d.N = N; d.K = K; d.batch = 1; d.hdiv = 1; d.alpha = 1.f;
  }
};

// true when bf16 products are routed to the CUDA-core kernel for debugging (see gemm.cu)
bool getenv_cuda_cores() {
  static const bool v = getenv("MSLT_BF16_CUDA_CORES") && atoi(getenv("MSLT_BF16_CUDA_CORES")) == 1;
  return v;
}

// true when attention runs as two batched products with a separate softmax (for A/B measurements)
bool getenv_unfused_attention() {
  static const bool v = getenv("MSLT_UNFUSED_ATTENTION") && atoi(getenv("MSLT_UNFUSED_ATTENTION")) == 1;
  return v;
}

// scores, masked softmax and context of one layer in one kernel (bf16, head width 64, S <= 128)
int run_attention(mslt_ctx* c, const void* qkv, void* probs, void* ctx, const int* seq_lens, int B, int S,
                  int A, int d, float scale) {
  char err[256] = "";
  const bool prof = c->profile && c->prec.size() * 2 + 2 <= c->pev.size();
  if (prof) cudaEventRecord(c->pev[2 * c->prec.size()], c->st);
  int rc = attn_fwd_launch(qkv, probs, ctx, seq_lens, B, S, A, d, scale, c->ws.scalars, c->st, err);
  if (prof) {
    cudaEventRecord(c->pev[2 * c->prec.size() + 1], c->st);
    c->prec.push_back({1, 4.0 * B * A * (double)S * S * d});
  }
  if (rc) return fail(rc, "%s", err);
  c->launches++;
  return 0;
}

int run_attention_bwd(mslt_ctx* c, const void* qkv, const void* probs, const void* dctx, void* dqkv, int B,
                      int S, int A, int d, float scale) {
  char err[256] = "";
  const bool prof = c->profile && c->prec.size() * 2 + 2 <= c->pev.size();
  if (prof) cudaEventRecord(c->pev[2 * c->prec.size()], c->st);
  int rc = attn_bwd_launch(qkv, probs, dctx, dqkv, B, S, A, d, scale, c->ws.scalars, c->st, err);
  if (prof) {
    cudaEventRecord(c->pev[2 * c->prec.size() + 1], c->st);
    c->prec.push_back({1, 8.0 * B * A * (double)S * S * d});
  }
  if (rc) return fail(rc, "%s", err);
  c->launches++;
  return 0;
}

int run_gemm(mslt_ctx* c, const mslt_gemm_desc& d) {
  if (d.M <= 0 || d.N <= 0 || d.K <= 0 || d.batch <= 0) return 0;
  char err[256] = "";
  const int64_t before = gemm_launches();
  const bool prof = c->profile && c->prec.size() * 2 + 2 <= c->pev.size();
  if (prof) cudaEventRecord(c->pev[2 * c->prec.size()], c->st);
  int rc = gemm_launch(d, c->ws.scalars, c->st, err);
  if (prof) {
    cudaEventRecord(c->pev[2 * c->prec.size() + 1], c->st);
    c->prec.push_back({d.batch > 1 ? 1 : 0, 2.0 * d.M * d.N * (double)d.K * d.batch});
  }
  c->launches += gemm_launches() - before;
  if (rc) return fail(rc, "%s", err);
  return 0;
}

// Y[T,N] = X[T,K] * W[N,K]^T (+ bias) with optional GELU / residual
int linear_fwd(mslt_ctx* c, const void* x, int T, int K, int64_t w_off, int64_t b_off, int N,
               void* y, int act, void* aux, const void* residual, bool out_fp32 = false,
               int64_t ldd = 0) {
  Lin g(c, T, N, K);
  g.d.A = x; g.d.a_rs = K; g.d.a_ks = 1;
  g.d.B = Wc(c, w_off); g.d.b_rs = K; g.d.b_ks = 1;
  g.d.D = y; g.d.ldd = ldd ? ldd : N;
  g.d.bias = Wv(c, b_off);
  g.d.act = act; g.d.aux = aux; g.d.residual = residual;
  g.d.d_fp32 = out_fp32 ? 1 : 0;
  return run_gemm(c, g.d);
}

// dX[T,K] = dY[T,N] * W[N,K]  (optionally * gelu'(aux), + residual)
int linear_dgrad(mslt_ctx* c, const void* dy, int T, int N, int64_t lda, int64_t w_off, int K,
                 void* dx, int act, void* aux, const void* residual) {
  Lin g(c, T, K, N);
  g.d.A = dy; g.d.a_rs = lda; g.d.a_ks = 1;
  g.d.B = Wc(c, w_off); g.d.b_rs = 1; g.d.b_ks = K;
  g.d.D = dx; g.d.ldd = K;
  g.d.act = act; g.d.aux = aux; g.d.residual = residual;
  return run_gemm(c, g.d);
}

// dW[N,K] += dY[T,N]^T * X[T,K]   (fp32, into the zeroed gradient arena)
int linear_wgrad(mslt_ctx* c, const void* dy, int T, int N, int64_t lddy, const void* x, int K,
                 int64_t w_off) {
  Lin g(c, N, K, T);
  g.d.A = dy; g.d.a_rs = 1; g.d.a_ks = lddy;
  g.d.B = x; g.d.b_rs = 1; g.d.b_ks = K;
  g.d.D = G(c, w_off); g.d.ldd = K;
  g.d.d_fp32 = 1; g.d.accumulate = 1;
  return run_gemm(c, g.d);
}

#define TRY(x)        \
  do {                \
    int rc_ = (x);    \
    if (rc_) return rc_; \
  } while (0)
// kernel classes of the per-launch profile (timing level 2)
enum { PC_LINEAR = 0, PC_ATTN_GEMM, PC_LN_FWD, PC_LN_BWD, PC_SOFTMAX_FWD, PC_SOFTMAX_BWD, PC_COLSUM,
       PC_CROSS_ENTROPY, PC_ADAM, PC_OTHER, PC_COUNT };

void prof_begin(mslt_ctx* c) {
  if (c->profile && c->prec.size() * 2 + 2 <= c->pev.size())
    cudaEventRecord(c->pev[2 * c->prec.size()], c->st);
}
void prof_end(mslt_ctx* c, int cls, double work) {
  if (c->profile && c->prec.size() * 2 + 2 <= c->pev.size()) {
    cudaEventRecord(c->pev[2 * c->prec.size() + 1], c->st);
    c->prec.push_back({cls, work});
  }
}

// launches one kernel; `work` is its algorithmic byte count (for the profile)
#define KL(cls, work, x)          \
  do {                            \
    prof_begin(c);                \
    x;                            \
    c->launches++;                \
    prof_end(c, cls, (double)(work)); \
  } while (0)

// ---- one encoder layer, forward ------------------------------------------------------------------
int layer_forward(mslt_ctx* c, int l, const void* x, LayerBuf& b, void* out, bool save, int B, int S,
                  const int* seq_lens) {
  const int H = c->a.hidden, F = c->a.ffn, A = c->a.heads, d = H / A, T = B * S;
  const int E = c->esz;
  const float scale = 1.0f / sqrtf((float)d);
  TRY(linear_fwd(c, x, T, H, toff(c, l, "qkv.weight"), toff(c, l, "qkv.bias"), 3 * H, b.qkv, 0,
                 nullptr, nullptr));
  if (c->bf && S <= 512 && d == 64 && !getenv_cuda_cores() && !getenv_unfused_attention()) {
    // the probabilities go to memory only where the backward pass will read them
    TRY(run_attention(c, b.qkv, save ? b.p : nullptr, b.c, seq_lens, B, S, A, d, scale));
  } else {
    {  // scores[b,h,i,j] = q_i . k_j / sqrt(d)
      Lin g(c, S, S, d);
      g.d.batch = B * A; g.d.hdiv = A; g.d.alpha = scale;
      g.d.A = b.qkv; g.d.a_rs = 3 * H; g.d.a_ks = 1; g.d.a_bo = (int64_t)S * 3 * H; g.d.a_bi = d;
      g.d.B = b.qkv + (int64_t)H * E; g.d.b_rs = 3 * H; g.d.b_ks = 1; g.d.b_bo = (int64_t)S * 3 * H; g.d.b_bi = d;
      g.d.D = b.p; g.d.ldd = S; g.d.d_bo = (int64_t)A * S * S; g.d.d_bi = (int64_t)S * S;
      // rows of at most 128 keys fit one tile: the tensor-core kernel applies the masked softmax
      // in its epilogue and writes probabilities straight away
      const bool fused = c->bf && S <= 128 && !getenv_cuda_cores();
      if (fused) { g.d.act = 3; g.d.seq_lens = seq_lens; }
      TRY(run_gemm(c, g.d));
      if (!fused)
        KL(PC_SOFTMAX_FWD, 2.0 * B * A * S * S * c->esz,
           launch_softmax_fwd(c->bf, b.p, b.p, seq_lens, B * A * S, S, A * S, 1.0f, c->st));
    }
    {  // context[b,i,h,:] = sum_j p[b,h,i,j] v_j
      Lin g(c, S, d, S);
      g.d.batch = B * A; g.d.hdiv = A;
      g.d.A = b.p; g.d.a_rs = S; g.d.a_ks = 1; g.d.a_bo = (int64_t)A * S * S; g.d.a_bi = (int64_t)S * S;
      g.d.B = b.qkv + (int64_t)2 * H * E; g.d.b_rs = 1; g.d.b_ks = 3 * H; g.d.b_bo = (int64_t)S * 3 * H; g.d.b_bi = d;
      g.d.D = b.c; g.d.ldd = H; g.d.d_bo = (int64_t)S * H; g.d.d_bi = d;
      TRY(run_gemm(c, g.d));
    }
  }
  TRY(linear_fwd(c, b.c, T, H, toff(c, l, "out.weight"), toff(c, l, "out.bias"), H, b.z1, 0, nullptr, x));
  KL(PC_LN_FWD, 2.0 * T * H * c->esz, launch_ln_fwd(c->bf, b.z1, Wv(c, toff(c, l, "ln1.gamma")), Wv(c, toff(c, l, "ln1.beta")), b.y,
                   save ? b.st1 : nullptr, T, H, c->a.ln_eps, c->st));
  TRY(linear_fwd(c, b.y, T, H, toff(c, l, "ffn1.weight"), toff(c, l, "ffn1.bias"), F, b.g, 1,
                 save ? b.u : nullptr, nullptr));
  TRY(linear_fwd(c, b.g, T, F, toff(c, l, "ffn2.weight"), toff(c, l, "ffn2.bias"), H, b.z2, 0, nullptr, b.y));
  KL(PC_LN_FWD, 2.0 * T * H * c->esz, launch_ln_fwd(c->bf, b.z2, Wv(c, toff(c, l, "ln2.gamma")), Wv(c, toff(c, l, "ln2.beta")), out,
                   save ? b.st2 : nullptr, T, H, c->a.ln_eps, c->st));
  return 0;
}

// ---- one encoder layer, backward -------------------------------------------------------------------
// dx: gradient w.r.t. the layer output; dx_out (if need_dx): gradient w.r.t. its input x_in.
int layer_backward(mslt_ctx* c, int l, const void* x_in, LayerBuf& b, const void* dx, void* dx_out,
                   bool need_dx, int B, int S) {
  const int H = c->a.hidden, F = c->a.ffn, A = c->a.heads, d = H / A, T = B * S;
  const int E = c->esz;
  Workspace& w = c->ws;
  const float scale = 1.0f / sqrtf((float)d);
  KL(PC_LN_BWD, 3.0 * T * H * c->esz, launch_ln_bwd(c->bf, dx, b.z2, b.st2, Wv(c, toff(c, l, "ln2.gamma")), w.dz2,
                   G(c, toff(c, l, "ln2.gamma")), G(c, toff(c, l, "ln2.beta")), G(c, toff(c, l, "ffn2.bias")), T, H, c->st));
  TRY(linear_wgrad(c, w.dz2, T, H, H, b.g, F, toff(c, l, "ffn2.weight")));
  TRY(linear_dgrad(c, w.dz2, T, H, H, toff(c, l, "ffn2.weight"), F, w.dg, 2, b.u, nullptr));
  TRY(linear_wgrad(c, w.dg, T, F, F, b.y, H, toff(c, l, "ffn1.weight")));
  KL(PC_COLSUM, 1.0 * T * F * c->esz, launch_colsum(c->bf, w.dg, F, T, F, G(c, toff(c, l, "ffn1.bias")), c->st));
  TRY(linear_dgrad(c, w.dg, T, F, F, toff(c, l, "ffn1.weight"), H, w.dy, 0, nullptr, w.dz2));
  KL(PC_LN_BWD, 3.0 * T * H * c->esz, launch_ln_bwd(c->bf, w.dy, b.z1, b.st1, Wv(c, toff(c, l, "ln1.gamma")), w.dz1,
                   G(c, toff(c, l, "ln1.gamma")), G(c, toff(c, l, "ln1.beta")), G(c, toff(c, l, "out.bias")), T, H, c->st));
  TRY(linear_wgrad(c, w.dz1, T, H, H, b.c, H, toff(c, l, "out.weight")));
  TRY(linear_dgrad(c, w.dz1, T, H, H, toff(c, l, "out.weight"), H, w.dc, 0, nullptr, nullptr));
  const int64_t qs = (int64_t)S * 3 * H, ps = (int64_t)A * S * S, cs = (int64_t)S * H;
  if (c->bf && S <= 128 && S % 8 == 0 && d == 64 && !getenv_cuda_cores() && !getenv_unfused_attention()) {
    // dV, dP, softmax backward, dQ and dK of the layer in one kernel
    TRY(run_attention_bwd(c, b.qkv, b.p, w.dc, w.dqkv, B, S, A, d, scale));
  } else {
    {  // dV[j,:] = sum_i p[i,j] dC[i,:]
      Lin g(c, S, d, S);
      g.d.batch = B * A; g.d.hdiv = A;
      g.d.A = b.p; g.d.a_rs = 1; g.d.a_ks = S; g.d.a_bo = ps; g.d.a_bi = (int64_t)S * S;
      g.d.B = w.dc; g.d.b_rs = 1; g.d.b_ks = H; g.d.b_bo = cs; g.d.b_bi = d;
      g.d.D = w.dqkv + (int64_t)2 * H * E; g.d.ldd = 3 * H; g.d.d_bo = qs; g.d.d_bi = d;
      TRY(run_gemm(c, g.d));
    }
    {  // dP[i,j] = dC[i,:] . v_j
      Lin g(c, S, S, d);
      g.d.batch = B * A; g.d.hdiv = A;
      g.d.A = w.dc; g.d.a_rs = H; g.d.a_ks = 1; g.d.a_bo = cs; g.d.a_bi = d;
      g.d.B = b.qkv + (int64_t)2 * H * E; g.d.b_rs = 3 * H; g.d.b_ks = 1; g.d.b_bo = qs; g.d.b_bi = d;
      g.d.D = w.dp; g.d.ldd = S; g.d.d_bo = ps; g.d.d_bi = (int64_t)S * S;
      TRY(run_gemm(c, g.d));
    }
    KL(PC_SOFTMAX_BWD, 3.0 * B * A * S * S * c->esz, launch_softmax_bwd(c->bf, w.dp, b.p, B * A * S, S, scale, c->st));
    {  // dQ[i,:] = sum_j dS[i,j] k_j
      Lin g(c, S, d, S);
      g.d.batch = B * A; g.d.hdiv = A;
      g.d.A = w.dp; g.d.a_rs = S; g.d.a_ks = 1; g.d.a_bo = ps; g.d.a_bi = (int64_t)S * S;
      g.d.B = b.qkv + (int64_t)H * E; g.d.b_rs = 1; g.d.b_ks = 3 * H; g.d.b_bo = qs; g.d.b_bi = d;
      g.d.D = w.dqkv; g.d.ldd = 3 * H; g.d.d_bo = qs; g.d.d_bi = d;
      TRY(run_gemm(c, g.d));
    }
    {  // dK[j,:] = sum_i dS[i,j] q_i
      Lin g(c, S, d, S);
      g.d.batch = B * A; g.d.hdiv = A;
      g.d.A = w.dp; g.d.a_rs = 1; g.d.a_ks = S; g.d.a_bo = ps; g.d.a_bi = (int64_t)S * S;
      g.d.B = b.qkv; g.d.b_rs = 1; g.d.b_ks = 3 * H; g.d.b_bo = qs; g.d.b_bi = d;
      g.d.D = w.dqkv + (int64_t)H * E; g.d.ldd = 3 * H; g.d.d_bo = qs; g.d.d_bi = d;
      TRY(run_gemm(c, g.d));
    }
  }
  TRY(linear_wgrad(c, w.dqkv, T, 3 * H, 3 * H, x_in, H, toff(c, l, "qkv.weight")));
  KL(PC_COLSUM, 3.0 * T * H * c->esz, launch_colsum(c->bf, w.dqkv, 3 * H, T, 3 * H, G(c, toff(c, l, "qkv.bias")), c->st));
  if (need_dx)  // the frozen boundary stops here: nothing below needs a gradient
    TRY(linear_dgrad(c, w.dqkv, T, 3 * H, 3 * H, toff(c, l, "qkv.weight"), H, dx_out, 0, nullptr, w.dz1));
  return 0;
}

int head_forward(mslt_ctx* c, const void* x, int R, bool save) {
  const int H = c->a.hidden, V = c->a.vocab;
  Workspace& w = c->ws;
  KL(PC_OTHER, 2.0 * R * H * c->esz, launch_gather_rows(c->bf, x, w.rowsrc, w.hm, R, H, c->st));
  TRY(linear_fwd(c, w.hm, R, H, toff(c, -1, "head.transform.weight"), toff(c, -1, "head.transform.bias"),
                 H, w.gt, 1, save ? w.ut : nullptr, nullptr));
  KL(PC_LN_FWD, 2.0 * R * H * c->esz, launch_ln_fwd(c->bf, w.gt, Wv(c, toff(c, -1, "head.ln.gamma")), Wv(c, toff(c, -1, "head.ln.beta")),
                   w.tm, save ? w.hst : nullptr, R, H, c->a.ln_eps, c->st));
  // tied decoder: logits = tm * E^T + bv, fp32, rows padded to Vp columns
  TRY(linear_fwd(c, w.tm, R, H, toff(c, -1, "emb.word"), toff(c, -1, "head.decoder.bias"), V, w.logits,
                 0, nullptr, nullptr, true, c->Vp));
  return 0;
}

int head_backward(mslt_ctx* c, int B, int S, int P, bool full) {
  const int H = c->a.hidden, V = c->a.vocab, R = B * P, Vp = c->Vp;
  Workspace& w = c->ws;
  KL(PC_COLSUM, 1.0 * R * Vp * c->esz, launch_colsum(c->bf, w.dlogits, Vp, R, Vp, G(c, toff(c, -1, "head.decoder.bias")), c->st));
  {  // dTm = dlogits * E
    Lin g(c, R, H, V);
    g.d.A = w.dlogits; g.d.a_rs = Vp; g.d.a_ks = 1;
    g.d.B = Wc(c, toff(c, -1, "emb.word")); g.d.b_rs = 1; g.d.b_ks = H;
    if (c->bf) {
      // few output tiles, a contraction over the whole vocabulary: split it across the machine
      // with fp32 partial sums, then round once to bf16
      CUDA_TRY(cudaMemsetAsync(w.dtm32, 0, (size_t)R * H * 4, c->st));
      g.d.D = w.dtm32; g.d.ldd = H; g.d.d_fp32 = 1; g.d.accumulate = 1;
      TRY(run_gemm(c, g.d));
      KL(PC_OTHER, 6.0 * R * H, launch_f32_to_bf16(w.dtm32, w.dtm, (int64_t)R * H, c->st));
    } else {
      g.d.D = w.dtm; g.d.ldd = H;
      TRY(run_gemm(c, g.d));
    }
  }
  if (full) {  // the shared word embedding moves only while every layer is trainable
    Lin g(c, V, H, R);
    g.d.A = w.dlogits; g.d.a_rs = 1; g.d.a_ks = Vp;
    g.d.B = w.tm; g.d.b_rs = 1; g.d.b_ks = H;
    g.d.D = G(c, toff(c, -1, "emb.word")); g.d.ldd = H; g.d.d_fp32 = 1; g.d.accumulate = 1;
    TRY(run_gemm(c, g.d));
  }
  KL(PC_LN_BWD, 3.0 * R * H * c->esz, launch_ln_bwd(c->bf, w.dtm, w.gt, w.hst, Wv(c, toff(c, -1, "head.ln.gamma")), w.dgt,
                   G(c, toff(c, -1, "head.ln.gamma")), G(c, toff(c, -1, "head.ln.beta")), nullptr, R, H, c->st));
  KL(PC_OTHER, 3.0 * R * H * c->esz, launch_dgelu(c->bf, w.dgt, w.ut, (int64_t)R * H, c->st));
  TRY(linear_wgrad(c, w.dgt, R, H, H, w.hm, H, toff(c, -1, "head.transform.weight")));
  KL(PC_COLSUM, 1.0 * R * H * c->esz, launch_colsum(c->bf, w.dgt, H, R, H, G(c, toff(c, -1, "head.transform.bias")), c->st));
  TRY(linear_dgrad(c, w.dgt, R, H, H, toff(c, -1, "head.transform.weight"), H, w.dhm, 0, nullptr, nullptr));
  CUDA_TRY(cudaMemsetAsync(w.dxa, 0, (size_t)B * S * H * c->esz, c->st));
  KL(PC_OTHER, 2.0 * B * P * H * c->esz, launch_scatter_rows(c->bf, w.dhm, w.rowsrc, w.dxa, B, P, H, c->st));
  return 0;
}

int zero_trainable_grads(mslt_ctx* c) {
  const int first = c->L - c->top_k;
  if (c->top_k == c->L) CUDA_TRY(cudaMemsetAsync(c->grad + c->emb_off, 0, c->emb_cnt * 4, c->st));
  if (c->top_k > 0)
    CUDA_TRY(cudaMemsetAsync(c->grad + c->layer0_off + (int64_t)(first / group_of(c->a)) * c->layer_cnt, 0,
                             (size_t)(c->top_k / group_of(c->a)) * c->layer_cnt * 4, c->st));
  CUDA_TRY(cudaMemsetAsync(c->grad + c->head_off, 0, c->head_cnt * 4, c->st));
  return 0;
}

// Gradient buckets in the order in which a step completes them: the output layer, the trainable
// layers from the top down, then (only when everything trains) the embeddings.  Each is one contiguous
// range of the fp32 gradient arena.
int num_buckets(const mslt_ctx* c) { return 1 + c->top_k / group_of(c->a) + (c->top_k == c->L ? 1 : 0); }
void bucket_range(const mslt_ctx* c, int i, int64_t* off, int64_t* cnt) {
  if (i == 0) { *off = c->head_off; *cnt = c->head_cnt; }
  else if (i <= c->top_k / group_of(c->a)) {  // parameter blocks from the top down
    *off = c->layer0_off + (int64_t)(c->L / group_of(c->a) - i) * c->layer_cnt;
    *cnt = c->layer_cnt;
  }
  else { *off = c->emb_off; *cnt = c->emb_cnt; }
}
int bucket_done(mslt_ctx* c, int i) {
  if (!c->bucket_fn) return 0;
  while ((int)c->bev.size() <= i) {
    cudaEvent_t e;
    CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    c->bev.push_back(e);
  }
  CUDA_TRY(cudaEventRecord(c->bev[i], c->st));
  CUDA_TRY(cudaStreamWaitEvent(c->comm, c->bev[i], 0));
  c->bucket_fn(c->bucket_user, i);
  return 0;
}

int check_batch(mslt_ctx* c, int B, int S, int P) {
  if (B < 1 || S < 1 || P < 0) return fail(MSLT_ERR_ARG, "bad batch shape");
  if (B > c->a.max_batch || S > c->a.max_seq || P > c->a.max_pred)
    return fail(MSLT_ERR_SIZE, "batch shape (%d,%d,%d) exceeds capacity (%d,%d,%d)", B, S, P,
                c->a.max_batch, c->a.max_seq, c->a.max_pred);
  if (S % 8) return fail(MSLT_ERR_ARG, "S must be a multiple of 8");
  return 0;
}

int finish(mslt_ctx* c, float* loss_out) {
  CUDA_TRY(cudaGetLastError());
  if (!loss_out) return 0;
  int h[4];
  CUDA_TRY(cudaStreamSynchronize(c->st));
  CUDA_TRY(cudaMemcpyAsync(h, c->ws.scalars, 16, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  memcpy(loss_out, &h[3], 4);
  if (h[0] != 0)
    return fail(MSLT_ERR_DEVICE, "device status 0x%x (1: kernel wait ran out, 2: token id, 4: MLM "
                "position, 8: MLM label, 16: sequence length out of range)", h[0]);
  return 0;
}

void mark(mslt_ctx* c, int i) {
  if (c->timing && c->have_events) cudaEventRecord(c->ev[i], c->st);
}

}  // namespace

// ======================================================================================
// C ABI
// ======================================================================================
extern "C" {

const char* mslt_last_error(const mslt_ctx*) { return g_err; }

int mslt_query_bytes(const mslt_arch* arch, size_t* param_bytes, size_t* workspace_bytes) {
  TRY(check_arch(arch));
  std::vector<Tensor> t;
  int64_t n = 0;
  build_tensor_table(*arch, t, n);
  Workspace w;
  plan_workspace(*arch, t, nullptr, w);
  if (param_bytes) *param_bytes = param_bytes_for(*arch, n);
  if (workspace_bytes) *workspace_bytes = w.bytes;
  return 0;
}

int mslt_create(const mslt_arch* arch, void* dev_params, size_t param_bytes, void* dev_workspace,
                size_t workspace_bytes, void* cuda_stream, mslt_ctx** out) {
  TRY(check_arch(arch));
  if (!dev_params || !dev_workspace || !out) return fail(MSLT_ERR_ARG, "null pointer");
  if (((uintptr_t)dev_params | (uintptr_t)dev_workspace) & 255)
    return fail(MSLT_ERR_ARG, "device buffers must be 256-byte aligned");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
    return fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  mslt_ctx* c = new mslt_ctx();
  c->a = *arch;
  c->bf = arch->dtype == 1;
  c->esz = c->bf ? 2 : 4;
  c->st = (cudaStream_t)cuda_stream;
  c->opt = {1e-3f, 0.9f, 0.999f, 1e-6f, 0.01f, 1, 0};
  c->L = arch->init_layers;
  c->top_k = std::min(c->L, trainable_slots(*arch));
  c->t_step = 0;
  c->launches = 0;
  c->timing = false;
  c->have_events = false;
  c->profile = 0;
  c->comm = nullptr;
  c->bucket_fn = nullptr;
  c->bucket_user = nullptr;
  c->comm_done = nullptr;
  c->pending_update = false;
  memset(c->prof, 0, sizeof(c->prof));
  c->Vp = (int)pad_to(arch->vocab, 8);
  build_tensor_table(*arch, c->tensors, c->n_elems);
  for (size_t i = 0; i < c->tensors.size(); i++) c->by_name[c->tensors[i].name] = (int)i;
  plan_workspace(*arch, c->tensors, (char*)dev_workspace, c->ws);
  if (param_bytes < param_bytes_for(*arch, c->n_elems) || workspace_bytes < c->ws.bytes) {
    delete c;
    return fail(MSLT_ERR_SIZE, "device buffers smaller than mslt_query_bytes reports");
  }
  char* p = (char*)dev_params;
  c->master = (float*)p; p += c->n_elems * 4;
  c->grad = (float*)p; p += c->n_elems * 4;
  c->m = (float*)p; p += c->n_elems * 4;
  c->v = (float*)p; p += c->n_elems * 4;
  c->wb = c->bf ? p : nullptr;
  c->emb_off = 0;
  c->layer0_off = c->tensors[c->by_name.at("layer.0.qkv.weight")].offset;
  c->emb_cnt = c->layer0_off;
  c->head_off = c->tensors[c->by_name.at("head.transform.weight")].offset;
  c->layer_cnt = (c->head_off - c->layer0_off) / (arch->max_layers / group_of(*arch));
  c->head_cnt = c->n_elems - c->head_off;
  cudaError_t e = cudaMemsetAsync(dev_params, 0, param_bytes_for(*arch, c->n_elems), c->st);
  if (e == cudaSuccess) e = cudaMemsetAsync(dev_workspace, 0, c->ws.bytes, c->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->st);
  if (e != cudaSuccess) {
    delete c;
    return fail(MSLT_ERR_CUDA, "clearing device buffers failed: %s", cudaGetErrorString(e));
  }
  int rc = rebuild_chunks(c);
  if (rc) { delete c; return rc; }
  *out = c;
  return 0;
}

int mslt_destroy(mslt_ctx* c) {
  if (!c) return 0;
  if (c->have_events)
    for (int i = 0; i < 6; i++) cudaEventDestroy(c->ev[i]);
  for (cudaEvent_t e : c->pev) cudaEventDestroy(e);
  for (cudaEvent_t e : c->bev) cudaEventDestroy(e);
  if (c->comm_done) cudaEventDestroy(c->comm_done);
  delete c;
  return 0;
}

int mslt_add_layers(mslt_ctx* c, int32_t k) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  const int g = group_of(c->a);
  if (c->pending_update) return fail(MSLT_ERR_STATE, "add_layers: a step is waiting for mslt_step_apply");
  if (k < 1 || k > c->L) return fail(MSLT_ERR_STATE, "add_layers: need 1 <= k <= L (k=%d, L=%d)", k, c->L);
  if (k % g) return fail(MSLT_ERR_STATE, "add_layers: k = %d is not a whole number of shared groups of %d layers", k, g);
  if (c->L + k > c->a.max_layers)
    return fail(MSLT_ERR_STATE, "add_layers: L + k = %d exceeds max_layers = %d", c->L + k, c->a.max_layers);
  const int64_t src = c->layer0_off + (int64_t)((c->L - k) / g) * c->layer_cnt;
  const int64_t dst = c->layer0_off + (int64_t)(c->L / g) * c->layer_cnt;
  const int64_t n = (int64_t)(k / g) * c->layer_cnt;
  CUDA_TRY(cudaMemcpyAsync(c->master + dst, c->master + src, n * 4, cudaMemcpyDeviceToDevice, c->st));
  if (c->bf)
    CUDA_TRY(cudaMemcpyAsync(c->wb + dst * 2, c->wb + src * 2, n * 2, cudaMemcpyDeviceToDevice, c->st));
  c->L += k;
  return reset_optimizer(c);
}

int mslt_set_trainable(mslt_ctx* c, int32_t top_k) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  if (c->pending_update) return fail(MSLT_ERR_STATE, "set_trainable: a step is waiting for mslt_step_apply");
  if (top_k < 0 || top_k > c->L) return fail(MSLT_ERR_STATE, "set_trainable: need 0 <= top_k <= L");
  if (top_k % group_of(c->a))
    return fail(MSLT_ERR_STATE, "set_trainable: top_k = %d is not a whole number of shared groups", top_k);
  if (top_k > trainable_slots(c->a))
    return fail(MSLT_ERR_SIZE, "set_trainable: top_k = %d exceeds max_trainable = %d, the number of saved-activation "
                "slots the workspace was sized for", top_k, trainable_slots(c->a));
  c->top_k = top_k;
  return reset_optimizer(c);
}

int mslt_set_optimizer(mslt_ctx* c, const mslt_opt* o) {
  if (!c || !o) return fail(MSLT_ERR_ARG, "null pointer");
  if (!(o->beta1 >= 0.f && o->beta1 < 1.f && o->beta2 >= 0.f && o->beta2 < 1.f && o->eps > 0.f))
    return fail(MSLT_ERR_ARG, "bad Adam hyper-parameters");
  if (o->lamb != 0 && o->lamb != 1) return fail(MSLT_ERR_ARG, "lamb must be 0 or 1");
  c->opt = *o;
  return 0;
}

static int apply_update(mslt_ctx* c);

// forward, loss and backward of one step; the optimizer runs too unless `defer_update`
static int step_impl(mslt_ctx* c, const int32_t* d_tokens, const int32_t* d_seq_lens,
                     const int32_t* d_pos, const int32_t* d_lab, int32_t B, int32_t S, int32_t P,
                     const int32_t* d_total_valid, bool defer_update, float* loss_out,
                     const int32_t* d_seg = nullptr, const int32_t* d_nsp_lab = nullptr) {
  if (!c || !d_tokens || !d_pos || !d_lab) return fail(MSLT_ERR_ARG, "null pointer");
  if ((d_seg || d_nsp_lab) && !c->a.nsp)
    return fail(MSLT_ERR_STATE, "segment ids / NSP labels need a context created with arch.nsp = 1");
  if (c->pending_update)
    return fail(MSLT_ERR_STATE, "mslt_step_backward was called: call mslt_step_apply before the next step");
  TRY(check_batch(c, B, S, P));
  if (P < 1) return fail(MSLT_ERR_ARG, "P must be >= 1");
  Workspace& w = c->ws;
  const int H = c->a.hidden, V = c->a.vocab, T = B * S, R = B * P;
  const int first = c->L - c->top_k;
  const bool full = c->top_k == c->L;
  int* status = w.scalars;
  float* inv_n = (float*)(w.scalars + 2);
  float* loss = (float*)(w.scalars + 3);
  if (c->timing && !c->have_events) {
    for (int i = 0; i < 6; i++) CUDA_TRY(cudaEventCreate(&c->ev[i]));
    c->have_events = true;
  }
  CUDA_TRY(cudaMemsetAsync(w.scalars, 0, 16, c->st));
  c->prec.clear();
  mark(c, 0);
  KL(PC_OTHER, 16.0 * B * P, launch_slots_prepare(d_pos, d_lab, d_seq_lens, B, S, P, V, w.rowsrc, w.rowlabel, w.scalars + 1,
                          inv_n, status, c->st));
  if (d_total_valid)  // the mean runs over the valid slots of every rank's batch
    KL(PC_OTHER, 8.0, launch_override_inv_n(d_total_valid, inv_n, c->st));
  // embeddings, then the frozen prefix: forward only, two buffers, nothing kept but the output
  KL(PC_LN_FWD, 2.0 * T * H * c->esz, launch_embed_ln(c->bf, d_tokens, d_seg, Wc(c, toff(c, -1, "emb.word")), Wc(c, toff(c, -1, "emb.pos")),
                     c->a.nsp ? Wc(c, toff(c, -1, "emb.type")) : nullptr,
                     Wv(c, toff(c, -1, "emb.ln.gamma")), Wv(c, toff(c, -1, "emb.ln.beta")), w.xa,
                     full ? w.z0 : nullptr, full ? w.st0 : nullptr, T, S, H, V, c->a.ln_eps, status,
                     c->st));
  char* cur = w.xa;
  for (int l = 0; l < first; l++) {
    char* out = cur == w.xa ? w.xb : w.xa;
    TRY(layer_forward(c, l, cur, w.scratch, out, false, B, S, d_seq_lens));
    cur = out;
  }
  const char* boundary = cur;  // the only output of the frozen prefix
  mark(c, 1);
  for (int l = first; l < c->L; l++) {
    LayerBuf& slot = w.layer[l - first];
    TRY(layer_forward(c, l, cur, slot, slot.xout, true, B, S, d_seq_lens));
    cur = slot.xout;
  }
  mark(c, 2);
  TRY(head_forward(c, cur, R, true));
  KL(PC_CROSS_ENTROPY, (double)R * c->Vp * (4 + c->esz), launch_cross_entropy(c->bf, w.logits, c->Vp, w.rowlabel, inv_n, w.dlogits, c->Vp, w.nll, R, V, c->st));
  KL(PC_OTHER, 4.0 * R, launch_loss_reduce(w.nll, R, inv_n, loss, c->st));
  const bool nsp = c->a.nsp && d_nsp_lab != nullptr;
  float* nsp_inv_n = (float*)(w.scalars + 7);
  if (nsp) {
    // second objective, forward: pooled = tanh(Wp x_L[b, 0] + bp)
    const int32_t* nsp_total = d_total_valid ? d_total_valid + 1 : nullptr;
    KL(PC_OTHER, 8.0 * B, launch_nsp_prepare(d_nsp_lab, B, S, w.nsp_rowsrc, nsp_inv_n, nsp_total, c->st));
    KL(PC_OTHER, 2.0 * B * H * c->esz, launch_gather_rows(c->bf, cur, w.nsp_rowsrc, w.cls, B, H, c->st));
    TRY(linear_fwd(c, w.cls, B, H, toff(c, -1, "head.pooler.weight"), toff(c, -1, "head.pooler.bias"), H, w.up, 0,
                   nullptr, nullptr));
    KL(PC_OTHER, 2.0 * B * H * c->esz, launch_tanh(c->bf, w.up, w.pooled, (int64_t)B * H, c->st));
  }
  TRY(zero_trainable_grads(c));
  TRY(head_backward(c, B, S, P, full));
  if (nsp) {
    // classifier, its loss (added to the MLM loss) and its gradients; then back through the pooler
    // into the first token's row of the last hidden state's gradient
    KL(PC_OTHER, 4.0 * B * H * c->esz, launch_nsp_head(c->bf, w.pooled, Wv(c, toff(c, -1, "head.nsp.weight")),
                     Wv(c, toff(c, -1, "head.nsp.bias")), d_nsp_lab, nsp_inv_n, w.dup,
                     G(c, toff(c, -1, "head.nsp.weight")), G(c, toff(c, -1, "head.nsp.bias")), loss, B, H, c->st));
    TRY(linear_wgrad(c, w.dup, B, H, H, w.cls, H, toff(c, -1, "head.pooler.weight")));
    KL(PC_COLSUM, 1.0 * B * H * c->esz, launch_colsum(c->bf, w.dup, H, B, H, G(c, toff(c, -1, "head.pooler.bias")), c->st));
    TRY(linear_dgrad(c, w.dup, B, H, H, toff(c, -1, "head.pooler.weight"), H, w.dcls, 0, nullptr, nullptr));
    KL(PC_OTHER, 2.0 * B * H * c->esz, launch_scatter_rows(c->bf, w.dcls, w.nsp_rowsrc, w.dxa, B, 1, H, c->st));
  }
  TRY(bucket_done(c, 0));
  mark(c, 3);
  char* dx = w.dxa;
  char* dx_other = w.dxb;
  for (int l = c->L - 1; l >= first; l--) {
    const void* x_in = l == first ? (const void*)boundary : (const void*)w.layer[l - 1 - first].xout;
    const bool need_dx = l > first || full;
    TRY(layer_backward(c, l, x_in, w.layer[l - first], dx, dx_other, need_dx, B, S));
    if (need_dx) std::swap(dx, dx_other);
    if (l % group_of(c->a) == 0)  // the lowest layer of a parameter block completes its gradients
      TRY(bucket_done(c, (c->L - l) / group_of(c->a)));
  }
  if (full) {
    KL(PC_LN_BWD, 3.0 * T * H * c->esz, launch_ln_bwd(c->bf, dx, w.z0, w.st0, Wv(c, toff(c, -1, "emb.ln.gamma")), w.dz2,
                     G(c, toff(c, -1, "emb.ln.gamma")), G(c, toff(c, -1, "emb.ln.beta")), nullptr, T, H, c->st));
    // rows grouped by token id (counting sort), one block per id, batch sum per position: no hot-row
    // atomics, same bits on every run
    KL(PC_OTHER, 2.0 * T * H * c->esz, launch_embed_grad_sorted(c->bf, w.dz2, d_tokens, G(c, toff(c, -1, "emb.word")),
                            G(c, toff(c, -1, "emb.pos")), B, S, H, V, w.es_counts, w.es_total, w.es_start,
                            w.es_rank, w.es_order, w.es_blocksum, w.es_hot, w.es_partial, c->st));
    c->launches += 8;
    if (c->a.nsp)
      KL(PC_OTHER, 1.0 * T * H * c->esz, launch_type_grad(c->bf, w.dz2, d_seg, G(c, toff(c, -1, "emb.type")), T, H, c->st));
    TRY(bucket_done(c, c->top_k / group_of(c->a) + 1));
  }
  mark(c, 4);
  if (defer_update) {
    c->pending_update = true;
    return finish(c, loss_out);
  }
  TRY(apply_update(c));
  mark(c, 5);
  if (c->timing && c->have_events) {
    CUDA_TRY(cudaEventSynchronize(c->ev[5]));
    for (int i = 0; i < 5; i++) cudaEventElapsedTime(&c->phase_ms[i], c->ev[i], c->ev[i + 1]);
  }
  if (c->profile) {
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (size_t i = 0; i < c->prec.size(); i++) {
      float ms = 0.f;
      cudaEventElapsedTime(&ms, c->pev[2 * i], c->pev[2 * i + 1]);
      double* a = c->prof[c->prec[i].cls];
      a[0] += 1.0; a[1] += c->prec[i].flops; a[2] += ms;
    }
  }
  return finish(c, loss_out);
}

// the optimizer on the trainable slice (Adam or LAMB), after any gradient exchange
static int apply_update(mslt_ctx* c) {
  Workspace& w = c->ws;
  if (c->bucket_fn && c->comm) {  // the reductions enqueued on the communication stream come first
    if (!c->comm_done) CUDA_TRY(cudaEventCreateWithFlags(&c->comm_done, cudaEventDisableTiming));
    CUDA_TRY(cudaEventRecord(c->comm_done, c->comm));
    CUDA_TRY(cudaStreamWaitEvent(c->st, c->comm_done, 0));
  }
  c->t_step += 1;
  AdamHyper h;
  h.lr = c->opt.lr; h.beta1 = c->opt.beta1; h.beta2 = c->opt.beta2; h.eps = c->opt.eps;
  h.weight_decay = c->opt.weight_decay;
  h.omb1 = (float)(1.0 - (double)c->opt.beta1);
  h.omb2 = (float)(1.0 - (double)c->opt.beta2);
  h.bc1 = h.bc2 = 1.f;  // formed on the device from the step count kept there
  if (c->opt.lamb) {
    KL(PC_ADAM, 42.0 * c->n_chunks * kAdamChunk, launch_lamb(w.chunks, c->n_chunks, c->master, c->grad, c->m, c->v, c->wb, h,
                   w.scalars + 4, (float*)(w.scalars + 5), c->opt.bias_correction, w.norms, (int)c->tensors.size(), c->st));
    c->launches += 2;  // step-count kernel, moments kernel, update kernel
  } else {
    KL(PC_ADAM, 30.0 * c->n_chunks * kAdamChunk, launch_adam(w.chunks, c->n_chunks, c->master, c->grad, c->m, c->v, c->wb, h, w.scalars + 4,
                   (float*)(w.scalars + 5), c->opt.bias_correction, c->st));
    c->launches++;  // step-count kernel and update kernel
  }
  return 0;
}

int mslt_step(mslt_ctx* c, const int32_t* d_tokens, const int32_t* d_seq_lens,
              const int32_t* d_pos, const int32_t* d_lab, int32_t B, int32_t S, int32_t P,
              float* loss_out) {
  return step_impl(c, d_tokens, d_seq_lens, d_pos, d_lab, B, S, P, nullptr, false, loss_out);
}

int mslt_step_nsp(mslt_ctx* c, const int32_t* d_tokens, const int32_t* d_seq_lens, const int32_t* d_seg,
                  const int32_t* d_pos, const int32_t* d_lab, const int32_t* d_nsp_lab, int32_t B, int32_t S,
                  int32_t P, float* loss_out) {
  if (c && !c->a.nsp) return fail(MSLT_ERR_STATE, "mslt_step_nsp needs a context created with arch.nsp = 1");
  return step_impl(c, d_tokens, d_seq_lens, d_pos, d_lab, B, S, P, nullptr, false, loss_out, d_seg, d_nsp_lab);
}

int mslt_step_backward(mslt_ctx* c, const int32_t* d_tokens, const int32_t* d_seq_lens,
                       const int32_t* d_pos, const int32_t* d_lab, int32_t B, int32_t S, int32_t P,
                       const int32_t* d_total_valid, float* loss_out) {
  return step_impl(c, d_tokens, d_seq_lens, d_pos, d_lab, B, S, P, d_total_valid, true, loss_out);
}

int mslt_step_apply(mslt_ctx* c) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  if (!c->pending_update) return fail(MSLT_ERR_STATE, "mslt_step_apply without a preceding mslt_step_backward");
  c->pending_update = false;
  TRY(apply_update(c));
  CUDA_TRY(cudaGetLastError());
  return 0;
}

int mslt_num_grad_buckets(const mslt_ctx* c) { return c ? num_buckets(c) : MSLT_ERR_ARG; }

int mslt_grad_bucket(mslt_ctx* c, int32_t i, float** d_ptr, int64_t* count) {
  if (!c || !d_ptr || !count) return fail(MSLT_ERR_ARG, "null pointer");
  if (i < 0 || i >= num_buckets(c)) return fail(MSLT_ERR_ARG, "no such gradient bucket");
  int64_t off, cnt;
  bucket_range(c, i, &off, &cnt);
  *d_ptr = c->grad + off;
  *count = cnt;
  return 0;
}

int mslt_set_bucket_hook(mslt_ctx* c, void* comm_stream, mslt_bucket_fn fn, void* user) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  if (fn && !comm_stream) return fail(MSLT_ERR_ARG, "a hook needs a communication stream");
  c->comm = (cudaStream_t)comm_stream;
  c->bucket_fn = fn;
  c->bucket_user = user;
  return 0;
}

int mslt_read_loss(mslt_ctx* c, float* loss_out) {
  if (!c || !loss_out) return fail(MSLT_ERR_ARG, "null pointer");
  return finish(c, loss_out);
}

int mslt_forward(mslt_ctx* c, const int32_t* d_tokens, const int32_t* d_seq_lens, int32_t B, int32_t S,
                 void* d_hidden_out, const int32_t* d_pos, int32_t P, float* d_logits_out) {
  if (!c || !d_tokens) return fail(MSLT_ERR_ARG, "null pointer");
  const bool head = d_pos != nullptr && d_logits_out != nullptr;
  TRY(check_batch(c, B, S, head ? P : 0));
  if (head && P < 1) return fail(MSLT_ERR_ARG, "P must be >= 1");
  Workspace& w = c->ws;
  const int H = c->a.hidden, V = c->a.vocab, T = B * S;
  CUDA_TRY(cudaMemsetAsync(w.scalars, 0, 16, c->st));
  if (head)
    KL(PC_OTHER, 8.0 * B * P, launch_slots_prepare(d_pos, nullptr, d_seq_lens, B, S, P, V, w.rowsrc, w.rowlabel,
                            w.scalars + 1, (float*)(w.scalars + 2), w.scalars, c->st));
  KL(PC_LN_FWD, 2.0 * T * H * c->esz, launch_embed_ln(c->bf, d_tokens, nullptr, Wc(c, toff(c, -1, "emb.word")), Wc(c, toff(c, -1, "emb.pos")),
                     c->a.nsp ? Wc(c, toff(c, -1, "emb.type")) : nullptr,
                     Wv(c, toff(c, -1, "emb.ln.gamma")), Wv(c, toff(c, -1, "emb.ln.beta")), w.xa,
                     nullptr, nullptr, T, S, H, V, c->a.ln_eps, w.scalars, c->st));
  char* cur = w.xa;
  for (int l = 0; l < c->L; l++) {
    char* out = cur == w.xa ? w.xb : w.xa;
    TRY(layer_forward(c, l, cur, w.scratch, out, false, B, S, d_seq_lens));
    cur = out;
  }
  if (d_hidden_out)
    CUDA_TRY(cudaMemcpyAsync(d_hidden_out, cur, (size_t)T * H * c->esz, cudaMemcpyDeviceToDevice, c->st));
  if (head) {
    TRY(head_forward(c, cur, B * P, false));
    CUDA_TRY(cudaMemcpy2DAsync(d_logits_out, (size_t)V * 4, w.logits, (size_t)c->Vp * 4, (size_t)V * 4,
                               (size_t)B * P, cudaMemcpyDeviceToDevice, c->st));
  }
  float dummy;
  return finish(c, &dummy);
}

int mslt_num_layers(const mslt_ctx* c) { return c ? c->L : MSLT_ERR_ARG; }
int mslt_num_trainable(const mslt_ctx* c) { return c ? c->top_k : MSLT_ERR_ARG; }

int mslt_num_tensors(const mslt_ctx* c) {
  if (!c) return MSLT_ERR_ARG;
  return n_emb_tensors(c->a) + 12 * (c->L / group_of(c->a)) + n_head_tensors(c->a);
}

static const Tensor* tensor_by_index(const mslt_ctx* c, int i) {
  const int n_layer_t = 12 * (c->L / group_of(c->a));
  if (i < 0) return nullptr;
  const int ne = n_emb_tensors(c->a);
  if (i < ne + n_layer_t) return &c->tensors[i];
  i -= ne + n_layer_t;
  if (i < n_head_tensors(c->a)) return &c->tensors[ne + 12 * (c->a.max_layers / group_of(c->a)) + i];
  return nullptr;
}

int mslt_tensor_info(const mslt_ctx* c, int32_t index, const char** name, int32_t* rank,
                     int64_t shape[2], int32_t* trainable) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  const Tensor* t = tensor_by_index(c, index);
  if (!t) return fail(MSLT_ERR_ARG, "tensor index out of range");
  if (name) *name = t->name.c_str();
  if (rank) *rank = t->rank;
  if (shape) { shape[0] = t->shape[0]; shape[1] = t->rank == 2 ? t->shape[1] : 1; }
  if (trainable) *trainable = is_trainable(c, *t) ? 1 : 0;
  return 0;
}

static int lookup(mslt_ctx* c, const char* name, size_t n, const Tensor** t) {
  if (!c || !name) return fail(MSLT_ERR_ARG, "null pointer");
  *t = find(c, name);
  if (!*t) return fail(MSLT_ERR_ARG, "unknown tensor '%s'", name);
  if (n != (size_t)(*t)->count)
    return fail(MSLT_ERR_ARG, "tensor '%s' has %lld elements, got %zu", name, (long long)(*t)->count, n);
  return 0;
}

int mslt_get_param(mslt_ctx* c, const char* name, float* dst, size_t n) {
  const Tensor* t;
  TRY(lookup(c, name, n, &t));
  if (!dst) return fail(MSLT_ERR_ARG, "null pointer");
  CUDA_TRY(cudaStreamSynchronize(c->st));
  CUDA_TRY(cudaMemcpyAsync(dst, c->master + t->offset, n * 4, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  return 0;
}

int mslt_set_param(mslt_ctx* c, const char* name, const float* src, size_t n) {
  const Tensor* t;
  TRY(lookup(c, name, n, &t));
  if (!src) return fail(MSLT_ERR_ARG, "null pointer");
  CUDA_TRY(cudaStreamSynchronize(c->st));
  // in the context's stream, so that the conversion kernel below is ordered after the copy even
  // when that stream does not synchronise with the default stream
  CUDA_TRY(cudaMemcpyAsync(c->master + t->offset, src, n * 4, cudaMemcpyHostToDevice, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  if (c->bf) {
    KL(PC_OTHER, 6.0 * n, launch_f32_to_bf16(c->master + t->offset, c->wb + t->offset * 2, (int64_t)n, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
  }
  return 0;
}

int mslt_get_param_raw(mslt_ctx* c, const char* name, void* dst, size_t bytes) {
  if (!c || !name || !dst) return fail(MSLT_ERR_ARG, "null pointer");
  const Tensor* t = find(c, name);
  if (!t) return fail(MSLT_ERR_ARG, "unknown tensor '%s'", name);
  const bool b = c->bf && t->rank == 2;
  const size_t want = (size_t)t->count * (b ? 2 : 4);
  if (bytes != want) return fail(MSLT_ERR_ARG, "tensor '%s' needs %zu raw bytes, got %zu", name, want, bytes);
  CUDA_TRY(cudaStreamSynchronize(c->st));
  const void* src = b ? (const void*)(c->wb + t->offset * 2) : (const void*)(c->master + t->offset);
  CUDA_TRY(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  return 0;
}

int mslt_get_grad(mslt_ctx* c, const char* name, float* dst, size_t n) {
  const Tensor* t;
  TRY(lookup(c, name, n, &t));
  if (!dst) return fail(MSLT_ERR_ARG, "null pointer");
  if (!is_trainable(c, *t)) return fail(MSLT_ERR_STATE, "tensor '%s' is frozen: it has no gradient", name);
  CUDA_TRY(cudaStreamSynchronize(c->st));
  CUDA_TRY(cudaMemcpyAsync(dst, c->grad + t->offset, n * 4, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  return 0;
}

int mslt_get_opt_state(mslt_ctx* c, const char* name, int32_t which, float* dst, size_t n) {
  const Tensor* t;
  TRY(lookup(c, name, n, &t));
  if (!dst || which < 0 || which > 1) return fail(MSLT_ERR_ARG, "bad argument");
  if (!is_trainable(c, *t)) return fail(MSLT_ERR_STATE, "tensor '%s' is frozen: it has no optimizer state", name);
  CUDA_TRY(cudaStreamSynchronize(c->st));
  CUDA_TRY(cudaMemcpyAsync(dst, (which ? c->v : c->m) + t->offset, n * 4, cudaMemcpyDeviceToHost, c->st));
  CUDA_TRY(cudaStreamSynchronize(c->st));
  return 0;
}

int64_t mslt_launch_count(const mslt_ctx* c) { return c ? c->launches : 0; }

int mslt_set_timing(mslt_ctx* c, int32_t on) {
  if (!c) return fail(MSLT_ERR_ARG, "null context");
  c->timing = on != 0;
  c->profile = on >= 2 ? 1 : 0;
  if (c->profile && c->pev.empty()) {
    c->pev.resize(2 * 1024);
    for (cudaEvent_t& e : c->pev) CUDA_TRY(cudaEventCreate(&e));
  }
  return 0;
}

int mslt_get_kernel_profile(mslt_ctx* c, double* out, int32_t n) {
  if (!c || !out || n < 3 * PC_COUNT) return fail(MSLT_ERR_ARG, "need room for 30 doubles");
  for (int k = 0; k < PC_COUNT; k++)
    for (int j = 0; j < 3; j++) out[3 * k + j] = c->prof[k][j];
  memset(c->prof, 0, sizeof(c->prof));
  return 0;
}

int mslt_get_timings(mslt_ctx* c, float* ms, int32_t n) {
  if (!c || !ms || n < 5) return fail(MSLT_ERR_ARG, "need room for 5 floats");
  if (!c->have_events) return fail(MSLT_ERR_STATE, "no timed step has run");
  for (int i = 0; i < 5; i++) ms[i] = c->phase_ms[i];
  return 0;
}

int mslt_debug_check_guards(mslt_ctx* c, int32_t* bad_out) {
  if (!c || !bad_out) return fail(MSLT_ERR_ARG, "null pointer");
  CUDA_TRY(cudaStreamSynchronize(c->st));
  const char* base = (const char*)c->ws.scalars;  // the first buffer of the workspace
  std::vector<uint64_t> host(32);
  int bad = 0;
  for (size_t off : c->ws.guards) {
    CUDA_TRY(cudaMemcpyAsync(host.data(), base + off, 256, cudaMemcpyDeviceToHost, c->st));
    CUDA_TRY(cudaStreamSynchronize(c->st));
    for (uint64_t v : host)
      if (v != 0) { bad++; break; }
  }
  *bad_out = bad;
  return 0;
}

int mslt_debug_starve_next_attention(int32_t on) {
  attn_starve_next(on);
  return 0;
}

int mslt_debug_starve_next_gemm(int32_t on) {
  gemm_tc_starve_next(on);
  return 0;
}

int mslt_debug_set_gemm_variant(int32_t variant) {
  if (variant < 0 || (variant & 3) > 2 || variant > 6) return fail(MSLT_ERR_ARG, "variant must be 0, 1 or 2, plus 4 or not");
  gemm_tc_set_variant(variant);
  return 0;
}

static int check_gemm_desc(const mslt_gemm_desc* d) {
  if (!d || !d->A || !d->B || !d->D) return fail(MSLT_ERR_ARG, "null pointer");
  if (d->M < 1 || d->N < 1 || d->K < 1 || d->batch < 1 || d->hdiv < 1)
    return fail(MSLT_ERR_ARG, "bad GEMM shape");
  if ((d->a_rs != 1 && d->a_ks != 1) || (d->b_rs != 1 && d->b_ks != 1))
    return fail(MSLT_ERR_ARG, "each operand needs one unit stride");
  if (d->accumulate && !d->d_fp32) return fail(MSLT_ERR_ARG, "accumulate needs an fp32 output");
  if (d->act == 2 && !d->aux) return fail(MSLT_ERR_ARG, "act 2 needs aux");
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0)
    return fail(MSLT_ERR_CUDA, "no CUDA device: this library has no CPU path");
  return 0;
}

int mslt_op_gemm_enqueue(const mslt_gemm_desc* d, void* cuda_stream, int32_t* d_status) {
  TRY(check_gemm_desc(d));
  char err[256] = "";
  int rc = gemm_launch(*d, d_status, (cudaStream_t)cuda_stream, err);
  if (rc) return fail(rc, "%s", err);
  CUDA_TRY(cudaGetLastError());
  return 0;
}

int mslt_op_gemm(const mslt_gemm_desc* d, void* cuda_stream, int32_t* d_status) {
  TRY(mslt_op_gemm_enqueue(d, cuda_stream, d_status));
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CUDA_TRY(cudaStreamSynchronize(st));
  if (d_status) {
    int h = 0;
    CUDA_TRY(cudaMemcpyAsync(&h, d_status, 4, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    if (h) return fail(MSLT_ERR_DEVICE, "device status 0x%x: a kernel wait ran out", h);
  }
  return 0;
}

}  // extern "C"
