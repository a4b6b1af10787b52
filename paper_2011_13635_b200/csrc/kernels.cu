// Fused memory-bound kernels of the MSLT stage step: embedding gather + LayerNorm,
// LayerNorm forward/backward, masked softmax forward/backward, MLM row
// gather/scatter, softmax cross-entropy with in-place gradient, column sums for
// bias gradients, embedding gradient scatter and Adam on the trainable slice.
// All are HBM-bound: rows are moved with 16-byte accesses, one warp (or one
// block) per row, reductions by warp shuffles, statistics in fp32.
#include "kernels.h"

#include <algorithm>

#include "common.cuh"

namespace mslt {

constexpr int LN_MAXE = 32;  // elements of a row held by one lane: hidden <= 1024

static inline int div_up(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// ---------------------------------------------------------------------------------------
// LayerNorm forward.  y = gamma * (z - mean) * rstd + beta, biased variance.
// ---------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void ln_finish_row(float (&x)[LN_MAXE], int lane, int H,
                                              const float* __restrict__ gamma,
                                              const float* __restrict__ beta, T* __restrict__ yrow,
                                              float* __restrict__ stat, float eps) {
  constexpr int VN = VecT<T>::N;
  constexpr int NV = LN_MAXE / VN;
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; i++) {
    if ((lane + 32 * i) * VN < H) {
#pragma unroll
      for (int e = 0; e < VN; e++) s += x[i * VN + e];
    }
  }
  const float mean = warp_sum(s) / (float)H;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < NV; i++) {
    if ((lane + 32 * i) * VN < H) {
#pragma unroll
      for (int e = 0; e < VN; e++) {
        float d = x[i * VN + e] - mean;
        q += d * d;
      }
    }
  }
  const float rstd = rsqrtf(warp_sum(q) / (float)H + eps);
  if (stat != nullptr && lane == 0) {
    stat[0] = mean;
    stat[1] = rstd;
  }
#pragma unroll
  for (int i = 0; i < NV; i++) {
    const int c = (lane + 32 * i) * VN;
    if (c < H) {
      float o[VN], g[VN], b[VN];
#pragma unroll
      for (int e = 0; e < VN; e += 4) {  // 16-byte loads: scalar ones flood L1 with strided sectors
        const float4 g4 = *reinterpret_cast<const float4*>(gamma + c + e);
        const float4 b4 = *reinterpret_cast<const float4*>(beta + c + e);
        g[e] = g4.x; g[e + 1] = g4.y; g[e + 2] = g4.z; g[e + 3] = g4.w;
        b[e] = b4.x; b[e + 1] = b4.y; b[e + 2] = b4.z; b[e + 3] = b4.w;
      }
#pragma unroll
      for (int e = 0; e < VN; e++) o[e] = g[e] * ((x[i * VN + e] - mean) * rstd) + b[e];
      VecT<T>::store(yrow + c, o);
    }
  }
}

// One warp normalises ROWS consecutive rows at once: all their 16-byte loads are issued before
// the first reduction, which keeps enough bytes in flight to approach HBM bandwidth, and gamma /
// beta are fetched once per column vector for all ROWS rows.  NV = 16-byte vectors per lane.
template <typename T, int NV, int ROWS>
__global__ void __launch_bounds__(256)
ln_fwd_kernel(const T* __restrict__ z, const float* __restrict__ gamma, const float* __restrict__ beta,
              T* __restrict__ y, float* __restrict__ stats, int rows, int H, float eps) {
  constexpr int VN = VecT<T>::N;
  typedef typename VecT<T>::Raw Raw;
  const int lane = threadIdx.x & 31;
  const int row0 = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * ROWS;
  if (row0 >= rows) return;
  Raw raw[ROWS][NV];
#pragma unroll
  for (int r = 0; r < ROWS; r++)
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (lane + 32 * i) * VN;
      if (c < H && row0 + r < rows) raw[r][i] = VecT<T>::load_raw(z + (int64_t)(row0 + r) * H + c);
    }
  // One reduction round for both moments: sums of (x - x0) and (x - x0)^2 with x0 the first element
  // of the row, which keeps the subtraction var = E[d^2] - E[d]^2 well conditioned (x0 lies within
  // the spread of the row).
  float mean[ROWS], rstd[ROWS];
#pragma unroll
  for (int r = 0; r < ROWS; r++) {
    float first[VN];
    VecT<T>::unpack(raw[r][0], first);
    const float x0 = __shfl_sync(0xffffffffu, first[0], 0);
    // packed two-wide fp32 arithmetic: the kernel is bound by instruction issue, not by memory
    float2 s1 = make_float2(0.f, 0.f), s2 = make_float2(0.f, 0.f);
    const float2 nx0 = make_float2(-x0, -x0);
#pragma unroll
    for (int i = 0; i < NV; i++) {
      if ((lane + 32 * i) * VN < H && row0 + r < rows) {
        float t[VN];
        VecT<T>::unpack(raw[r][i], t);
#pragma unroll
        for (int e = 0; e < VN; e += 2) {
          const float2 d = __fadd2_rn(make_float2(t[e], t[e + 1]), nx0);
          s1 = __fadd2_rn(s1, d);
          s2 = __ffma2_rn(d, d, s2);
        }
      }
    }
    mean[r] = s1.x + s1.y;
    rstd[r] = s2.x + s2.y;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
    for (int r = 0; r < ROWS; r++) {
      mean[r] += __shfl_xor_sync(0xffffffffu, mean[r], o);
      rstd[r] += __shfl_xor_sync(0xffffffffu, rstd[r], o);
    }
  }
#pragma unroll
  for (int r = 0; r < ROWS; r++) {
    float first[VN];
    VecT<T>::unpack(raw[r][0], first);
    const float x0 = __shfl_sync(0xffffffffu, first[0], 0);
    const float m1 = mean[r] / (float)H;
    const float var = fmaxf(rstd[r] / (float)H - m1 * m1, 0.f);
    mean[r] = x0 + m1;
    rstd[r] = rsqrtf(var + eps);
  }
  if (stats != nullptr && lane == 0) {
#pragma unroll
    for (int r = 0; r < ROWS; r++)
      if (row0 + r < rows) {
        stats[2 * (int64_t)(row0 + r)] = mean[r];
        stats[2 * (int64_t)(row0 + r) + 1] = rstd[r];
      }
  }
#pragma unroll
  for (int i = 0; i < NV; i++) {
    const int c = (lane + 32 * i) * VN;
    if (c < H) {
      float g[VN], b[VN];
#pragma unroll
      for (int e = 0; e < VN; e += 4) {
        const float4 g4 = *reinterpret_cast<const float4*>(gamma + c + e);
        const float4 b4 = *reinterpret_cast<const float4*>(beta + c + e);
        g[e] = g4.x; g[e + 1] = g4.y; g[e + 2] = g4.z; g[e + 3] = g4.w;
        b[e] = b4.x; b[e + 1] = b4.y; b[e + 2] = b4.z; b[e + 3] = b4.w;
      }
#pragma unroll
      for (int r = 0; r < ROWS; r++) {
        if (row0 + r < rows) {
          // y = x * (gamma * rstd) + (beta - mean * rstd * gamma)
          float t[VN], o[VN];
          VecT<T>::unpack(raw[r][i], t);
          const float2 r2 = make_float2(rstd[r], rstd[r]), nm2 = make_float2(-mean[r] * rstd[r], -mean[r] * rstd[r]);
#pragma unroll
          for (int e = 0; e < VN; e += 2) {
            const float2 g2 = make_float2(g[e], g[e + 1]);
            const float2 o2 = __ffma2_rn(make_float2(t[e], t[e + 1]), __fmul2_rn(g2, r2),
                                         __ffma2_rn(nm2, g2, make_float2(b[e], b[e + 1])));
            o[e] = o2.x; o[e + 1] = o2.y;
          }
          VecT<T>::store(y + (int64_t)(row0 + r) * H + c, o);
        }
      }
    }
  }
}

// Embedding: z = word[token] + pos[s]; optional stash of z; then LayerNorm.
template <typename T>
__global__ void __launch_bounds__(256)
embed_ln_kernel(const int* __restrict__ tokens, const int* __restrict__ segments,
                const T* __restrict__ word, const T* __restrict__ pos, const T* __restrict__ type,
                const float* __restrict__ gamma,
                const float* __restrict__ beta, T* __restrict__ y, T* __restrict__ zstash,
                float* __restrict__ stats, int rows, int S, int H, int V, float eps,
                int* __restrict__ status) {
  constexpr int VN = VecT<T>::N;
  constexpr int NV = LN_MAXE / VN;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  int tok = tokens[row];
  if (tok < 0 || tok >= V) {
    if (lane == 0) atomicOr(status, ST_BAD_TOKEN);
    tok = 0;
  }
  const T* wr = word + (int64_t)tok * H;
  const T* pr = pos + (int64_t)(row % S) * H;
  // segment (token-type) row: table of two rows; ids outside {0, 1} are reported and read as 0
  const T* tr = nullptr;
  if (type != nullptr) {
    int sg = segments ? segments[row] : 0;
    if (sg < 0 || sg > 1) {
      if (lane == 0) atomicOr(status, ST_BAD_TOKEN);
      sg = 0;
    }
    tr = type + (int64_t)sg * H;
  }
  float x[LN_MAXE];
#pragma unroll
  for (int i = 0; i < NV; i++) {
    const int c = (lane + 32 * i) * VN;
    if (c < H) {
      float a[VN], b[VN];
      VecT<T>::load(wr + c, a);
      VecT<T>::load(pr + c, b);
      if (tr != nullptr) {
        float t3[VN];
        VecT<T>::load(tr + c, t3);
#pragma unroll
        for (int e = 0; e < VN; e++) b[e] += t3[e];
      }
      // round the sum to the storage type first: the backward pass normalises the stashed copy
#pragma unroll
      for (int e = 0; e < VN; e++) a[e] = to_f<T>(from_f<T>(a[e] + b[e]));
      if (zstash != nullptr) VecT<T>::store(zstash + (int64_t)row * H + c, a);
#pragma unroll
      for (int e = 0; e < VN; e++) x[i * VN + e] = a[e];
    }
  }
  ln_finish_row<T>(x, lane, H, gamma, beta, y + (int64_t)row * H,
                   stats ? stats + 2 * (int64_t)row : nullptr, eps);
}

// ---------------------------------------------------------------------------------------
// LayerNorm backward: dz = rstd * (dxhat - mean(dxhat) - xhat * mean(dxhat * xhat)),
// dgamma += sum_rows dy * xhat, dbeta += sum_rows dy and, when asked for, dbias += sum_rows dz
// (the bias gradient of the linear layer whose output was normalised) - fp32 atomics, one per
// column per block.
// A row is split over NSLICE warps, each owning one 16-byte vector per lane, so that the column
// accumulators cost a lane 3 x 8 registers instead of 3 x 24 and twice as many loads are in
// flight per SM; a warp works on LN_BWD_ROWS rows at once and the NSLICE partial row sums meet in shared
// memory (double-buffered: one block barrier per LR rows).
// ---------------------------------------------------------------------------------------
template <typename T, int NSLICE, int RG, int LN_BWD_ROWS>
__global__ void __launch_bounds__(NSLICE * RG * 32, 1)
ln_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ z, const float* __restrict__ stats,
              const float* __restrict__ gamma, T* __restrict__ dz, float* __restrict__ dgamma,
              float* __restrict__ dbeta, float* __restrict__ dbias, int rows, int H) {
  constexpr int VN = VecT<T>::N;
  constexpr int LR = LN_BWD_ROWS;  // rows a warp has in flight
  typedef typename VecT<T>::Raw Raw;
  __shared__ float part[2][RG][LR][NSLICE][2];
  __shared__ float red[RG][NSLICE * 32 * VN];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slice = warp % NSLICE, rg = warp / NSLICE;
  const int c = (slice * 32 + lane) * VN;
  const bool col_ok = c < H;
  float g[VN], ag[VN], ab[VN], az[VN];
#pragma unroll
  for (int e = 0; e < VN; e++) { g[e] = 0.f; ag[e] = 0.f; ab[e] = 0.f; az[e] = 0.f; }
  if (col_ok) {
#pragma unroll
    for (int e = 0; e < VN; e += 4) {
      const float4 g4 = *reinterpret_cast<const float4*>(gamma + c + e);
      g[e] = g4.x; g[e + 1] = g4.y; g[e + 2] = g4.z; g[e + 3] = g4.w;
    }
  }
  const float invH = 1.0f / (float)H;
  int buf = 0;
  for (int base = blockIdx.x * (RG * LR); base < rows; base += gridDim.x * (RG * LR), buf ^= 1) {
    const int row0 = base + rg * LR;
    Raw ra[LR], rb[LR];
    float mean[LR], rstd[LR];
#pragma unroll
    for (int k = 0; k < LR; k++) {
      const bool ok = col_ok && row0 + k < rows;
      if (ok) {
        ra[k] = VecT<T>::load_raw(dy + (int64_t)(row0 + k) * H + c);
        rb[k] = VecT<T>::load_raw(z + (int64_t)(row0 + k) * H + c);
      }
      const int rr = min(row0 + k, rows - 1);
      mean[k] = stats[2 * (int64_t)rr];
      rstd[k] = stats[2 * (int64_t)rr + 1];
    }
    // Packed two-wide fp32 arithmetic and row constants folded once per row keep this at a few
    // instructions per element (the plain form was bound by instruction issue, not by memory):
    //   q = sum dy*gamma*z gives sum dy*gamma*xhat = rstd * (q - mean * s1);
    //   xhat = z * rstd + nmr;  dz = dy * (gamma * rstd) + z * c2 + c3.
    float s1[LR], s2[LR];
#pragma unroll
    for (int k = 0; k < LR; k++) {
      float2 t1 = make_float2(0.f, 0.f), tq = make_float2(0.f, 0.f);
      if (col_ok && row0 + k < rows) {
        float a[VN], b[VN];
        VecT<T>::unpack(ra[k], a);
        VecT<T>::unpack(rb[k], b);
        const float2 r2 = make_float2(rstd[k], rstd[k]), n2 = make_float2(-mean[k] * rstd[k], -mean[k] * rstd[k]);
#pragma unroll
        for (int e = 0; e < VN; e += 2) {
          const float2 a2 = make_float2(a[e], a[e + 1]), b2 = make_float2(b[e], b[e + 1]);
          const float2 dxh = __fmul2_rn(a2, make_float2(g[e], g[e + 1]));
          t1 = __fadd2_rn(t1, dxh);
          tq = __ffma2_rn(dxh, b2, tq);
          const float2 xhat = __ffma2_rn(b2, r2, n2);
          const float2 ga = __ffma2_rn(a2, xhat, make_float2(ag[e], ag[e + 1]));
          const float2 ba = __fadd2_rn(a2, make_float2(ab[e], ab[e + 1]));
          ag[e] = ga.x; ag[e + 1] = ga.y;
          ab[e] = ba.x; ab[e + 1] = ba.y;
        }
      }
      s1[k] = t1.x + t1.y;
      s2[k] = tq.x + tq.y;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int k = 0; k < LR; k++) {
        s1[k] += __shfl_xor_sync(0xffffffffu, s1[k], o);
        s2[k] += __shfl_xor_sync(0xffffffffu, s2[k], o);
      }
    if (NSLICE > 1) {
      if (lane < LR) {
        float v1 = s1[0], v2 = s2[0];
#pragma unroll
        for (int k = 1; k < LR; k++)
          if (lane == k) { v1 = s1[k]; v2 = s2[k]; }
        part[buf][rg][lane][slice][0] = v1;
        part[buf][rg][lane][slice][1] = v2;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < LR; k++) {
        float t1 = 0.f, t2 = 0.f;
#pragma unroll
        for (int w = 0; w < NSLICE; w++) { t1 += part[buf][rg][k][w][0]; t2 += part[buf][rg][k][w][1]; }
        s1[k] = t1; s2[k] = t2;
      }
    }
#pragma unroll
    for (int k = 0; k < LR; k++) {
      if (col_ok && row0 + k < rows) {
        float a[VN], b[VN], o[VN];
        VecT<T>::unpack(ra[k], a);
        VecT<T>::unpack(rb[k], b);
        const float m1 = s1[k] * invH, m2 = rstd[k] * (s2[k] - mean[k] * s1[k]) * invH;
        const float c2 = -rstd[k] * rstd[k] * m2, c3 = -rstd[k] * m1 - c2 * mean[k];
        const float2 r2 = make_float2(rstd[k], rstd[k]), c22 = make_float2(c2, c2), c32 = make_float2(c3, c3);
#pragma unroll
        for (int e = 0; e < VN; e += 2) {
          const float2 gr = __fmul2_rn(make_float2(g[e], g[e + 1]), r2);
          const float2 o2 = __ffma2_rn(make_float2(a[e], a[e + 1]), gr,
                                       __ffma2_rn(make_float2(b[e], b[e + 1]), c22, c32));
          const float2 za = __fadd2_rn(o2, make_float2(az[e], az[e + 1]));
          o[e] = o2.x; o[e + 1] = o2.y;
          az[e] = za.x; az[e + 1] = za.y;
        }
        VecT<T>::store(dz + (int64_t)(row0 + k) * H + c, o);
      }
    }
  }
  // block reduction of the column sums over the row groups, then one atomic per column
#pragma unroll
  for (int pass = 0; pass < 3; pass++) {
    float* dst = pass == 0 ? dgamma : (pass == 1 ? dbeta : dbias);
    if (dst == nullptr) continue;  // uniform over the block
    __syncthreads();
#pragma unroll
    for (int e = 0; e < VN; e++)
      red[rg][(slice * 32 + lane) * VN + e] = pass == 0 ? ag[e] : (pass == 1 ? ab[e] : az[e]);
    __syncthreads();
    for (int cc = threadIdx.x; cc < H; cc += NSLICE * RG * 32) {
      float t = 0.f;
#pragma unroll
      for (int w = 0; w < RG; w++) t += red[w][cc];
      atomicAdd(dst + cc, t);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Scaled masked softmax over the last axis of [rows, S]; key j valid iff j < len(sequence).
// ---------------------------------------------------------------------------------------
// A group of LPR lanes (16 or 32) owns a row and handles two rows per pass, so that several 16-byte
// loads per lane are in flight before the first reduction.  NV = vectors per lane.
template <typename T, int LPR, int NV>
__global__ void __launch_bounds__(256)
softmax_fwd_kernel(const T* __restrict__ sc, T* __restrict__ p, const int* __restrict__ seq_lens,
                   int rows, int S, int rows_per_seq, float scale) {
  constexpr int VN = VecT<T>::N;
  typedef typename VecT<T>::Raw Raw;
  constexpr int GPW = 32 / LPR;
  constexpr int RPG = 2;
  const int lane = threadIdx.x & 31, gl = lane % LPR;
  const int group = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * GPW + lane / LPR;
  const int row0 = group * RPG;
  if (row0 >= rows) return;   // whole groups leave together; shuffles below stay inside a group
  const unsigned gmask = LPR == 32 ? 0xffffffffu : (0xffffu << (16 * (lane / 16)));
  Raw raw[RPG][NV];
  int len[RPG];
#pragma unroll
  for (int r = 0; r < RPG; r++) {
    const int row = min(row0 + r, rows - 1);
    const int l = seq_lens ? seq_lens[row / rows_per_seq] : S;
    len[r] = min(max(l, 1), S);
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (gl + LPR * i) * VN;
      if (c < S && row0 + r < rows) raw[r][i] = VecT<T>::load_raw(sc + (int64_t)(row0 + r) * S + c);
    }
  }
  float x[RPG][NV][VN];
  float mx[RPG], sum[RPG];
#pragma unroll
  for (int r = 0; r < RPG; r++) {
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (gl + LPR * i) * VN;
      float t[VN];
      if (c < S && row0 + r < rows) VecT<T>::unpack(raw[r][i], t);
#pragma unroll
      for (int e = 0; e < VN; e++) {
        const float v = (c + e < len[r] && row0 + r < rows) ? t[e] * scale : -INFINITY;
        x[r][i][e] = v;
        m = fmaxf(m, v);
      }
    }
    mx[r] = m;
  }
#pragma unroll
  for (int r = 0; r < RPG; r++)
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) mx[r] = fmaxf(mx[r], __shfl_xor_sync(gmask, mx[r], o));
#pragma unroll
  for (int r = 0; r < RPG; r++) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < NV; i++)
#pragma unroll
      for (int e = 0; e < VN; e++) {
        const float v = x[r][i][e] == -INFINITY ? 0.f : __expf(x[r][i][e] - mx[r]);
        x[r][i][e] = v;
        s += v;
      }
    sum[r] = s;
  }
#pragma unroll
  for (int r = 0; r < RPG; r++)
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) sum[r] += __shfl_xor_sync(gmask, sum[r], o);
#pragma unroll
  for (int r = 0; r < RPG; r++) {
    const float inv = 1.0f / sum[r];
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (gl + LPR * i) * VN;
      if (c < S && row0 + r < rows) {
        float o[VN];
#pragma unroll
        for (int e = 0; e < VN; e++) o[e] = x[r][i][e] * inv;
        VecT<T>::store(p + (int64_t)(row0 + r) * S + c, o);
      }
    }
  }
}

// ds = p * (dp - sum_j dp * p) * scale, written over dp
// A group of LPR lanes (16 or 32) owns a row; each group handles two rows per pass so that four
// 16-byte loads per lane are in flight before the first reduction.  NV = vectors per lane.
template <typename T, int LPR, int NV>
__global__ void __launch_bounds__(256)
softmax_bwd_kernel(T* __restrict__ dp, const T* __restrict__ p, int rows, int S, float scale) {
  constexpr int VN = VecT<T>::N;
  typedef typename VecT<T>::Raw Raw;
  constexpr int GPW = 32 / LPR;  // groups per warp
  constexpr int RPG = 2;         // rows per group and pass
  const int lane = threadIdx.x & 31, gl = lane % LPR;
  const int group = (blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * GPW + lane / LPR;
  const int row0 = group * RPG;
  if (row0 >= rows) return;   // whole groups leave together; shuffles below stay inside a group
  const unsigned gmask = LPR == 32 ? 0xffffffffu : (0xffffu << (16 * (lane / 16)));
  Raw ra[RPG][NV], rb[RPG][NV];
#pragma unroll
  for (int r = 0; r < RPG; r++)
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (gl + LPR * i) * VN;
      if (c < S && row0 + r < rows) {
        ra[r][i] = VecT<T>::load_raw(dp + (int64_t)(row0 + r) * S + c);
        rb[r][i] = VecT<T>::load_raw(p + (int64_t)(row0 + r) * S + c);
      }
    }
  float dot[RPG];
#pragma unroll
  for (int r = 0; r < RPG; r++) {
    float d = 0.f;
#pragma unroll
    for (int i = 0; i < NV; i++) {
      if ((gl + LPR * i) * VN < S && row0 + r < rows) {
        float a[VN], b[VN];
        VecT<T>::unpack(ra[r][i], a);
        VecT<T>::unpack(rb[r][i], b);
#pragma unroll
        for (int e = 0; e < VN; e++) d += a[e] * b[e];
      }
    }
    dot[r] = d;
  }
#pragma unroll
  for (int r = 0; r < RPG; r++)
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) dot[r] += __shfl_xor_sync(gmask, dot[r], o);
#pragma unroll
  for (int r = 0; r < RPG; r++)
#pragma unroll
    for (int i = 0; i < NV; i++) {
      const int c = (gl + LPR * i) * VN;
      if (c < S && row0 + r < rows) {
        float a[VN], b[VN], o[VN];
        VecT<T>::unpack(ra[r][i], a);
        VecT<T>::unpack(rb[r][i], b);
#pragma unroll
        for (int e = 0; e < VN; e++) o[e] = b[e] * (a[e] - dot[r]) * scale;
        VecT<T>::store(dp + (int64_t)(row0 + r) * S + c, o);
      }
    }
}

// ---------------------------------------------------------------------------------------
// MLM slots: validity, source rows, labels, count; sequence-length check.
// ---------------------------------------------------------------------------------------
__global__ void slots_prepare_kernel(const int* __restrict__ positions,
                                     const int* __restrict__ labels,
                                     const int* __restrict__ seq_lens, int B, int S, int P, int V,
                                     int* __restrict__ rowsrc, int* __restrict__ rowlabel,
                                     int* __restrict__ n_valid, float* __restrict__ inv_n,
                                     int* __restrict__ status) {
  __shared__ int cnt;
  if (threadIdx.x == 0) cnt = 0;
  __syncthreads();
  int local = 0, bad = 0;
  for (int r = threadIdx.x; r < B * P; r += blockDim.x) {
    const int b = r / P;
    const int pos = positions[r];
    const int lab = labels ? labels[r] : 0;
    bool ok = pos >= 0 && lab >= 0;
    // a position at or beyond the sequence's length would read a padded row, whose content is unspecified
    int len = S;
    if (seq_lens != nullptr) len = min(max(seq_lens[b], 1), S);
    if (pos >= len) { bad |= ST_BAD_POSITION; ok = false; }
    if (lab >= V) { bad |= ST_BAD_LABEL; ok = false; }
    rowsrc[r] = ok ? b * S + pos : -1;
    rowlabel[r] = ok ? lab : -1;
    local += ok ? 1 : 0;
  }
  if (seq_lens != nullptr) {
    for (int b = threadIdx.x; b < B; b += blockDim.x)
      if (seq_lens[b] < 1 || seq_lens[b] > S) bad |= ST_BAD_LENGTH;
  }
  if (local) atomicAdd(&cnt, local);
  if (bad) atomicOr(status, bad);
  __syncthreads();
  if (threadIdx.x == 0) {
    *n_valid = cnt;
    *inv_n = cnt > 0 ? 1.0f / (float)cnt : 0.f;
  }
}

// hm[r,:] = x[rowsrc[r],:], or zero for an empty slot
template <typename T>
__global__ void gather_rows_kernel(const T* __restrict__ x, const int* __restrict__ rowsrc,
                                   T* __restrict__ out, int R, int H) {
  constexpr int VN = VecT<T>::N;
  const int r = blockIdx.x;
  const int src = rowsrc[r];
  for (int c = threadIdx.x * VN; c < H; c += blockDim.x * VN) {
    float t[VN];
    if (src >= 0) {
      VecT<T>::load(x + (int64_t)src * H + c, t);
    } else {
#pragma unroll
      for (int e = 0; e < VN; e++) t[e] = 0.f;
    }
    VecT<T>::store(out + (int64_t)r * H + c, t);
  }
}

// dx[rowsrc[r],:] += d[r,:]; one block per sequence walks its slots in order, so repeated
// positions add up without atomics.  dx must be zeroed beforehand.
template <typename T>
__global__ void scatter_rows_kernel(const T* __restrict__ d, const int* __restrict__ rowsrc,
                                    T* __restrict__ dx, int P, int H) {
  constexpr int VN = VecT<T>::N;
  const int b = blockIdx.x;
  for (int c = threadIdx.x * VN; c < H; c += blockDim.x * VN) {
    for (int j = 0; j < P; j++) {
      const int r = b * P + j;
      const int src = rowsrc[r];
      if (src < 0) continue;
      float a[VN], t[VN];
      VecT<T>::load(dx + (int64_t)src * H + c, a);
      VecT<T>::load(d + (int64_t)r * H + c, t);
#pragma unroll
      for (int e = 0; e < VN; e++) a[e] += t[e];
      VecT<T>::store(dx + (int64_t)src * H + c, a);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Softmax cross-entropy over the vocabulary, one block per slot.  nll = logsumexp - logit[label];
// dlogits = (softmax - onehot) * inv_n.  Empty slots get nll 0 and a zero gradient row.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
cross_entropy_kernel(const float* __restrict__ logits, int64_t ldl, const int* __restrict__ rowlabel,
                     const float* __restrict__ inv_n, T* __restrict__ dlogits, int64_t ldd,
                     float* __restrict__ nll, int V) {
  constexpr int VN = VecT<T>::N;
  __shared__ float sm[8], ss[8];
  __shared__ float s_lse;
  const int r = blockIdx.x;
  const int label = rowlabel[r];
  const float* lr = logits + (int64_t)r * ldl;
  T* dr = dlogits ? dlogits + (int64_t)r * ldd : nullptr;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (label < 0) {
    if (threadIdx.x == 0) nll[r] = 0.f;
    if (dr != nullptr) {
      float zero[VN];
#pragma unroll
      for (int e = 0; e < VN; e++) zero[e] = 0.f;
      for (int64_t c = (int64_t)threadIdx.x * VN; c < ldd; c += 256 * VN) VecT<T>::store(dr + c, zero);
    }
    return;
  }
  // pass 1: running maximum and rescaled sum
  float m = -INFINITY, s = 0.f;
  for (int c = threadIdx.x * 4; c < V; c += 256 * 4) {
    float4 v = *reinterpret_cast<const float4*>(lr + c);
    float t[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; e++) {
      if (c + e < V) {
        const float nm = fmaxf(m, t[e]);
        s = s * expf(m - nm) + expf(t[e] - nm);
        m = nm;
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, o);
    const float os = __shfl_xor_sync(0xffffffffu, s, o);
    const float nm = fmaxf(m, om);
    s = (m == -INFINITY ? 0.f : s * expf(m - nm)) + (om == -INFINITY ? 0.f : os * expf(om - nm));
    m = nm;
  }
  if (lane == 0) { sm[warp] = m; ss[warp] = s; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float M = sm[0], Sx = ss[0];
    for (int w = 1; w < 8; w++) {
      const float nm = fmaxf(M, sm[w]);
      Sx = (M == -INFINITY ? 0.f : Sx * expf(M - nm)) + (sm[w] == -INFINITY ? 0.f : ss[w] * expf(sm[w] - nm));
      M = nm;
    }
    const float lse = M + logf(Sx);
    s_lse = lse;
    nll[r] = lse - lr[label];
  }
  __syncthreads();
  if (dr == nullptr) return;
  const float lse = s_lse;
  const float inv = *inv_n;
  for (int64_t c = (int64_t)threadIdx.x * VN; c < ldd; c += 256 * VN) {
    float o[VN];
#pragma unroll
    for (int h = 0; h < VN / 4; h++) {
      float4 v = *reinterpret_cast<const float4*>(lr + c + 4 * h);
      o[4 * h] = v.x; o[4 * h + 1] = v.y; o[4 * h + 2] = v.z; o[4 * h + 3] = v.w;
    }
#pragma unroll
    for (int e = 0; e < VN; e++) {
      const int64_t j = c + e;
      o[e] = j < V ? (expf(o[e] - lse) - (j == label ? 1.f : 0.f)) * inv : 0.f;
    }
    VecT<T>::store(dr + c, o);
  }
}

// The same for rows of up to 32768 logits, with the whole row held in the registers of a
// 1024-thread block: the logits are read from HBM exactly once (eight independent 16-byte loads
// per thread keep 128 KB in flight per SM) and one exponential per element is evaluated.
constexpr int CE_REG_V4 = 8;  // float4 per thread

template <typename T>
__global__ void __launch_bounds__(1024)
cross_entropy_regs_kernel(const float* __restrict__ logits, int64_t ldl, const int* __restrict__ rowlabel,
                          const float* __restrict__ inv_n, T* __restrict__ dlogits, int64_t ldd,
                          float* __restrict__ nll, int V) {
  __shared__ float red[32];
  __shared__ float bcast;
  const int r = blockIdx.x, tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int label = rowlabel[r];
  const float* lr = logits + (int64_t)r * ldl;
  T* dr = dlogits ? dlogits + (int64_t)r * ldd : nullptr;
  if (label < 0) {
    if (tid == 0) nll[r] = 0.f;
    if (dr != nullptr)
      for (int64_t c = (int64_t)tid * 4; c < ldd; c += 1024 * 4) {
#pragma unroll
        for (int e = 0; e < 4; e++) dr[c + e] = from_f<T>(0.f);
      }
    return;
  }
  float x[CE_REG_V4][4];
  float m = -INFINITY;
#pragma unroll
  for (int i = 0; i < CE_REG_V4; i++) {
    const int c = (tid + i * 1024) * 4;
    float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (c < ldl) v = *reinterpret_cast<const float4*>(lr + c);
    x[i][0] = c + 0 < V ? v.x : -INFINITY;
    x[i][1] = c + 1 < V ? v.y : -INFINITY;
    x[i][2] = c + 2 < V ? v.z : -INFINITY;
    x[i][3] = c + 3 < V ? v.w : -INFINITY;
  }
#pragma unroll
  for (int i = 0; i < CE_REG_V4; i++)
#pragma unroll
    for (int e = 0; e < 4; e++) m = fmaxf(m, x[i][e]);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (warp == 0) {
    float t = warp_max(red[lane]);
    if (lane == 0) bcast = t;
  }
  __syncthreads();
  m = bcast;
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < CE_REG_V4; i++)
#pragma unroll
    for (int e = 0; e < 4; e++) {
      x[i][e] = expf(x[i][e] - m);  // exp(-inf) = 0 for the padding
      s += x[i][e];
    }
  s = warp_sum(s);
  __syncthreads();  // bcast and red are reused
  if (lane == 0) red[warp] = s;
  __syncthreads();
  if (warp == 0) {
    float t = warp_sum(red[lane]);
    if (lane == 0) {
      bcast = t;
      nll[r] = m + logf(t) - lr[label];
    }
  }
  __syncthreads();
  if (dr == nullptr) return;
  const float scale = (*inv_n) / bcast;
  const float inv = *inv_n;
#pragma unroll
  for (int i = 0; i < CE_REG_V4; i++) {
    const int c = (tid + i * 1024) * 4;
    if (c < ldd) {
      T o[4];
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const float g = c + e < V ? x[i][e] * scale - (c + e == label ? inv : 0.f) : 0.f;
        o[e] = from_f<T>(g);
      }
      if (sizeof(T) == 4) *reinterpret_cast<float4*>(dr + c) = *reinterpret_cast<const float4*>(o);
      else *reinterpret_cast<uint2*>(dr + c) = *reinterpret_cast<const uint2*>(o);
    }
  }
}

__global__ void loss_reduce_kernel(const float* __restrict__ nll, int R,
                                   const float* __restrict__ inv_n, float* __restrict__ loss) {
  __shared__ float part[32];
  float s = 0.f;
  for (int r = threadIdx.x; r < R; r += blockDim.x) s += nll[r];
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); w++) t += part[w];
    *loss = t * (*inv_n);
  }
}

__global__ void override_inv_n_kernel(const int* __restrict__ total_valid, float* __restrict__ inv_n) {
  const int n = *total_valid;
  *inv_n = n > 0 ? 1.0f / (float)n : 0.f;
}

// ---------------------------------------------------------------------------------------
// Column sums (bias gradients): out[n] += sum_rows x[row, n].
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
colsum_kernel(const T* __restrict__ x, int64_t ld, int rows, int N, int rows_per_block,
              float* __restrict__ out) {
  constexpr int VN = VecT<T>::N;
  __shared__ float red[8][32 * VN];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int c = (blockIdx.x * 32 + tx) * VN;
  const int r0 = blockIdx.y * rows_per_block;
  const int r1 = min(rows, r0 + rows_per_block);
  float acc[VN];
#pragma unroll
  for (int e = 0; e < VN; e++) acc[e] = 0.f;
  if (c < N) {
    for (int r = r0 + ty; r < r1; r += 8) {
      float t[VN];
      VecT<T>::load(x + (int64_t)r * ld + c, t);
#pragma unroll
      for (int e = 0; e < VN; e++) acc[e] += t[e];
    }
  }
#pragma unroll
  for (int e = 0; e < VN; e++) red[ty][tx * VN + e] = acc[e];
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * VN; i += 256) {
    const int col = blockIdx.x * 32 * VN + i;
    if (col < N) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; w++) s += red[w][i];
      atomicAdd(out + col, s);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Embedding gradient: dword[token[t], :] += dz[t, :], dpos[t % S, :] += dz[t, :].
// Without atomics on hot rows, and with the same bits on every run: the rows are
// grouped by token id with a counting sort whose order is fixed (block of 256 rows, then position
// inside the block), one thread block per token id then adds its rows in that order, and the
// position table gets a plain sum over the batch.
//   counts [nb][V]  (nb = ceil(T / 256)): rows of block b with token v, turned into the exclusive
//                   prefix over blocks;  total[V], start[V];  order[T]: rows sorted by (token, row).
// ---------------------------------------------------------------------------------------
constexpr int ES_BLOCK = 256;   // rows per sort block
constexpr int ES_TOKENS = 8;    // token ids per block of the reduction kernel
constexpr int ES_CHUNK = 64;    // rows one block adds for a frequent token
constexpr int ES_MAX_SLOTS = 2048;  // chunk slots: at most T / ES_CHUNK + (tokens above ES_CHUNK) <= 2 T / ES_CHUNK

// counts is laid out [V][nb] so that a token's per-block counts are contiguous
__global__ void __launch_bounds__(ES_BLOCK)
embed_sort_count_kernel(const int* __restrict__ tokens, int T, int V, int nb, int* __restrict__ counts,
                        int* __restrict__ rank) {
  __shared__ int tk[ES_BLOCK];
  const int t = blockIdx.x * ES_BLOCK + threadIdx.x;
  int tok = t < T ? tokens[t] : -1;
  if (t < T && (tok < 0 || tok >= V)) tok = 0;
  tk[threadIdx.x] = tok;
  __syncthreads();
  if (t >= T) return;
  int r = 0;
  for (int j = 0; j < (int)threadIdx.x; j++) r += tk[j] == tok ? 1 : 0;  // rows of this block before me with my token
  rank[t] = r;
  atomicAdd(counts + (int64_t)tok * nb + blockIdx.x, 1);  // integer: the result does not depend on the order
}

// Per token: exclusive prefix of its counts over the row blocks and its total; per block of 256
// tokens: exclusive scan of the totals (local start) and the block's sum.
__global__ void __launch_bounds__(256)
embed_sort_prefix_kernel(int* __restrict__ counts, int nb, int V, int* __restrict__ total,
                         int* __restrict__ start_local, int* __restrict__ blocksum, int* __restrict__ hot) {
  __shared__ int part[256];
  const int v = blockIdx.x * 256 + threadIdx.x;
  int run = 0;
  if (v < V) {
    int* row = counts + (int64_t)v * nb;
    for (int b = 0; b < nb; b++) {
      const int c = row[b];
      row[b] = run;
      run += c;
    }
    total[v] = run;
    // A token with more than ES_CHUNK rows is summed in chunks of ES_CHUNK rows by several blocks.
    // hot[0] = chunks handed out, hot[1] = such tokens; then per chunk slot (token, chunk index) and
    // per hot token (token, first slot).  Which slot a token gets is arbitrary and changes nothing:
    // the rows of a chunk and the chunks of a token are always added in the same order.
    if (run > ES_CHUNK) {
      const int nch = (run + ES_CHUNK - 1) / ES_CHUNK;
      const int base = atomicAdd(hot, nch);
      const int h = atomicAdd(hot + 1, 1);
      hot[2 + 2 * ES_MAX_SLOTS + 2 * h] = v;
      hot[2 + 2 * ES_MAX_SLOTS + 2 * h + 1] = base;
      for (int k = 0; k < nch; k++) {
        hot[2 + 2 * (base + k)] = v;
        hot[2 + 2 * (base + k) + 1] = k;
      }
    }
  }
  part[threadIdx.x] = run;
  __syncthreads();
  for (int o = 1; o < 256; o <<= 1) {
    const int add = threadIdx.x >= o ? part[threadIdx.x - o] : 0;
    __syncthreads();
    part[threadIdx.x] += add;
    __syncthreads();
  }
  if (v < V) start_local[v] = part[threadIdx.x] - run;
  if (threadIdx.x == 255) blocksum[blockIdx.x] = part[255];
}

// exclusive scan of the block sums (at most 1024 blocks of 256 tokens) in place
__global__ void __launch_bounds__(1024)
embed_sort_scan_kernel(int* __restrict__ blocksum, int n) {
  __shared__ int part[1024];
  const int mine = threadIdx.x < n ? blocksum[threadIdx.x] : 0;
  part[threadIdx.x] = mine;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {
    const int add = threadIdx.x >= o ? part[threadIdx.x - o] : 0;
    __syncthreads();
    part[threadIdx.x] += add;
    __syncthreads();
  }
  if (threadIdx.x < n) blocksum[threadIdx.x] = part[threadIdx.x] - mine;
}

__global__ void embed_sort_place_kernel(const int* __restrict__ tokens, int T, int V, int nb,
                                        const int* __restrict__ counts, const int* __restrict__ rank,
                                        const int* __restrict__ start_local, const int* __restrict__ blockoff,
                                        int* __restrict__ order) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  int tok = tokens[t];
  if (tok < 0 || tok >= V) tok = 0;
  order[blockoff[tok >> 8] + start_local[tok] + counts[(int64_t)tok * nb + t / ES_BLOCK] + rank[t]] = t;
}

// Adds the rows order[first .. first + n) of dz in that order: H / VN column threads times G row
// groups; group g takes the rows g, g + G, ... with eight loads in flight and the groups' partial sums
// meet in shared memory in a fixed order.  The result is added to dst[0 .. H) (add) or stored there.
template <typename T, int NT>
__device__ __forceinline__ void es_sum_rows(const T* __restrict__ dz, const int* __restrict__ seg, int n, int H,
                                            float* es_part, float* __restrict__ dst, bool add) {
  constexpr int VN = VecT<T>::N;
  const int colthreads = H / VN;
  const int G = NT / colthreads;
  const int ct = threadIdx.x % colthreads, g = threadIdx.x / colthreads;
  float acc[VN];
#pragma unroll
  for (int e = 0; e < VN; e++) acc[e] = 0.f;
  if (g < G) {
    int i = g;
    for (; i + 7 * G < n; i += 8 * G) {
      float a[8][VN];
#pragma unroll
      for (int u = 0; u < 8; u++) VecT<T>::load(dz + (int64_t)seg[i + u * G] * H + ct * VN, a[u]);
#pragma unroll
      for (int u = 0; u < 8; u++)
#pragma unroll
        for (int e = 0; e < VN; e++) acc[e] += a[u][e];
    }
    for (; i < n; i += G) {
      float a[VN];
      VecT<T>::load(dz + (int64_t)seg[i] * H + ct * VN, a);
#pragma unroll
      for (int e = 0; e < VN; e++) acc[e] += a[e];
    }
#pragma unroll
    for (int e = 0; e < VN; e++) es_part[g * H + ct * VN + e] = acc[e];
  }
  __syncthreads();
  const int used = min(G, n);  // groups beyond the segment's length hold zeros: skip them
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    float s = 0.f;
    for (int k = 0; k < used; k++) s += es_part[k * H + c];
    dst[c] = add ? dst[c] + s : s;
  }
  __syncthreads();
}

// dword[v, :] += sum of the dz rows of token v, for the tokens with at most ES_CHUNK rows.  Token ids
// are dealt out with a stride of the grid size: frequent ids are neighbours (ids follow frequency rank
// in natural text and in the synthetic batches) and must not share a block.
template <typename T>
__global__ void __launch_bounds__(256)
embed_word_grad_kernel(const T* __restrict__ dz, const int* __restrict__ order, const int* __restrict__ start_local,
                       const int* __restrict__ blockoff, const int* __restrict__ total,
                       float* __restrict__ dword, int H, int V) {
  extern __shared__ float es_part[];  // [G][H]
  for (int v = blockIdx.x; v < V; v += gridDim.x) {
    const int n = total[v];
    if (n == 0 || n > ES_CHUNK) continue;  // the same for every thread of the block
    es_sum_rows<T, 256>(dz, order + blockoff[v >> 8] + start_local[v], n, H, es_part, dword + (int64_t)v * H, true);
  }
}

// frequent tokens, first half: block = chunk slot, partial[slot, :] = sum of the chunk's rows
template <typename T>
__global__ void __launch_bounds__(1024)
embed_word_hot_chunk_kernel(const T* __restrict__ dz, const int* __restrict__ order,
                            const int* __restrict__ start_local, const int* __restrict__ blockoff,
                            const int* __restrict__ total, const int* __restrict__ hot,
                            float* __restrict__ partial, int H) {
  extern __shared__ float es_part[];
  const int slot = blockIdx.x;
  if (slot >= min(hot[0], ES_MAX_SLOTS)) return;
  const int v = hot[2 + 2 * slot], k = hot[2 + 2 * slot + 1];
  const int n = min(ES_CHUNK, total[v] - k * ES_CHUNK);
  es_sum_rows<T, 1024>(dz, order + blockoff[v >> 8] + start_local[v] + k * ES_CHUNK, n, H, es_part,
                 partial + (int64_t)slot * H, false);
}

// second half: block = frequent token, dword[v, :] += its chunks' partial sums in chunk order
__global__ void embed_word_hot_sum_kernel(const int* __restrict__ total, const int* __restrict__ hot,
                                          const float* __restrict__ partial, float* __restrict__ dword, int H) {
  const int h = blockIdx.x;
  if (h >= min(hot[1], ES_MAX_SLOTS / 2)) return;
  const int v = hot[2 + 2 * ES_MAX_SLOTS + 2 * h], base = hot[2 + 2 * ES_MAX_SLOTS + 2 * h + 1];
  const int nch = (total[v] + ES_CHUNK - 1) / ES_CHUNK;
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    float s = 0.f;
    for (int k = 0; k < nch; k++) s += partial[(int64_t)(base + k) * H + c];
    dword[(int64_t)v * H + c] += s;
  }
}

// dpos[s, :] += sum over the batch of dz[b * S + s, :].  Block (s, column slab of 32 vectors): 32
// column threads times 8 row groups over the batch, combined in shared memory in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256)
embed_pos_grad_kernel(const T* __restrict__ dz, float* __restrict__ dpos, int B, int S, int H) {
  constexpr int VN = VecT<T>::N;
  __shared__ float part[8][32 * VN];
  const int s = blockIdx.x;
  const int lane = threadIdx.x & 31, g = threadIdx.x >> 5;
  const int c = (blockIdx.y * 32 + lane) * VN;
  float acc[VN];
#pragma unroll
  for (int e = 0; e < VN; e++) acc[e] = 0.f;
  if (c < H) {
    int b = g;
    for (; b + 24 < B; b += 32) {
      float a[4][VN];
#pragma unroll
      for (int u = 0; u < 4; u++) VecT<T>::load(dz + ((int64_t)(b + 8 * u) * S + s) * H + c, a[u]);
#pragma unroll
      for (int u = 0; u < 4; u++)
#pragma unroll
        for (int e = 0; e < VN; e++) acc[e] += a[u][e];
    }
    for (; b < B; b += 8) {
      float a[VN];
      VecT<T>::load(dz + ((int64_t)b * S + s) * H + c, a);
#pragma unroll
      for (int e = 0; e < VN; e++) acc[e] += a[e];
    }
  }
#pragma unroll
  for (int e = 0; e < VN; e++) part[g][lane * VN + e] = acc[e];
  __syncthreads();
  for (int i = threadIdx.x; i < 32 * VN; i += 256) {
    const int col = blockIdx.y * 32 * VN + i;
    if (col < H) {
      float t = 0.f;
      for (int k = 0; k < 8; k++) t += part[k][i];
      dpos[(int64_t)s * H + col] += t;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Adam with decoupled weight decay over a table of chunks of the trainable slice.
// ---------------------------------------------------------------------------------------
// Advances the step count kept in device memory and forms the bias corrections 1 / (1 - beta^t)
// there, so that a captured step (CUDA graph) replays with the right values.
__global__ void adam_tick_kernel(int* __restrict__ t, float* __restrict__ bc, float beta1, float beta2,
                                 int bias_correction) {
  const int n = *t + 1;
  *t = n;
  bc[0] = bias_correction ? (float)(1.0 / (1.0 - pow((double)beta1, (double)n))) : 1.f;
  bc[1] = bias_correction ? (float)(1.0 / (1.0 - pow((double)beta2, (double)n))) : 1.f;
}

__global__ void __launch_bounds__(256)
adam_kernel(const AdamChunk* __restrict__ chunks, float* __restrict__ w,
            const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
            bf16* __restrict__ wb, AdamHyper h, const float* __restrict__ bc) {
  h.bc1 = bc[0];
  h.bc2 = bc[1];
  const AdamChunk ch = chunks[blockIdx.x];
  const float decay = h.weight_decay * ch.decay;
  for (int i = threadIdx.x * 4; i < ch.count; i += 256 * 4) {
    const int64_t o = ch.offset + i;
    float4 wv = *reinterpret_cast<float4*>(w + o);
    const float4 gv = *reinterpret_cast<const float4*>(g + o);
    float4 mv = *reinterpret_cast<float4*>(m + o);
    float4 vv = *reinterpret_cast<float4*>(v + o);
    float* wp = &wv.x; const float* gp = &gv.x; float* mp = &mv.x; float* vp = &vv.x;
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float mm = h.beta1 * mp[e] + h.omb1 * gp[e];
      const float vn = h.beta2 * vp[e] + h.omb2 * gp[e] * gp[e];
      const float mh = mm * h.bc1, vh = vn * h.bc2;
      wp[e] = wp[e] - h.lr * (mh / (sqrtf(vh) + h.eps) + decay * wp[e]);
      mp[e] = mm;
      vp[e] = vn;
    }
    *reinterpret_cast<float4*>(w + o) = wv;
    *reinterpret_cast<float4*>(m + o) = mv;
    *reinterpret_cast<float4*>(v + o) = vv;
    if (wb != nullptr) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(wv.x, wv.y), hi = __floats2bfloat162_rn(wv.z, wv.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(wb + o) = pk;
    }
  }
}

// ---------------------------------------------------------------------------------------
// Next-sentence-prediction head (the second BERT objective): per sequence b, on the pooled first
// token, logits = Wn pooled + bn (two classes), nll = logsumexp - logit[label], mean over the
// sequences with label >= 0.  One block per sequence; it also forms the gradients of Wn and bn
// (atomics into the zeroed arena) and, fused with the tanh derivative of the pooler, the gradient
// at the pooler's pre-activation: dup = (dlogit . Wn) * (1 - pooled^2).
// ---------------------------------------------------------------------------------------
__global__ void nsp_prepare_kernel(const int* __restrict__ labels, int B, int S, int* __restrict__ rowsrc,
                                   float* __restrict__ inv_n, const int* __restrict__ total_valid) {
  __shared__ int cnt;
  if (threadIdx.x == 0) cnt = 0;
  __syncthreads();
  int local = 0;
  for (int b = threadIdx.x; b < B; b += blockDim.x) {
    rowsrc[b] = b * S;  // the first token of sequence b
    local += (labels != nullptr && labels[b] >= 0 && labels[b] <= 1) ? 1 : 0;
  }
  if (local) atomicAdd(&cnt, local);
  __syncthreads();
  if (threadIdx.x == 0) {
    const int n = total_valid ? *total_valid : cnt;
    *inv_n = n > 0 ? 1.0f / (float)n : 0.f;
  }
}

template <typename T>
__global__ void __launch_bounds__(128)
nsp_head_kernel(const T* __restrict__ pooled, const float* __restrict__ wn, const float* __restrict__ bn,
                const int* __restrict__ labels, const float* __restrict__ inv_n, T* __restrict__ dup,
                float* __restrict__ dwn, float* __restrict__ dbn, float* __restrict__ loss, int H) {
  const int b = blockIdx.x;
  const T* pr = pooled + (int64_t)b * H;
  float s0 = 0.f, s1 = 0.f;
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    const float p = to_f<T>(pr[c]);
    s0 += p * wn[c];
    s1 += p * wn[H + c];
  }
  __shared__ float red[2][4];
  s0 = warp_sum(s0);
  s1 = warp_sum(s1);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = s0; red[1][threadIdx.x >> 5] = s1; }
  __syncthreads();
  const float l0 = red[0][0] + red[0][1] + red[0][2] + red[0][3] + bn[0];
  const float l1 = red[1][0] + red[1][1] + red[1][2] + red[1][3] + bn[1];
  const int lab = labels ? labels[b] : -1;
  const bool ok = lab == 0 || lab == 1;
  const float mx = fmaxf(l0, l1);
  const float e0 = expf(l0 - mx), e1 = expf(l1 - mx);
  const float lse = mx + logf(e0 + e1);
  const float scale = ok ? *inv_n : 0.f;
  const float d0 = (e0 / (e0 + e1) - (lab == 0 ? 1.f : 0.f)) * scale;
  const float d1 = (e1 / (e0 + e1) - (lab == 1 ? 1.f : 0.f)) * scale;
  if (threadIdx.x == 0 && ok) {
    atomicAdd(loss, (lse - (lab == 0 ? l0 : l1)) * scale);
    atomicAdd(dbn, d0);
    atomicAdd(dbn + 1, d1);
  }
  for (int c = threadIdx.x; c < H; c += blockDim.x) {
    const float p = to_f<T>(pr[c]);
    dup[(int64_t)b * H + c] = from_f<T>((d0 * wn[c] + d1 * wn[H + c]) * (1.f - p * p));
    if (ok) {
      atomicAdd(dwn + c, d0 * p);
      atomicAdd(dwn + H + c, d1 * p);
    }
  }
}

// y = tanh(x), elementwise
template <typename T>
__global__ void tanh_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t n) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    y[i] = from_f<T>(tanhf(to_f<T>(x[i])));
}

// Gradient of the two-row segment table: dtype[seg[t], c] += dz[t, c].  A thread owns a column of a
// block of rows and keeps one sum per segment, so the table sees two atomics per thread.
template <typename T>
__global__ void __launch_bounds__(128)
type_grad_kernel(const T* __restrict__ dz, const int* __restrict__ segments, float* __restrict__ dtype,
                 int rows, int H, int rows_per_block) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= H) return;
  const int r0 = blockIdx.y * rows_per_block, r1 = min(rows, r0 + rows_per_block);
  float a0 = 0.f, a1 = 0.f;
  for (int r = r0; r < r1; r++) {
    const float v = to_f<T>(dz[(int64_t)r * H + c]);
    const int sg = segments ? segments[r] : 0;
    if (sg == 1) a1 += v; else a0 += v;
  }
  atomicAdd(dtype + c, a0);
  atomicAdd(dtype + H + c, a1);
}

// LAMB, first kernel: new moments, and the per-tensor sums of w^2 and r^2
__global__ void __launch_bounds__(256)
lamb_moments_kernel(const AdamChunk* __restrict__ chunks, const float* __restrict__ w,
                    const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v, AdamHyper h,
                    const float* __restrict__ bc, float* __restrict__ norms) {
  h.bc1 = bc[0];
  h.bc2 = bc[1];
  const AdamChunk ch = chunks[blockIdx.x];
  const float decay = h.weight_decay * ch.decay;
  float sw = 0.f, sr = 0.f;
  for (int i = threadIdx.x * 4; i < ch.count; i += 256 * 4) {
    const int64_t o = ch.offset + i;
    const float4 wv = *reinterpret_cast<const float4*>(w + o);
    const float4 gv = *reinterpret_cast<const float4*>(g + o);
    float4 mv = *reinterpret_cast<float4*>(m + o);
    float4 vv = *reinterpret_cast<float4*>(v + o);
    const float* wp = &wv.x; const float* gp = &gv.x; float* mp = &mv.x; float* vp = &vv.x;
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float mm = h.beta1 * mp[e] + h.omb1 * gp[e];
      const float vn = h.beta2 * vp[e] + h.omb2 * gp[e] * gp[e];
      const float r = (mm * h.bc1) / (sqrtf(vn * h.bc2) + h.eps) + decay * wp[e];
      sw += wp[e] * wp[e];
      sr += r * r;
      mp[e] = mm;
      vp[e] = vn;
    }
    *reinterpret_cast<float4*>(m + o) = mv;
    *reinterpret_cast<float4*>(v + o) = vv;
  }
  __shared__ float red[2][8];
  sw = warp_sum(sw);
  sr = warp_sum(sr);
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = sw; red[1][threadIdx.x >> 5] = sr; }
  __syncthreads();
  if (threadIdx.x < 32) {
    float a = threadIdx.x < 8 ? red[0][threadIdx.x] : 0.f, b = threadIdx.x < 8 ? red[1][threadIdx.x] : 0.f;
    a = warp_sum(a);
    b = warp_sum(b);
    if (threadIdx.x == 0) {
      atomicAdd(norms + 2 * ch.tensor, a);
      atomicAdd(norms + 2 * ch.tensor + 1, b);
    }
  }
}

// LAMB, second kernel: the step, scaled by the tensor's trust ratio
__global__ void __launch_bounds__(256)
lamb_apply_kernel(const AdamChunk* __restrict__ chunks, float* __restrict__ w, const float* __restrict__ m,
                  const float* __restrict__ v, bf16* __restrict__ wb, AdamHyper h,
                  const float* __restrict__ bc, const float* __restrict__ norms) {
  h.bc1 = bc[0];
  h.bc2 = bc[1];
  const AdamChunk ch = chunks[blockIdx.x];
  const float decay = h.weight_decay * ch.decay;
  const float wn = sqrtf(norms[2 * ch.tensor]), rn = sqrtf(norms[2 * ch.tensor + 1]);
  const float step = h.lr * ((wn > 0.f && rn > 0.f) ? wn / rn : 1.f);
  for (int i = threadIdx.x * 4; i < ch.count; i += 256 * 4) {
    const int64_t o = ch.offset + i;
    float4 wv = *reinterpret_cast<float4*>(w + o);
    const float4 mv = *reinterpret_cast<const float4*>(m + o);
    const float4 vv = *reinterpret_cast<const float4*>(v + o);
    float* wp = &wv.x; const float* mp = &mv.x; const float* vp = &vv.x;
#pragma unroll
    for (int e = 0; e < 4; e++) {
      const float r = (mp[e] * h.bc1) / (sqrtf(vp[e] * h.bc2) + h.eps) + decay * wp[e];
      wp[e] = wp[e] - step * r;
    }
    *reinterpret_cast<float4*>(w + o) = wv;
    if (wb != nullptr) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(wv.x, wv.y), hi = __floats2bfloat162_rn(wv.z, wv.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(wb + o) = pk;
    }
  }
}

// d[i] *= gelu'(u[i]) (MLM transform backward)
template <typename T>
__global__ void dgelu_kernel(T* __restrict__ d, const T* __restrict__ u, int64_t n) {
  constexpr int VN = VecT<T>::N;
  for (int64_t i = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) * VN; i < n;
       i += (int64_t)gridDim.x * blockDim.x * VN) {
    float a[VN], b[VN];
    VecT<T>::load(d + i, a);
    VecT<T>::load(u + i, b);
#pragma unroll
    for (int e = 0; e < VN; e++) a[e] *= gelu_grad_f(b[e]);
    VecT<T>::store(d + i, a);
  }
}

__global__ void f32_to_bf16_kernel(const float* __restrict__ src, bf16* __restrict__ dst, int64_t n) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}

// ---------------------------------------------------------------------------------------
// host launchers
// ---------------------------------------------------------------------------------------
#define DISPATCH_T(bf, ...)                 \
  do {                                      \
    if (bf) { using T = bf16; __VA_ARGS__; } \
    else { using T = float; __VA_ARGS__; }   \
  } while (0)

void launch_ln_fwd(bool bf, const void* z, const float* gamma, const float* beta, void* y,
                   float* stats, int rows, int H, float eps, cudaStream_t st) {
  if (rows <= 0) return;
  const int vn = bf ? 8 : 4;
  const int nv = (H + 32 * vn - 1) / (32 * vn);
#define LN_FWD(NV, ROWS)                                                                             \
  DISPATCH_T(bf, (ln_fwd_kernel<T, NV, ROWS><<<div_up(rows, 4 * ROWS), 128, 0, st>>>(                  \
                     (const T*)z, gamma, beta, (T*)y, stats, rows, H, eps)))
  if (nv <= 1) LN_FWD(1, 4);
  else if (nv <= 2) LN_FWD(2, 2);
  else if (nv <= 3) LN_FWD(3, 2);
  else if (nv <= 4) LN_FWD(4, 2);
  else if (nv <= 6) LN_FWD(6, 2);
  else LN_FWD(8, 2);
#undef LN_FWD
}

void launch_embed_ln(bool bf, const int* tokens, const int* segments, const void* word, const void* pos,
                     const void* type, const float* gamma, const float* beta, void* y, void* zstash,
                     float* stats, int rows, int S, int H, int V, float eps, int* status, cudaStream_t st) {
  if (rows <= 0) return;
  DISPATCH_T(bf, (embed_ln_kernel<T><<<div_up(rows, 8), 256, 0, st>>>(
                     tokens, segments, (const T*)word, (const T*)pos, (const T*)type, gamma, beta, (T*)y,
                     (T*)zstash, stats, rows, S, H, V, eps, status)));
}

void launch_ln_bwd(bool bf, const void* dy, const void* z, const float* stats, const float* gamma,
                   void* dz, float* dgamma, float* dbeta, float* dbias, int rows, int H, cudaStream_t st) {
  if (rows <= 0) return;
  // warps per row: one 16-byte vector per lane; row groups fill the block up to 12-16 warps
  const int vn = bf ? 8 : 4;
  const int nslice = (H + 32 * vn - 1) / (32 * vn);
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  // one block per SM walks the rows: the column sums end in one atomic per column and block
#define LN_BWD(NS, RG)                                                                                   \
  DISPATCH_T(bf, (ln_bwd_kernel<T, NS, RG, 4><<<std::min(div_up(rows, RG * 4), sms), NS * RG * 32, 0, st>>>( \
                     (const T*)dy, (const T*)z, stats, gamma, (T*)dz, dgamma, dbeta, dbias, rows, H)))
  if (nslice <= 1) LN_BWD(1, 8);
  else if (nslice <= 2) LN_BWD(2, 6);
  else if (nslice <= 3) LN_BWD(3, 4);
  else if (nslice <= 4) LN_BWD(4, 3);
  else if (nslice <= 6) LN_BWD(6, 2);
  else LN_BWD(8, 2);
#undef LN_BWD
}

void launch_softmax_fwd(bool bf, const void* sc, void* p, const int* seq_lens, int rows, int S,
                        int rows_per_seq, float scale, cudaStream_t st) {
  if (rows <= 0) return;
  const int vn = bf ? 8 : 4;
  const int nvec = (S + vn - 1) / vn;  // 16-byte vectors per row
#define SM_FWD(LPR, NV)                                                                        \
  DISPATCH_T(bf, (softmax_fwd_kernel<T, LPR, NV><<<div_up(rows, 8 * (32 / LPR) * 2), 256, 0, st>>>( \
                     (const T*)sc, (T*)p, seq_lens, rows, S, rows_per_seq, scale)))
  if (nvec <= 16) SM_FWD(16, 1);
  else if (nvec <= 32) SM_FWD(32, 1);
  else if (nvec <= 64) SM_FWD(32, 2);
  else SM_FWD(32, 4);
#undef SM_FWD
}

void launch_softmax_bwd(bool bf, void* dp, const void* p, int rows, int S, float scale,
                        cudaStream_t st) {
  if (rows <= 0) return;
  const int vn = bf ? 8 : 4;
  const int nvec = (S + vn - 1) / vn;  // 16-byte vectors per row
#define SM_BWD(LPR, NV)                                                                        \
  DISPATCH_T(bf, (softmax_bwd_kernel<T, LPR, NV><<<div_up(rows, 8 * (32 / LPR) * 2), 256, 0, st>>>( \
                     (T*)dp, (const T*)p, rows, S, scale)))
  if (nvec <= 16) SM_BWD(16, 1);
  else if (nvec <= 32) SM_BWD(32, 1);
  else if (nvec <= 64) SM_BWD(32, 2);
  else SM_BWD(32, 4);
#undef SM_BWD
}

void launch_slots_prepare(const int* positions, const int* labels, const int* seq_lens, int B,
                          int S, int P, int V, int* rowsrc, int* rowlabel, int* n_valid,
                          float* inv_n, int* status, cudaStream_t st) {
  slots_prepare_kernel<<<1, 256, 0, st>>>(positions, labels, seq_lens, B, S, P, V, rowsrc, rowlabel,
                                          n_valid, inv_n, status);
}

void launch_gather_rows(bool bf, const void* x, const int* rowsrc, void* out, int R, int H,
                        cudaStream_t st) {
  if (R <= 0) return;
  DISPATCH_T(bf, (gather_rows_kernel<T><<<R, 128, 0, st>>>((const T*)x, rowsrc, (T*)out, R, H)));
}

void launch_scatter_rows(bool bf, const void* d, const int* rowsrc, void* dx, int B, int P, int H,
                         cudaStream_t st) {
  if (B <= 0 || P <= 0) return;
  DISPATCH_T(bf, (scatter_rows_kernel<T><<<B, 128, 0, st>>>((const T*)d, rowsrc, (T*)dx, P, H)));
}

void launch_cross_entropy(bool bf, const float* logits, int64_t ldl, const int* rowlabel,
                          const float* inv_n, void* dlogits, int64_t ldd, float* nll, int R, int V,
                          cudaStream_t st) {
  if (R <= 0) return;
  if (ldl <= CE_REG_V4 * 1024 * 4)
    DISPATCH_T(bf, (cross_entropy_regs_kernel<T><<<R, 1024, 0, st>>>(logits, ldl, rowlabel, inv_n,
                                                                     (T*)dlogits, ldd, nll, V)));
  else
    DISPATCH_T(bf, (cross_entropy_kernel<T><<<R, 256, 0, st>>>(logits, ldl, rowlabel, inv_n,
                                                              (T*)dlogits, ldd, nll, V)));
}

void launch_override_inv_n(const int* total_valid, float* inv_n, cudaStream_t st) {
  override_inv_n_kernel<<<1, 1, 0, st>>>(total_valid, inv_n);
}

void launch_loss_reduce(const float* nll, int R, const float* inv_n, float* loss, cudaStream_t st) {
  loss_reduce_kernel<<<1, 1024, 0, st>>>(nll, R, inv_n, loss);
}

void launch_colsum(bool bf, const void* x, int64_t ld, int rows, int N, float* out,
                   cudaStream_t st) {
  if (rows <= 0 || N <= 0) return;
  const int vn = bf ? 8 : 4;
  const int gx = div_up(N, 32 * vn);
  int gy = std::max(1, std::min(div_up(rows, 64), (148 * 4 + gx - 1) / gx));
  const int rpb = div_up(rows, gy);
  gy = div_up(rows, rpb);
  DISPATCH_T(bf, (colsum_kernel<T><<<dim3(gx, gy), 256, 0, st>>>((const T*)x, ld, rows, N, rpb, out)));
}

void launch_embed_grad_sorted(bool bf, const void* dz, const int* tokens, float* dword, float* dpos, int B, int S,
                              int H, int V, int* counts, int* total, int* start, int* rank, int* order,
                              int* blocksum, int* hot, float* partial, cudaStream_t st) {
  const int T = B * S;
  if (T <= 0) return;
  const int nb = div_up(T, ES_BLOCK), vb = div_up(V, 256);
  cudaMemsetAsync(counts, 0, (size_t)nb * V * sizeof(int), st);
  cudaMemsetAsync(hot, 0, 2 * sizeof(int), st);
  embed_sort_count_kernel<<<nb, ES_BLOCK, 0, st>>>(tokens, T, V, nb, counts, rank);
  embed_sort_prefix_kernel<<<vb, 256, 0, st>>>(counts, nb, V, total, start, blocksum, hot);
  embed_sort_scan_kernel<<<1, 1024, 0, st>>>(blocksum, vb);
  embed_sort_place_kernel<<<div_up(T, 256), 256, 0, st>>>(tokens, T, V, nb, counts, rank, start, blocksum, order);
  const int vn = bf ? 8 : 4;
  const size_t smem = (size_t)(1024 / (H / vn)) * H * sizeof(float), smem_small = (size_t)(256 / (H / vn)) * H * sizeof(float);
  // at most T / ES_CHUNK tokens have more than ES_CHUNK rows, and they have at most 2 T / ES_CHUNK chunks
  const int max_hot = std::min(ES_MAX_SLOTS / 2, T / ES_CHUNK), max_slots = std::min(ES_MAX_SLOTS, 2 * (T / ES_CHUNK));
  DISPATCH_T(bf, (embed_word_grad_kernel<T><<<div_up(V, ES_TOKENS), 256, smem_small, st>>>(
                     (const T*)dz, order, start, blocksum, total, dword, H, V)));
  if (max_slots > 0) {
    DISPATCH_T(bf, (embed_word_hot_chunk_kernel<T><<<max_slots, 1024, smem, st>>>((const T*)dz, order, start, blocksum,
                                                                              total, hot, partial, H)));
    embed_word_hot_sum_kernel<<<max_hot, 256, 0, st>>>(total, hot, partial, dword, H);
  }
  DISPATCH_T(bf, (embed_pos_grad_kernel<T><<<dim3(S, div_up(H, 32 * vn)), 256, 0, st>>>((const T*)dz, dpos, B, S, H)));
}

void launch_adam(const AdamChunk* chunks, int n_chunks, float* w, const float* g, float* m, float* v,
                 void* wb, const AdamHyper& h, int* t_dev, float* bc_dev, int bias_correction,
                 cudaStream_t st) {
  adam_tick_kernel<<<1, 1, 0, st>>>(t_dev, bc_dev, h.beta1, h.beta2, bias_correction);
  if (n_chunks <= 0) return;
  adam_kernel<<<n_chunks, 256, 0, st>>>(chunks, w, g, m, v, (bf16*)wb, h, bc_dev);
}

void launch_lamb(const AdamChunk* chunks, int n_chunks, float* w, const float* g, float* m, float* v,
                 void* wb, const AdamHyper& h, int* t_dev, float* bc_dev, int bias_correction,
                 float* norms, int n_tensors, cudaStream_t st) {
  adam_tick_kernel<<<1, 1, 0, st>>>(t_dev, bc_dev, h.beta1, h.beta2, bias_correction);
  if (n_chunks <= 0) return;
  cudaMemsetAsync(norms, 0, (size_t)n_tensors * 2 * sizeof(float), st);
  lamb_moments_kernel<<<n_chunks, 256, 0, st>>>(chunks, w, g, m, v, h, bc_dev, norms);
  lamb_apply_kernel<<<n_chunks, 256, 0, st>>>(chunks, w, m, v, (bf16*)wb, h, bc_dev, norms);
}

void launch_nsp_prepare(const int* labels, int B, int S, int* rowsrc, float* inv_n, const int* total_valid,
                        cudaStream_t st) {
  nsp_prepare_kernel<<<1, 128, 0, st>>>(labels, B, S, rowsrc, inv_n, total_valid);
}

void launch_nsp_head(bool bf, const void* pooled, const float* wn, const float* bn, const int* labels,
                     const float* inv_n, void* dup, float* dwn, float* dbn, float* loss, int B, int H,
                     cudaStream_t st) {
  if (B <= 0) return;
  DISPATCH_T(bf, (nsp_head_kernel<T><<<B, 128, 0, st>>>((const T*)pooled, wn, bn, labels, inv_n, (T*)dup, dwn, dbn,
                                                       loss, H)));
}

void launch_tanh(bool bf, const void* x, void* y, int64_t n, cudaStream_t st) {
  if (n <= 0) return;
  int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
  DISPATCH_T(bf, (tanh_kernel<T><<<blocks, 256, 0, st>>>((const T*)x, (T*)y, n)));
}

void launch_type_grad(bool bf, const void* dz, const int* segments, float* dtype, int rows, int H,
                      cudaStream_t st) {
  if (rows <= 0) return;
  const int rpb = 512;
  DISPATCH_T(bf, (type_grad_kernel<T><<<dim3(div_up(H, 128), div_up(rows, rpb)), 128, 0, st>>>(
                     (const T*)dz, segments, dtype, rows, H, rpb)));
}

void launch_dgelu(bool bf, void* d, const void* u, int64_t n, cudaStream_t st) {
  if (n <= 0) return;
  const int vn = bf ? 8 : 4;
  int blocks = (int)std::min<int64_t>((n / vn + 255) / 256, 148 * 8);
  DISPATCH_T(bf, (dgelu_kernel<T><<<blocks, 256, 0, st>>>((T*)d, (const T*)u, n)));
}

void launch_f32_to_bf16(const float* src, void* dst, int64_t n, cudaStream_t st) {
  if (n <= 0) return;
  int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
  f32_to_bf16_kernel<<<blocks, 256, 0, st>>>(src, (bf16*)dst, n);
}

}  // namespace mslt
