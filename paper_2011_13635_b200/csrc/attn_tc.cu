// Fused attention forward for rows of at most 128 keys and 64-wide heads (sm_100a, bf16):
//   P = softmax(mask(scale * Q K^T)),  C = P V      per (sequence, head),
// in one persistent kernel, so the scores never leave the SM and the probabilities reach HBM only
// when the backward pass needs them.  Unfused, the two products are bound by HBM traffic (about
// 32 flop per byte at head width 64); fused, a layer's attention reads Q, K, V once and writes the
// context once.
//   warp 0   : TMA producer: the Q, K and V tiles of a (sequence, head) item, three items deep.
//   warp 1   : one thread issues tcgen05.mma: S = Q K^T into one of two 128-column accumulators,
//              and, once the epilogue warps have put P into shared memory, C = P V.
//   warps 2-9: scaled masked softmax on the accumulator (two warps per 32-row quarter, each half
//              of the columns; row maxima and sums exchanged through shared memory), P written as
//              the bf16 A operand of the second product (128-byte swizzle, by hand) and, for
//              layers that run backward, to global memory; then the context tile is read back
//              from tensor memory and stored.
// P is rounded to bf16 before the second product, exactly as when it is stored and read back.
// Every wait is bounded: when one runs out the CTA raises a status bit, drains and returns.
#include <atomic>

#include "gemm.h"
#include "tc_common.cuh"

namespace mslt {

namespace {

constexpr int AT_STAGES = 3;
constexpr int AT_TILE_BYTES = 128 * 64 * 2;          // one of Q, K, V: 16 KB
constexpr int AT_STAGE_BYTES = 3 * AT_TILE_BYTES;    // 48 KB
constexpr int AT_P_BYTES = 128 * 128 * 2;            // probabilities as an MMA operand: 32 KB
constexpr int AT_STAGING = 2048;                     // per epilogue warp
constexpr uint32_t AT_TMEM_COLS = 512;
constexpr uint32_t AT_O_COL = 256;                   // context accumulator after the two score buffers

struct AttnParams {
  int S, heads, items;
  float scale;
  const int* seq_lens;
  bf16* P;            // [B, A, S, S] or null
  long long p_bo, p_bi;
  bf16* C;            // element (b, i, h, e) at C + b * c_bo + h * c_bi + i * c_ld + e
  long long c_ld, c_bo, c_bi;
  int vec_ok_p, vec_ok_c;
  int q_perm[3], k_perm[3], v_perm[3];
  long long wait_limit;
  int* status;
  uint32_t idesc_s, idesc_o;
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* p_smem = smem + AT_STAGES * AT_STAGE_BYTES;
  uint8_t* staging = p_smem + AT_P_BYTES;
  uint64_t* bars = (uint64_t*)(staging + NUM_EPI_WARPS * AT_STAGING);
  uint64_t* full_bar = bars;                 // [AT_STAGES] tiles of an item have landed
  uint64_t* empty_bar = bars + AT_STAGES;    // [AT_STAGES] both products of an item have read them
  uint64_t* sfull_bar = bars + 2 * AT_STAGES;      // [2] scores complete
  uint64_t* sempty_bar = bars + 2 * AT_STAGES + 2; // [2] scores read by every epilogue warp
  uint64_t* pready_bar = bars + 2 * AT_STAGES + 4; // probabilities in shared memory
  uint64_t* ofull_bar = bars + 2 * AT_STAGES + 5;  // context complete
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * AT_STAGES + 6);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  volatile int* xflag = (volatile int*)((uint8_t*)bars + 256);
  float* xmax = (float*)((uint8_t*)bars + 256 + 64);
  float* xsum = xmax + NUM_EPI_WARPS * 32;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < AT_STAGES; s++) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(smem_u32(&sfull_bar[a]), 1);
      mbar_init(smem_u32(&sempty_bar[a]), NUM_EPI_WARPS);
    }
    mbar_init(smem_u32(pready_bar), NUM_EPI_WARPS);
    mbar_init(smem_u32(ofull_bar), 1);
    *abort_flag = 0;
    *reinterpret_cast<volatile long long*>(abort_flag + 1) = p.wait_limit;
    for (int i = 0; i < NUM_EPI_WARPS; i++) xflag[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(AT_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int n_my = ((int)blockIdx.x < p.items) ? (p.items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;

  if (warp == 0 && lane == 0) {
    // ------------------------------- TMA producer -------------------------------
    bool ok = true;
    int issued = 0;
    for (int i = 0; i < n_my && ok; i++) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int zo = w / p.heads, zi = w - zo * p.heads;
      const uint32_t s = (uint32_t)(i % AT_STAGES), round = (uint32_t)(i / AT_STAGES);
      if (!mbar_wait(smem_u32(&empty_bar[s]), (round & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      const uint32_t fb = smem_u32(&full_bar[s]);
      mbar_expect_tx(fb, AT_STAGE_BYTES);
      const uint32_t sq = smem_u32(smem + (size_t)s * AT_STAGE_BYTES);
      int c[4];
      c[0] = 0; c[p.q_perm[0]] = 0; c[p.q_perm[1]] = zi; c[p.q_perm[2]] = zo;
      tma_load_4d(sq, &tmQ, fb, c[0], c[1], c[2], c[3]);
      c[0] = 0; c[p.k_perm[0]] = 0; c[p.k_perm[1]] = zi; c[p.k_perm[2]] = zo;
      tma_load_4d(sq + AT_TILE_BYTES, &tmK, fb, c[0], c[1], c[2], c[3]);
      // V is read with the head dimension contiguous: two boxes of 64 keys
      c[0] = 0; c[p.v_perm[1]] = zi; c[p.v_perm[2]] = zo;
      c[p.v_perm[0]] = 0;
      tma_load_4d(sq + 2 * AT_TILE_BYTES, &tmV, fb, c[0], c[1], c[2], c[3]);
      c[p.v_perm[0]] = 64;
      tma_load_4d(sq + 2 * AT_TILE_BYTES + AT_TILE_BYTES / 2, &tmV, fb, c[0], c[1], c[2], c[3]);
      issued = i + 1;
    }
    if (!ok || *abort_flag) {
      // give up: let the copies already in flight land before the CTA leaves
      const int n = issued < AT_STAGES ? issued : AT_STAGES;
      for (int k = 0; k < n; k++) {
        const int j = issued - 1 - k;
        const uint32_t fb = smem_u32(&full_bar[j % AT_STAGES]);
        const long long t0 = now_cycles();
        while (!mbar_try_wait(fb, (uint32_t)(j / AT_STAGES) & 1) && now_cycles() - t0 < 200000000ll) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------- MMA issuer -------------------------------
    bool ok = true;
    const uint32_t p_desc_lo = (uint32_t)make_smem_desc(smem_u32(p_smem), 16);
    const uint32_t hi_k = (uint32_t)(make_smem_desc(0, 16) >> 32);
    const uint32_t hi_mn = (uint32_t)(make_smem_desc(0, 64 * BK * 2) >> 32);
    const uint32_t lbo_mn_lo = (uint32_t)make_smem_desc(0, 64 * BK * 2);  // low word carries the LBO field
    auto issue_pv = [&](int j) {  // C = P V of item j
      const uint32_t s = (uint32_t)(j % AT_STAGES);
      const uint32_t sv = smem_u32(smem + (size_t)s * AT_STAGE_BYTES + 2 * AT_TILE_BYTES);
      const uint32_t v_lo = lbo_mn_lo | ((sv & 0x3FFFFu) >> 4);
      uint32_t accum = 0;
#pragma unroll
      for (int kb = 0; kb < 2; kb++)
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; k++) {
          const uint64_t ad = ((uint64_t)hi_k << 32) | (p_desc_lo + kb * (128 * 128 / 16) + k * (UMMA_K * 2 / 16));
          const uint64_t bd = ((uint64_t)hi_mn << 32) | (v_lo + kb * (AT_TILE_BYTES / 2 / 16) + k * (UMMA_K * 128 / 16));
          tc_mma(tmem_base + AT_O_COL, ad, bd, p.idesc_o, accum);
          accum = 1;
        }
      tc_commit(smem_u32(ofull_bar));
      tc_commit(smem_u32(&empty_bar[s]));  // Q, K, V of the item are no longer needed
    };
    for (int i = 0; i < n_my && ok; i++) {
      const uint32_t s = (uint32_t)(i % AT_STAGES), round = (uint32_t)(i / AT_STAGES);
      const uint32_t b = (uint32_t)i & 1, use = (uint32_t)i >> 1;
      if (!mbar_wait(smem_u32(&full_bar[s]), round & 1, abort_flag, p.status)) { ok = false; break; }
      if (!mbar_wait(smem_u32(&sempty_bar[b]), (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const uint32_t sq = smem_u32(smem + (size_t)s * AT_STAGE_BYTES);
      const uint32_t q_lo = (uint32_t)make_smem_desc(sq, 16), k_lo = (uint32_t)make_smem_desc(sq + AT_TILE_BYTES, 16);
#pragma unroll
      for (int k = 0; k < BK / UMMA_K; k++) {
        const uint64_t ad = ((uint64_t)hi_k << 32) | (q_lo + k * (UMMA_K * 2 / 16));
        const uint64_t bd = ((uint64_t)hi_k << 32) | (k_lo + k * (UMMA_K * 2 / 16));
        tc_mma(tmem_base + b * 128, ad, bd, p.idesc_s, k > 0 ? 1u : 0u);
      }
      tc_commit(smem_u32(&sfull_bar[b]));
      if (i > 0) {  // the previous item's probabilities should be ready by now
        if (!mbar_wait(smem_u32(pready_bar), (uint32_t)(i - 1) & 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        issue_pv(i - 1);
      }
    }
    if (ok && n_my > 0) {
      if (mbar_wait(smem_u32(pready_bar), (uint32_t)(n_my - 1) & 1, abort_flag, p.status)) {
        tc_fence_after();
        issue_pv(n_my - 1);
      } else {
        ok = false;
      }
    }
    if (!ok || *abort_flag) {
      // make sure no MMA is still writing tensor memory before it is freed
      tc_commit(smem_u32(&sfull_bar[0]));
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < 2000000ll) {}
    }
  } else if (warp >= 2) {
    // ------------------------------- softmax and context epilogue -------------------------------
    const int q = warp & 3;              // TMEM lane quarter this warp may read
    const int hsel = (warp - 2) >> 2;    // which of the two warps of the quarter
    uint8_t* stg = staging + (size_t)(warp - 2) * AT_STAGING;
    const int me = q * 2 + hsel, other = q * 2 + (hsel ^ 1);
    const int r = q * 32 + lane;         // row of the item this lane owns
    bool ok = true;
    for (int i = 0; i < n_my && ok; i++) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int zo = w / p.heads, zi = w - zo * p.heads;
      const uint32_t b = (uint32_t)i & 1, use = (uint32_t)i >> 1;
      int len = p.seq_lens ? p.seq_lens[zo] : p.S;
      len = min(max(len, 1), p.S);
      if (!mbar_wait(smem_u32(&sfull_bar[b]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const int c0 = hsel, c1 = hsel + 2;  // this warp's two 32-column chunks
      float2 v0[16], v1[16];
      float mx = -INFINITY;
      const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + b * 128;
      tc_ld32(trow + c0 * 32, v0);
      tc_ld32(trow + c1 * 32, v1);
#pragma unroll
      for (int j = 0; j < 16; j++) {
        v0[j].x = (c0 * 32 + 2 * j < len) ? v0[j].x * p.scale : -INFINITY;
        v0[j].y = (c0 * 32 + 2 * j + 1 < len) ? v0[j].y * p.scale : -INFINITY;
        v1[j].x = (c1 * 32 + 2 * j < len) ? v1[j].x * p.scale : -INFINITY;
        v1[j].y = (c1 * 32 + 2 * j + 1 < len) ? v1[j].y * p.scale : -INFINITY;
        mx = fmaxf(mx, fmaxf(fmaxf(v0[j].x, v0[j].y), fmaxf(v1[j].x, v1[j].y)));
      }
      // the scores are in registers: hand the accumulator back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sempty_bar[b]));
      const int seq = i * 2 + 1;
      xmax[me * 32 + lane] = mx;
      if (!pair_sync(xflag, me, other, seq, lane, abort_flag, p.status)) { ok = false; break; }
      mx = fmaxf(mx, xmax[other * 32 + lane]);
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 16; j++) {
        v0[j].x = __expf(v0[j].x - mx);
        v0[j].y = __expf(v0[j].y - mx);
        v1[j].x = __expf(v1[j].x - mx);
        v1[j].y = __expf(v1[j].y - mx);
        sum += (v0[j].x + v0[j].y) + (v1[j].x + v1[j].y);
      }
      xsum[me * 32 + lane] = sum;
      if (!pair_sync(xflag, me, other, seq + 1, lane, abort_flag, p.status)) { ok = false; break; }
      sum += xsum[other * 32 + lane];
      const float2 inv = splat2(1.0f / sum);
#pragma unroll
      for (int j = 0; j < 16; j++) {
        v0[j] = __fmul2_rn(v0[j], inv);
        v1[j] = __fmul2_rn(v1[j], inv);
      }
      // P as the A operand of the second product: k block = 64 keys, row r at 128 * r, its eight
      // 16-byte pieces permuted by r mod 8 (the 128-byte swizzle the tensor core expects)
#pragma unroll
      for (int half = 0; half < 2; half++) {
        const int c = half ? c1 : c0;
        uint8_t* blk = p_smem + (c >> 1) * (128 * 128) + r * 128;
#pragma unroll
        for (int j = 0; j < 4; j++) {
          uint4 pk;
          __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
          for (int e = 0; e < 4; e++) h[e] = __float22bfloat162_rn(half ? v1[4 * j + e] : v0[4 * j + e]);
          *reinterpret_cast<uint4*>(blk + ((((c & 1) * 4 + j) ^ (r & 7)) << 4)) = pk;
        }
      }
      // make the generic-proxy writes visible to the tensor core, then tell the MMA thread
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(pready_bar));
      if (p.P != nullptr) {
        bf16* pg = p.P + zo * p.p_bo + zi * p.p_bi;
        if (c0 * 32 < p.S) stage_store_bf16(stg, lane, v0, pg, p.S, q * 32, c0 * 32, p.S, p.S, p.vec_ok_p);
        if (c1 * 32 < p.S) stage_store_bf16(stg, lane, v1, pg, p.S, q * 32, c1 * 32, p.S, p.S, p.vec_ok_p);
      }
      // context tile: 64 columns, one 32-column chunk per warp of the quarter
      if (!mbar_wait(smem_u32(ofull_bar), (uint32_t)i & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      tc_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + AT_O_COL + hsel * 32, v0);
      tc_fence_before();
      stage_store_bf16(stg, lane, v0, p.C + zo * p.c_bo + zi * p.c_bi, p.c_ld, q * 32, hsel * 32, p.S, 64,
                       p.vec_ok_c);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(AT_TMEM_COLS)
                 : "memory");
  }
}

}  // namespace

static std::atomic<long long> g_attn_launches{0};
long long attn_launches() { return g_attn_launches.load(); }

int attn_fwd_launch(const void* qkv, void* probs, void* ctx, const int* seq_lens, int B, int S, int A, int d,
                    float scale, int* status, cudaStream_t st, char* err) {
  static int num_sms = 0, smem_optin = 0;
  if (num_sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (num_sms <= 0) { snprintf(err, 256, "attention: no CUDA device"); return MSLT_ERR_CUDA; }
  }
  if (d != 64 || S < 1 || S > 128 || B < 1 || A < 1 || !status) {
    snprintf(err, 256, "attention: the fused kernel needs head width 64 and 1 <= S <= 128");
    return MSLT_ERR_ARG;
  }
  const long long H = (long long)A * d;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.S = S; p.heads = A; p.items = B * A; p.scale = scale; p.seq_lens = seq_lens;
  p.P = (bf16*)probs; p.p_bo = (long long)A * S * S; p.p_bi = (long long)S * S;
  p.C = (bf16*)ctx; p.c_ld = H; p.c_bo = (long long)S * H; p.c_bi = d;
  p.vec_ok_p = (S % 8 == 0 && ((uintptr_t)probs & 15) == 0) ? 1 : 0;
  p.vec_ok_c = (H % 8 == 0 && ((uintptr_t)ctx & 15) == 0) ? 1 : 0;
  p.wait_limit = WAIT_LIMIT_CYCLES;
  p.status = status;
  // fp32 accumulate, bf16 x bf16; scores: both operands k-contiguous, N = 128; context: V row-contiguous, N = 64
  p.idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  p.idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  const bf16* base = (const bf16*)qkv;
  MapVal mq, mk, mv;
  int rc = get_map(base, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mq, err);
  if (rc) return rc;
  rc = get_map(base + H, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mk, err);
  if (rc) return rc;
  rc = get_map(base + 2 * H, d, S, 1, 3 * H, (long long)S * 3 * H, d, A, B, 64, &mv, err);
  if (rc) return rc;
  for (int i = 0; i < 3; i++) { p.q_perm[i] = mq.perm[i]; p.k_perm[i] = mk.perm[i]; p.v_perm[i] = mv.perm[i]; }
  const size_t smem_bytes = (size_t)AT_STAGES * AT_STAGE_BYTES + AT_P_BYTES + NUM_EPI_WARPS * AT_STAGING + 1024 +
                            256 + 64 + 2 * NUM_EPI_WARPS * 32 * 4;
  if ((int)smem_bytes > smem_optin) { snprintf(err, 256, "attention: not enough shared memory"); return MSLT_ERR_CUDA; }
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
    if (e != cudaSuccess) { snprintf(err, 256, "attention: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
    attr_set = true;
  }
  const int grid = p.items < num_sms ? p.items : num_sms;
  attn_fwd_kernel<<<grid, NUM_THREADS, smem_bytes, st>>>(mq.map, mk.map, mv.map, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { snprintf(err, 256, "attention: launch failed: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
  g_attn_launches++;
  return 0;
}

}  // namespace mslt
