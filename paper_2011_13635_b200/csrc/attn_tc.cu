// Fused attention forward for rows of at most 128 keys and 64-wide heads (sm_100a, bf16):
//   P = softmax(mask(scale * Q K^T)),  C = P V      per (sequence, head),
// in one persistent kernel, so the scores never leave the SM and the probabilities reach HBM only
// when the backward pass needs them.  Unfused, the two products are bound by HBM traffic (about
// 32 flop per byte at head width 64); fused, a layer's attention reads Q, K, V once and writes the
// context once.
//   warp 0   : TMA producer: the Q, K and V tiles of a (sequence, head) item, four items deep.
//   warp 1   : one thread issues tcgen05.mma: S = Q K^T into one of two 128-column accumulators,
//              and, once a softmax group has put P into shared memory, C = P V into one of two
//              64-column accumulators.
//   warps 2-5, 6-9: two softmax groups that take alternate items, so that the exponentials of one
//              item overlap the second product and the stores of the other.  A thread owns one
//              query row: it reads the row's 128 scores from tensor memory, applies scale and
//              mask, forms max, exponentials and sum with no exchange between threads, writes the
//              normalised row as the bf16 A operand of the second product (128-byte swizzle, by
//              hand, over the item's dead Q and K tiles) and, for layers that run backward, to
//              global memory; then reads the context tile back from tensor memory and stores it.
// P is rounded to bf16 before the second product, exactly as when it is stored and read back.
// Every wait is bounded: when one runs out the CTA raises a status bit, drains and returns.
#include <atomic>

#include "gemm.h"
#include "tc_common.cuh"

namespace mslt {

namespace {

constexpr int AT_STAGES = 4;
constexpr int AT_TILE_BYTES = 128 * 64 * 2;          // one of Q, K, V: 16 KB
constexpr int AT_STAGE_BYTES = 3 * AT_TILE_BYTES;    // 48 KB
constexpr int AT_STAGING = 2048;                     // per epilogue warp
constexpr uint32_t AT_TMEM_COLS = 512;
constexpr uint32_t AT_O_COL = 256;                   // two context accumulators after the two score buffers
constexpr int AT_GROUP_WARPS = 4;                    // warps of a softmax group

struct AttnParams {
  int S, heads, items;
  float scale;
  const int* seq_lens;
  bf16* P;            // [B, A, S, S] or null
  long long p_bo, p_bi;
  bf16* C;            // element (b, i, h, e) at C + b * c_bo + h * c_bi + i * c_ld + e
  long long c_ld, c_bo, c_bi;
  int vec_ok_p, vec_ok_c;
  int fast_p, fast_c;  // rows may be stored directly with 32-byte stores
  int q_perm[3], k_perm[3], v_perm[3];
  long long wait_limit;
  int starve;         // test hook: the producer issues no copies, so the first wait runs out
  int* status;
  uint32_t idesc_s, idesc_o;
};

// A thread that owns a whole row stores 32 of its columns (64 contiguous bytes of bf16) with two
// 32-byte stores: every store fills a full sector, and no trip through shared memory is needed.
// dst must be 32-byte aligned (row_fast says whether a buffer qualifies).
__device__ __forceinline__ void store_row32_bf16(bf16* dst, const float2 (&w)[16]) {
  uint32_t h[16];
#pragma unroll
  for (int e = 0; e < 16; e++) {
    const __nv_bfloat162 t = __float22bfloat162_rn(w[e]);
    h[e] = *reinterpret_cast<const uint32_t*>(&t);
  }
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(h[0]), "r"(h[1]), "r"(h[2]),
               "r"(h[3]), "r"(h[4]), "r"(h[5]), "r"(h[6]), "r"(h[7])
               : "memory");
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 16), "r"(h[8]), "r"(h[9]),
               "r"(h[10]), "r"(h[11]), "r"(h[12]), "r"(h[13]), "r"(h[14]), "r"(h[15])
               : "memory");
}
inline int row_fast(const void* ptr, long long ld_elems) {
  return (((uintptr_t)ptr & 31) == 0 && (ld_elems * 2) % 32 == 0) ? 1 : 0;
}

// Four 32-column reads of a row in flight together, one wait for all.
__device__ __forceinline__ void tc_ld128(uint32_t taddr, float2 (&v)[4][16]) {
  uint32_t r0[32], r1[32], r2[32], r3[32];
  tc_ld32_issue(taddr, r0);
  tc_ld32_issue(taddr + 32, r1);
  tc_ld32_issue(taddr + 64, r2);
  tc_ld32_issue(taddr + 96, r3);
  tc_ld32_wait(r0);
  tc_ld32_wait(r1);
  tc_ld32_wait(r2);
  tc_ld32_wait(r3);
#pragma unroll
  for (int i = 0; i < 16; i++) {
    v[0][i] = make_float2(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
    v[1][i] = make_float2(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
    v[2][i] = make_float2(__uint_as_float(r2[2 * i]), __uint_as_float(r2[2 * i + 1]));
    v[3][i] = make_float2(__uint_as_float(r3[2 * i]), __uint_as_float(r3[2 * i + 1]));
  }
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = smem + AT_STAGES * AT_STAGE_BYTES;
  uint64_t* bars = (uint64_t*)(staging + NUM_EPI_WARPS * AT_STAGING);
  uint64_t* full_bar = bars;                 // [AT_STAGES] tiles of an item have landed
  uint64_t* empty_bar = bars + AT_STAGES;    // [AT_STAGES] both products of an item have read them
  uint64_t* sfull_bar = bars + 2 * AT_STAGES;      // [2] scores complete
  uint64_t* sempty_bar = bars + 2 * AT_STAGES + 2; // [2] scores read by every epilogue warp
  uint64_t* pready_bar = bars + 2 * AT_STAGES + 4; // [2] probabilities of a group's item in shared memory
  uint64_t* ofull_bar = bars + 2 * AT_STAGES + 6;  // [2] context of a group's item complete
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * AT_STAGES + 8);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < AT_STAGES; s++) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(smem_u32(&sfull_bar[a]), 1);
      mbar_init(smem_u32(&sempty_bar[a]), AT_GROUP_WARPS);
      mbar_init(smem_u32(&pready_bar[a]), AT_GROUP_WARPS);
      mbar_init(smem_u32(&ofull_bar[a]), 1);
    }
    *abort_flag = 0;
    *reinterpret_cast<volatile long long*>(abort_flag + 1) = p.wait_limit;
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

  if (warp == 0 && lane == 0 && !p.starve) {
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
    const uint32_t hi = (uint32_t)(make_smem_desc(0, 16) >> 32);           // same for both operand forms
    const uint32_t lbo_mn_lo = (uint32_t)make_smem_desc(0, 64 * BK * 2);   // low word carries the LBO field
    auto issue_pv = [&](int j) {  // C = P V of item j; P lies over the item's Q and K tiles
      const uint32_t s = (uint32_t)(j % AT_STAGES), g = (uint32_t)j & 1;
      const uint32_t sq = smem_u32(smem + (size_t)s * AT_STAGE_BYTES);
      const uint32_t p_lo = (uint32_t)make_smem_desc(sq, 16);
      const uint32_t v_lo = lbo_mn_lo | (((sq + 2 * AT_TILE_BYTES) & 0x3FFFFu) >> 4);
      uint32_t accum = 0;
#pragma unroll
      for (int kb = 0; kb < 2; kb++)
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; k++) {
          const uint64_t ad = ((uint64_t)hi << 32) | (p_lo + kb * (AT_TILE_BYTES / 16) + k * (UMMA_K * 2 / 16));
          const uint64_t bd = ((uint64_t)hi << 32) | (v_lo + kb * (AT_TILE_BYTES / 2 / 16) + k * (UMMA_K * 128 / 16));
          tc_mma(tmem_base + AT_O_COL + g * 64, ad, bd, p.idesc_o, accum);
          accum = 1;
        }
      tc_commit(smem_u32(&ofull_bar[g]));
      tc_commit(smem_u32(&empty_bar[s]));  // the item's tiles are no longer needed
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
        const uint64_t ad = ((uint64_t)hi << 32) | (q_lo + k * (UMMA_K * 2 / 16));
        const uint64_t bd = ((uint64_t)hi << 32) | (k_lo + k * (UMMA_K * 2 / 16));
        tc_mma(tmem_base + b * 128, ad, bd, p.idesc_s, k > 0 ? 1u : 0u);
      }
      tc_commit(smem_u32(&sfull_bar[b]));
      if (i > 0) {  // the previous item's probabilities: its group has been at work since S(i-1)
        const uint32_t g = (uint32_t)(i - 1) & 1, guse = (uint32_t)(i - 1) >> 1;
        if (!mbar_wait(smem_u32(&pready_bar[g]), guse & 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        issue_pv(i - 1);
      }
    }
    if (ok && n_my > 0) {
      const uint32_t g = (uint32_t)(n_my - 1) & 1, guse = (uint32_t)(n_my - 1) >> 1;
      if (mbar_wait(smem_u32(&pready_bar[g]), guse & 1, abort_flag, p.status)) {
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
    // ------------------------------- softmax groups -------------------------------
    const int q = warp & 3;              // TMEM lane quarter this warp may read
    const int g = (warp - 2) >> 2;       // softmax group: items g, g + 2, ...
    uint8_t* stg = staging + (size_t)(warp - 2) * AT_STAGING;
    const int r = q * 32 + lane;         // query row this thread owns
    bool ok = true;
    for (int i = g; i < n_my && ok; i += 2) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int zo = w / p.heads, zi = w - zo * p.heads;
      const uint32_t s = (uint32_t)(i % AT_STAGES), use = (uint32_t)i >> 1;
      int len = p.seq_lens ? p.seq_lens[zo] : p.S;
      len = min(max(len, 1), p.S);
      if (!mbar_wait(smem_u32(&sfull_bar[g]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      float2 v[4][16];  // the row's 128 scores, then its probabilities
      const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)g * 128;
#pragma unroll
      for (int c = 0; c < 4; c++) tc_ld32(trow + c * 32, v[c]);
      // the scores are in registers: hand the accumulator back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sempty_bar[g]));
      // Row maximum over the valid keys: one chain per 32-column chunk keeps the dependent
      // chains short; only a chunk that crosses the length needs element-wise masking.
      float mc[4];
#pragma unroll
      for (int c = 0; c < 4; c++) {
        mc[c] = -INFINITY;
        if ((c + 1) * 32 > len) {
#pragma unroll
          for (int j = 0; j < 16; j++) {
            if (c * 32 + 2 * j >= len) v[c][j].x = -INFINITY;
            if (c * 32 + 2 * j + 1 >= len) v[c][j].y = -INFINITY;
          }
        }
#pragma unroll
        for (int j = 0; j < 16; j++) mc[c] = fmaxf(mc[c], fmaxf(v[c][j].x, v[c][j].y));
      }
      const float mx = fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
      // exp(scale * (x - max)) as 2^(x * scale * log2(e) - max * scale * log2(e)): one packed
      // multiply-add per pair and one exponential per element; masked keys give 2^(-inf) = 0
      const float sl2 = p.scale * 1.4426950408889634f;
      const float2 k2 = splat2(sl2), nm2 = splat2(-mx * sl2);
      float2 sc[4];
#pragma unroll
      for (int c = 0; c < 4; c++) {
        sc[c] = make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 16; j++) {
          const float2 t = __ffma2_rn(v[c][j], k2, nm2);
          v[c][j].x = fast_exp2(t.x);
          v[c][j].y = fast_exp2(t.y);
          sc[c] = __fadd2_rn(sc[c], v[c][j]);
        }
      }
      const float sum = ((sc[0].x + sc[0].y) + (sc[1].x + sc[1].y)) + ((sc[2].x + sc[2].y) + (sc[3].x + sc[3].y));
      const float2 inv = splat2(1.0f / sum);
      // P as the A operand of the second product, over the item's Q and K tiles (both products
      // of the first kind have completed): k block = 64 keys = 16 KB, row r at 128 * r, its eight
      // 16-byte pieces permuted by r mod 8 (the 128-byte swizzle the tensor core expects)
      uint8_t* prow = smem + (size_t)s * AT_STAGE_BYTES + r * 128;
#pragma unroll
      for (int c = 0; c < 4; c++) {
#pragma unroll
        for (int j = 0; j < 16; j++) v[c][j] = __fmul2_rn(v[c][j], inv);
#pragma unroll
        for (int j = 0; j < 4; j++) {
          uint4 pk;
          __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
          for (int e = 0; e < 4; e++) h[e] = __float22bfloat162_rn(v[c][4 * j + e]);
          *reinterpret_cast<uint4*>(prow + (c >> 1) * AT_TILE_BYTES + ((((c & 1) * 4 + j) ^ (r & 7)) << 4)) = pk;
        }
      }
      // make the generic-proxy writes visible to the tensor core, then tell the MMA thread
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&pready_bar[g]));
      if (p.P != nullptr) {
        bf16* pg = p.P + zo * p.p_bo + zi * p.p_bi;
        if (p.fast_p) {  // S a multiple of 32: whole 32-column pieces only
          if (r < p.S) {
#pragma unroll
            for (int c = 0; c < 4; c++)
              if (c * 32 < p.S) store_row32_bf16(pg + (long long)r * p.S + c * 32, v[c]);
          }
        } else {
#pragma unroll
          for (int c = 0; c < 4; c++)
            if (c * 32 < p.S) stage_store_bf16(stg, lane, v[c], pg, p.S, q * 32, c * 32, p.S, p.S, p.vec_ok_p);
        }
      }
      // context tile: 64 columns of this group's accumulator
      if (!mbar_wait(smem_u32(&ofull_bar[g]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const uint32_t orow = tmem_base + ((uint32_t)(q * 32) << 16) + AT_O_COL + (uint32_t)g * 64;
      tc_ld32(orow, v[0]);
      tc_ld32(orow + 32, v[1]);
      tc_fence_before();
      bf16* cg = p.C + zo * p.c_bo + zi * p.c_bi;
      if (p.fast_c) {
        if (r < p.S) {
          store_row32_bf16(cg + (long long)r * p.c_ld, v[0]);
          store_row32_bf16(cg + (long long)r * p.c_ld + 32, v[1]);
        }
      } else {
        stage_store_bf16(stg, lane, v[0], cg, p.c_ld, q * 32, 0, p.S, 64, p.vec_ok_c);
        stage_store_bf16(stg, lane, v[1], cg, p.c_ld, q * 32, 32, p.S, 64, p.vec_ok_c);
      }
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

// ---- forward for rows of 129..512 keys -----------------------------------------------------------
// A work item is (sequence, head, tile of 128 queries); the keys come in blocks of 128.  The scores
// of a row do not fit tensor memory next to the context, so an item runs two passes over the key
// blocks.  When the probabilities are wanted: pass 1 forms the row maximum and the sum of
// exponentials (S = Q K_j^T only), pass 2 forms the scores again, writes P_j = exp(.)/sum as bf16
// and accumulates C += P_j V_j: an exact softmax with no rescaling of the context, and
// probabilities that can be stored as they are.  When they are not wanted (a frozen layer), pass 1
// forms the maximum only, pass 2 uses exp(s - max) as it is, sums it on the way, and the context
// is divided by the sum at the end: half the exponentials.
// Each of the two softmax groups owns every second item of the CTA, whole: its own Q tile, ring of
// K / V tiles, score and context accumulators, P block, producer thread and MMA-issuing thread.  A
// thread owns one query row of its group's item through all key blocks, so nothing is exchanged
// between the groups, and the waits of one item (loads, the P hand-over, the last second product,
// the context store) are covered by the other item's arithmetic.  Measured on the earlier form, in
// which the two groups shared one item: 21 k cycles per item of which 8 k were exponentials.
constexpr int AL_THREADS = NUM_THREADS + 64;     // warps 10 and 11: MMA issuer and producer of group 1
constexpr int AL_RING = 3;                       // 16 KB tiles (a K block or a V block) per group
constexpr int AL_P_BYTES = 2 * AT_TILE_BYTES;    // P_j as an MMA operand: 32 KB
constexpr int AL_BARS_PER_GROUP = 4 + 2 * AL_RING + 6;
constexpr long long AL_GROUP_SKEW_CYCLES = 2000;

__global__ void __launch_bounds__(AL_THREADS, 1)
attn_fwd_long_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* q_smem = smem;                                        // [group] Q tile
  uint8_t* ring_smem = q_smem + 2 * AT_TILE_BYTES;               // [group][AL_RING] K or V tile
  uint8_t* p_smem = ring_smem + 2 * AL_RING * AT_TILE_BYTES;     // [group] P block
  uint8_t* staging = p_smem + 2 * AL_P_BYTES;
  uint64_t* bars = (uint64_t*)(staging + NUM_EPI_WARPS * AT_STAGING);
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * AL_BARS_PER_GROUP);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int g = 0; g < 2; g++) {
      uint64_t* b = bars + g * AL_BARS_PER_GROUP;
      for (int a = 0; a < 2 + 2 * AL_RING + 1; a++) mbar_init(smem_u32(&b[a]), 1);  // qfull, qempty, tfull[], tempty[], sfull
      mbar_init(smem_u32(&b[2 + 2 * AL_RING + 1]), AT_GROUP_WARPS);  // sempty
      mbar_init(smem_u32(&b[2 + 2 * AL_RING + 2]), AT_GROUP_WARPS);  // pready
      mbar_init(smem_u32(&b[2 + 2 * AL_RING + 3]), 1);               // pfree
      mbar_init(smem_u32(&b[2 + 2 * AL_RING + 4]), 1);               // ofull
      mbar_init(smem_u32(&b[2 + 2 * AL_RING + 5]), AT_GROUP_WARPS);  // oempty
    }
    *abort_flag = 0;
    *reinterpret_cast<volatile long long*>(abort_flag + 1) = p.wait_limit;
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
  const int nqt = (p.S + 127) >> 7;   // query tiles per (sequence, head); key blocks likewise
  const int nzh = p.items / nqt;      // (sequence, head) pairs
  // Keys at or beyond the sequence's length have probability 0: an item covers only the
  // ceil(len / 128) key blocks that hold valid keys, and a query tile that lies wholly in the
  // padding is not computed at all (its context rows, which nothing may depend on, are zeroed).
  // Every role derives the same counts from seq_lens.
  auto item_len = [&](int zo) {
    int len = p.seq_lens ? p.seq_lens[zo] : p.S;
    return min(max(len, 1), p.S);
  };
  const int n_my = ((int)blockIdx.x < p.items) ? (p.items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  // Which group this thread serves, and that group's barriers.  Running counts per group: ig items,
  // tt ring tiles, sp score products, pv second products; each barrier's phase is the parity of
  // the count it is used by.
  const int g = warp == 0 ? 0 : (warp == 1 ? 0 : (warp >= 10 ? 1 : (warp - 2) >> 2));
  uint64_t* gb = bars + g * AL_BARS_PER_GROUP;
  const uint32_t qfull = smem_u32(&gb[0]), qempty = smem_u32(&gb[1]);
  const uint32_t tfull0 = smem_u32(&gb[2]), tempty0 = smem_u32(&gb[2 + AL_RING]);
  const uint32_t sfull = smem_u32(&gb[2 + 2 * AL_RING]), sempty = smem_u32(&gb[2 + 2 * AL_RING + 1]);
  const uint32_t pready = smem_u32(&gb[2 + 2 * AL_RING + 2]), pfree = smem_u32(&gb[2 + 2 * AL_RING + 3]);
  const uint32_t ofull = smem_u32(&gb[2 + 2 * AL_RING + 4]), oempty = smem_u32(&gb[2 + 2 * AL_RING + 5]);
  uint8_t* my_q = q_smem + g * AT_TILE_BYTES;
  uint8_t* my_ring = ring_smem + (size_t)g * AL_RING * AT_TILE_BYTES;
  uint8_t* my_p = p_smem + (size_t)g * AL_P_BYTES;
  const bool want_p = p.P != nullptr;
  // Tiles of an item in the order the MMA thread uses them: pass 1: K_0 .. K_{n-1}; pass 2: K_0, then
  // (K_j, V_{j-1}) for j = 1 .. n-1, then V_{n-1} (the scores of block j are issued before the second
  // product of block j - 1, which has to wait for that block's probabilities).

  if ((warp == 0 || warp == 11) && lane == 0 && !p.starve) {
    // ------------------------------- TMA producer of group g -------------------------------
    bool ok = true;
    uint32_t tt = 0, ig = 0;
    for (int i = g; i < n_my && ok; i += 2) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int qt = w / nzh, zh = w - qt * nzh;  // query tile slowest: tiles that may be padding come last
      const int zo = zh / p.heads, zi = zh - zo * p.heads;
      const int len = item_len(zo);
      if (qt * 128 >= len) continue;
      const int nkb = (len + 127) >> 7;
      if (!mbar_wait(qempty, (ig & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      ig++;
      int c[4];
      c[0] = 0; c[p.q_perm[0]] = qt * 128; c[p.q_perm[1]] = zi; c[p.q_perm[2]] = zo;
      mbar_expect_tx(qfull, AT_TILE_BYTES);
      tma_load_4d(smem_u32(my_q), &tmQ, qfull, c[0], c[1], c[2], c[3]);
      for (int idx = 0; idx < 3 * nkb; idx++, tt++) {
        // which block, and K or V
        int j = idx;
        bool is_v = false;
        if (idx >= nkb) {
          const int k = idx - nkb;
          if (k == 0) j = 0;
          else if (k == 2 * nkb - 1) { j = nkb - 1; is_v = true; }
          else if (k & 1) j = (k + 1) >> 1;
          else { j = (k >> 1) - 1; is_v = true; }
        }
        const uint32_t slot = tt % AL_RING, round = tt / AL_RING;
        if (!mbar_wait(tempty0 + slot * 8, (round & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
        const uint32_t fb = tfull0 + slot * 8;
        mbar_expect_tx(fb, AT_TILE_BYTES);
        const int* perm = is_v ? p.v_perm : p.k_perm;
        c[0] = 0; c[1] = 0; c[2] = 0; c[3] = 0;
        c[perm[0]] = j * 128; c[perm[1]] = zi; c[perm[2]] = zo;
        tma_load_4d(smem_u32(my_ring + (size_t)slot * AT_TILE_BYTES), is_v ? &tmV : &tmK, fb, c[0], c[1], c[2], c[3]);
      }
    }
    if (!ok || *abort_flag) {  // give the copies in flight time to land before the CTA leaves
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < 4000000ll) {}
    }
  } else if ((warp == 1 || warp == 10) && lane == 0) {
    // ------------------------------- MMA issuer of group g -------------------------------
    bool ok = true;
    const uint32_t hi = (uint32_t)(make_smem_desc(0, 16) >> 32);
    const uint32_t lbo_mn_lo = (uint32_t)make_smem_desc(0, 64 * BK * 2);
    const uint32_t p_lo = (uint32_t)make_smem_desc(smem_u32(my_p), 16);
    const uint32_t q_lo = (uint32_t)make_smem_desc(smem_u32(my_q), 16);
    const uint32_t s_tmem = tmem_base + (uint32_t)g * 128, o_tmem = tmem_base + AT_O_COL + (uint32_t)g * 64;
    uint32_t tt = 0, sp = 0, pv = 0, ig = 0;
    if (g == 1) {
      // The two groups do the same work at the same pace: started together they would want the
      // exponential unit at the same moments and leave it idle at the same moments.  Half a block
      // period of head start for group 0 keeps them out of step.
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < AL_GROUP_SKEW_CYCLES) {}
    }
    for (int i = g; i < n_my && ok; i += 2) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int qt = w / nzh, zh = w - qt * nzh;
      const int len = item_len(zh / p.heads);
      if (qt * 128 >= len) continue;
      const int nkb = (len + 127) >> 7;
      if (!mbar_wait(qfull, ig & 1, abort_flag, p.status)) { ok = false; break; }
      auto issue_scores = [&]() -> bool {  // S = Q K^T with the K tile in ring position tt
        const uint32_t slot = tt % AL_RING, round = tt / AL_RING;
        if (!mbar_wait(tfull0 + slot * 8, round & 1, abort_flag, p.status)) return false;
        if (!mbar_wait(sempty, (sp & 1) ^ 1, abort_flag, p.status)) return false;
        tc_fence_after();
        const uint32_t k_lo = (uint32_t)make_smem_desc(smem_u32(my_ring + (size_t)slot * AT_TILE_BYTES), 16);
#pragma unroll
        for (int k = 0; k < BK / UMMA_K; k++) {
          const uint64_t ad = ((uint64_t)hi << 32) | (q_lo + k * (UMMA_K * 2 / 16));
          const uint64_t bd = ((uint64_t)hi << 32) | (k_lo + k * (UMMA_K * 2 / 16));
          tc_mma(s_tmem, ad, bd, p.idesc_s, k > 0 ? 1u : 0u);
        }
        tc_commit(sfull);
        tc_commit(tempty0 + slot * 8);  // the K tile is free once the product has completed
        tt++; sp++;
        return true;
      };
      auto issue_pv = [&](int j) -> bool {  // C (+)= P_j V_j with the V tile in ring position tt
        const uint32_t slot = tt % AL_RING, round = tt / AL_RING;
        if (!mbar_wait(pready, pv & 1, abort_flag, p.status)) return false;
        if (j == 0 && !mbar_wait(oempty, (ig & 1) ^ 1, abort_flag, p.status)) return false;
        if (!mbar_wait(tfull0 + slot * 8, round & 1, abort_flag, p.status)) return false;
        tc_fence_after();
        const uint32_t sv = smem_u32(my_ring + (size_t)slot * AT_TILE_BYTES);
        const uint32_t v_lo = lbo_mn_lo | ((sv & 0x3FFFFu) >> 4);
#pragma unroll
        for (int kb = 0; kb < 2; kb++)
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            const uint64_t ad = ((uint64_t)hi << 32) | (p_lo + kb * (AT_TILE_BYTES / 16) + k * (UMMA_K * 2 / 16));
            const uint64_t bd = ((uint64_t)hi << 32) | (v_lo + kb * (AT_TILE_BYTES / 2 / 16) + k * (UMMA_K * 128 / 16));
            tc_mma(o_tmem, ad, bd, p.idesc_o, (j > 0 || kb > 0 || k > 0) ? 1u : 0u);
          }
        tc_commit(pfree);
        tc_commit(tempty0 + slot * 8);
        tt++; pv++;
        return true;
      };
      for (int j = 0; j < nkb && ok; j++) ok = issue_scores();  // pass 1
      if (ok) ok = issue_scores();                                 // pass 2
      for (int j = 1; j < nkb && ok; j++) {
        ok = issue_scores();
        if (ok && j == nkb - 1) tc_commit(qempty);  // the last product that reads Q has been issued
        if (ok) ok = issue_pv(j - 1);
      }
      if (ok && nkb == 1) tc_commit(qempty);
      if (ok) ok = issue_pv(nkb - 1);
      if (ok) tc_commit(ofull);
      ig++;
    }
    if (!ok || *abort_flag) {
      tc_commit(sfull);
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < 2000000ll) {}
    }
  } else if (warp >= 2 && warp < 2 + NUM_EPI_WARPS) {
    // ------------------------------- softmax group g -------------------------------
    const int q = warp & 3;
    uint8_t* stg = staging + (size_t)(warp - 2) * AT_STAGING;
    const int r = q * 32 + lane;
    const float sl2 = p.scale * 1.4426950408889634f;
    const float2 k2 = splat2(sl2);
    bool ok = true;
    uint32_t sp = 0, pv = 0, ig = 0;
    const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)g * 128;
    const uint32_t orow = tmem_base + ((uint32_t)(q * 32) << 16) + AT_O_COL + (uint32_t)g * 64;
    for (int i = g; i < n_my && ok; i += 2) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int qt = w / nzh, zh = w - qt * nzh;
      const int zo = zh / p.heads, zi = zh - zo * p.heads;
      const int len = item_len(zo);
      float2 v[4][16];
      bf16* cg = p.C + zo * p.c_bo + zi * p.c_bi + (long long)qt * 128 * p.c_ld;
      bf16* pg = want_p ? p.P + zo * p.p_bo + zi * p.p_bi + (long long)qt * 128 * p.S : nullptr;
      if (qt * 128 >= len) {
        // a query tile in the padding: zero context rows (finite, so that masked reads stay harmless)
#pragma unroll
        for (int e = 0; e < 16; e++) v[0][e] = make_float2(0.f, 0.f);
        stage_store_bf16(stg, lane, v[0], cg, p.c_ld, q * 32, 0, p.S - qt * 128, 64, p.vec_ok_c);
        stage_store_bf16(stg, lane, v[0], cg, p.c_ld, q * 32, 32, p.S - qt * 128, 64, p.vec_ok_c);
        if (pg != nullptr)
          for (int n0 = 0; n0 < p.S; n0 += 32)
            stage_store_bf16(stg, lane, v[0], pg, p.S, q * 32, n0, p.S - qt * 128, p.S, p.vec_ok_p);
        continue;
      }
      const int nkb = (len + 127) >> 7;
      // reads the group's next score block into v, masks it; returns its row maximum
      auto load_block = [&](int j, float& bm) -> bool {
        if (!mbar_wait(sfull, sp & 1, abort_flag, p.status)) return false;
        sp++;
        tc_fence_after();
        tc_ld128(trow, v);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(sempty);
        float mc[4];
#pragma unroll
        for (int c = 0; c < 4; c++) {
          mc[c] = -INFINITY;
          const int k0 = j * 128 + c * 32;
          if (k0 + 32 > len) {
#pragma unroll
            for (int e = 0; e < 16; e++) {
              if (k0 + 2 * e >= len) v[c][e].x = -INFINITY;
              if (k0 + 2 * e + 1 >= len) v[c][e].y = -INFINITY;
            }
          }
#pragma unroll
          for (int e = 0; e < 16; e++) mc[c] = fmaxf(mc[c], fmaxf(v[c][e].x, v[c][e].y));
        }
        bm = fmaxf(fmaxf(mc[0], mc[1]), fmaxf(mc[2], mc[3]));
        return true;
      };
      // pass 1: running maximum of the raw scores; with probabilities wanted also the running sum
      // of 2^((s - max) * scale * log2 e)
      float mr = -INFINITY, l = 0.f;
      for (int j = 0; j < nkb && ok; j++) {
        float bm;
        if (!load_block(j, bm)) { ok = false; break; }
        const float mn = fmaxf(mr, bm);
        if (want_p && mn != -INFINITY) {
          const float2 nm2 = splat2(-mn * sl2);
          float2 sc[4];
#pragma unroll
          for (int c = 0; c < 4; c++) {
            sc[c] = make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < 16; e++) {
              const float2 a = __ffma2_rn(v[c][e], k2, nm2);
              sc[c] = __fadd2_rn(sc[c], make_float2(fast_exp2(a.x), fast_exp2(a.y)));
            }
          }
          const float bs = ((sc[0].x + sc[0].y) + (sc[1].x + sc[1].y)) + ((sc[2].x + sc[2].y) + (sc[3].x + sc[3].y));
          l = l * fast_exp2((mr - mn) * sl2) + bs;  // 2^(-inf) = 0 on the first valid block
        }
        mr = mn;
      }
      if (!ok) break;
      // mr is finite: at least one key of the row is valid
      const float2 nM2 = splat2(-mr * sl2);
      const float2 inv = splat2(want_p ? 1.0f / l : 1.0f);
      float2 ls = make_float2(0.f, 0.f);  // without stored probabilities: the sum, formed in pass 2
      // pass 2
      for (int j = 0; j < nkb && ok; j++) {
        float bm;
        if (!load_block(j, bm)) { ok = false; break; }
#pragma unroll
        for (int c = 0; c < 4; c++)
#pragma unroll
          for (int e = 0; e < 16; e++) {
            const float2 a = __ffma2_rn(v[c][e], k2, nM2);
            const float2 ex = make_float2(fast_exp2(a.x), fast_exp2(a.y));
            if (want_p) {
              v[c][e] = __fmul2_rn(ex, inv);
            } else {
              v[c][e] = ex;
              ls = __fadd2_rn(ls, ex);
            }
          }
        // the group's P block is free once its previous second product has read it
        if (!mbar_wait(pfree, (pv & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
        pv++;
        uint8_t* prow = my_p + r * 128;
#pragma unroll
        for (int c = 0; c < 4; c++)
#pragma unroll
          for (int e4 = 0; e4 < 4; e4++) {
            uint4 pk;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
            for (int e = 0; e < 4; e++) h[e] = __float22bfloat162_rn(v[c][4 * e4 + e]);
            *reinterpret_cast<uint4*>(prow + (c >> 1) * AT_TILE_BYTES + ((((c & 1) * 4 + e4) ^ (r & 7)) << 4)) = pk;
          }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(pready);
        if (pg != nullptr) {
          if (p.fast_p) {
            if (qt * 128 + r < p.S) {
#pragma unroll
              for (int c = 0; c < 4; c++)
                if (j * 128 + c * 32 < p.S) store_row32_bf16(pg + (long long)r * p.S + j * 128 + c * 32, v[c]);
            }
          } else {
#pragma unroll
            for (int c = 0; c < 4; c++)
              if (j * 128 + c * 32 < p.S)
                stage_store_bf16(stg, lane, v[c], pg, p.S, q * 32, j * 128 + c * 32, p.S - qt * 128, p.S, p.vec_ok_p);
          }
        }
      }
      if (!ok) break;
      // key blocks past the length: their probabilities are 0
      if (pg != nullptr && nkb * 128 < p.S) {
        float2 zr[16];
#pragma unroll
        for (int e = 0; e < 16; e++) zr[e] = make_float2(0.f, 0.f);
        for (int n0 = nkb * 128; n0 < p.S; n0 += 32)
          stage_store_bf16(stg, lane, zr, pg, p.S, q * 32, n0, p.S - qt * 128, p.S, p.vec_ok_p);
      }
      // context tile: the row's 64 columns
      if (!mbar_wait(ofull, ig & 1, abort_flag, p.status)) { ok = false; break; }
      ig++;
      tc_fence_after();
      tc_ld32(orow, v[0]);
      tc_ld32(orow + 32, v[1]);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(oempty);
      if (!want_p) {
        const float2 il = splat2(1.0f / (ls.x + ls.y));
#pragma unroll
        for (int e = 0; e < 16; e++) {
          v[0][e] = __fmul2_rn(v[0][e], il);
          v[1][e] = __fmul2_rn(v[1][e], il);
        }
      }
      if (p.fast_c) {
        if (qt * 128 + r < p.S) {
          store_row32_bf16(cg + (long long)r * p.c_ld, v[0]);
          store_row32_bf16(cg + (long long)r * p.c_ld + 32, v[1]);
        }
      } else {
        stage_store_bf16(stg, lane, v[0], cg, p.c_ld, q * 32, 0, p.S - qt * 128, 64, p.vec_ok_c);
        stage_store_bf16(stg, lane, v[1], cg, p.c_ld, q * 32, 32, p.S - qt * 128, 64, p.vec_ok_c);
      }
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

// ---- backward ---------------------------------------------------------------------------------------
// Per (sequence, head) item, with P the saved probabilities and dC the gradient of the context:
//   dV = P^T dC,  dP = dC V^T,  dS = P o (dP - rowsum(dP o P)) * scale,  dQ = dS K,  dK = dS^T Q.
// The same roles as the forward kernel.  One shared-memory stage holds the item's Q, K, V, dC and
// P tiles, every tile as 128-byte-swizzled rows indexed by position, which serves both operand
// forms: rows as the m/n index with k contiguous, or rows as the k index with m/n contiguous.
// dS (bf16) overwrites P once the first two products have completed.  A softmax group's thread
// owns row r of its item: query r of dP, dS and dQ, key r of dK and dV.  Tensor memory per group:
// dP in 128 columns, later reused by dQ and dK, and dV in 64.
constexpr int AB_STAGE_BYTES = 6 * AT_TILE_BYTES;  // Q, K, V, dC, P (two tiles): 96 KB
constexpr uint32_t AB_GROUP_COLS = 192;

struct AttnBwdParams {
  int S, heads, items;
  float scale;
  bf16* dQKV;         // element (b, i, which, h, e) at dQKV + b * g_bo + i * g_ld + which * H + h * 64 + e
  long long g_ld, g_bo, H;
  int vec_ok, fast;
  int q_perm[3], k_perm[3], v_perm[3], c_perm[3], p_perm[3];
  long long wait_limit;
  int starve;         // test hook, as in the forward kernels
  int* status;
  uint32_t idesc_dv, idesc_dp, idesc_dq, idesc_dk;
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmC,
                const __grid_constant__ CUtensorMap tmP, const AttnBwdParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint8_t* staging = smem + 2 * AB_STAGE_BYTES;
  uint64_t* bars = (uint64_t*)(staging + NUM_EPI_WARPS * AT_STAGING);
  uint64_t* full_bar = bars;           // [2] the item's tiles have landed (stage = group = item parity)
  uint64_t* empty_bar = bars + 2;      // [2] every product of the item has read them
  uint64_t* dpfull_bar = bars + 4;     // [2] dV and dP complete
  uint64_t* dsready_bar = bars + 6;    // [2] dS in shared memory, dP read by the whole group
  uint64_t* gfull_bar = bars + 8;      // [2] dQ and dK complete
  uint64_t* accfree_bar = bars + 10;   // [2] the group has read dQ, dK, dV of its item
  uint32_t* tmem_slot = (uint32_t*)(bars + 12);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int a = 0; a < 2; a++) {
      mbar_init(smem_u32(&full_bar[a]), 1);
      mbar_init(smem_u32(&empty_bar[a]), 1);
      mbar_init(smem_u32(&dpfull_bar[a]), 1);
      mbar_init(smem_u32(&dsready_bar[a]), AT_GROUP_WARPS);
      mbar_init(smem_u32(&gfull_bar[a]), 1);
      mbar_init(smem_u32(&accfree_bar[a]), AT_GROUP_WARPS);
    }
    *abort_flag = 0;
    *reinterpret_cast<volatile long long*>(abort_flag + 1) = p.wait_limit;
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

  if (warp == 0 && lane == 0 && !p.starve) {
    // ------------------------------- TMA producer -------------------------------
    bool ok = true;
    int issued = 0;
    for (int i = 0; i < n_my && ok; i++) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int zo = w / p.heads, zi = w - zo * p.heads;
      const uint32_t s = (uint32_t)i & 1, round = (uint32_t)i >> 1;
      if (!mbar_wait(smem_u32(&empty_bar[s]), (round & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      const uint32_t fb = smem_u32(&full_bar[s]);
      mbar_expect_tx(fb, AB_STAGE_BYTES);
      const uint32_t base = smem_u32(smem + (size_t)s * AB_STAGE_BYTES);
      int c[4];
      c[0] = 0; c[p.q_perm[0]] = 0; c[p.q_perm[1]] = zi; c[p.q_perm[2]] = zo;
      tma_load_4d(base, &tmQ, fb, c[0], c[1], c[2], c[3]);
      c[0] = 0; c[p.k_perm[0]] = 0; c[p.k_perm[1]] = zi; c[p.k_perm[2]] = zo;
      tma_load_4d(base + AT_TILE_BYTES, &tmK, fb, c[0], c[1], c[2], c[3]);
      c[0] = 0; c[p.v_perm[0]] = 0; c[p.v_perm[1]] = zi; c[p.v_perm[2]] = zo;
      tma_load_4d(base + 2 * AT_TILE_BYTES, &tmV, fb, c[0], c[1], c[2], c[3]);
      c[0] = 0; c[p.c_perm[0]] = 0; c[p.c_perm[1]] = zi; c[p.c_perm[2]] = zo;
      tma_load_4d(base + 3 * AT_TILE_BYTES, &tmC, fb, c[0], c[1], c[2], c[3]);
      // P: two tiles of 64 keys, each 128 query rows of 128 bytes
      c[p.p_perm[0]] = 0; c[p.p_perm[1]] = zi; c[p.p_perm[2]] = zo;
      c[0] = 0;
      tma_load_4d(base + 4 * AT_TILE_BYTES, &tmP, fb, c[0], c[1], c[2], c[3]);
      c[0] = 64;
      tma_load_4d(base + 5 * AT_TILE_BYTES, &tmP, fb, c[0], c[1], c[2], c[3]);
      issued = i + 1;
    }
    if (!ok || *abort_flag) {
      const int n = issued < 2 ? issued : 2;
      for (int k = 0; k < n; k++) {
        const int j = issued - 1 - k;
        const uint32_t fb = smem_u32(&full_bar[j & 1]);
        const long long t0 = now_cycles();
        while (!mbar_try_wait(fb, (uint32_t)(j >> 1) & 1) && now_cycles() - t0 < 200000000ll) {}
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------- MMA issuer -------------------------------
    bool ok = true;
    const uint32_t hi = (uint32_t)(make_smem_desc(0, 16) >> 32);
    const uint32_t lbo_k = (uint32_t)make_smem_desc(0, 16);            // k-contiguous operand
    const uint32_t lbo_mn1 = (uint32_t)make_smem_desc(0, 8192);        // rows = k, one 64-wide m/n block
    const uint32_t lbo_mn2 = (uint32_t)make_smem_desc(0, AT_TILE_BYTES);  // two 64-wide blocks 16 KB apart
    auto addr16 = [](uint32_t a) { return (a & 0x3FFFFu) >> 4; };
    auto mma_k128 = [&](uint32_t d_tmem, uint32_t a_lo, uint32_t a_kb, uint32_t a_ks, uint32_t b_lo,
                        uint32_t b_kb, uint32_t b_ks, uint32_t idesc) {  // contraction over 128 = 2 x 4 x 16
      uint32_t accum = 0;
#pragma unroll
      for (int kb = 0; kb < 2; kb++)
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const uint64_t ad = ((uint64_t)hi << 32) | (a_lo + kb * a_kb + k * a_ks);
          const uint64_t bd = ((uint64_t)hi << 32) | (b_lo + kb * b_kb + k * b_ks);
          tc_mma(d_tmem, ad, bd, idesc, accum);
          accum = 1;
        }
    };
    constexpr uint32_t KS_K = UMMA_K * 2 / 16;      // 16 k values of a k-contiguous tile, in 16-byte units
    constexpr uint32_t KS_MN = UMMA_K * 128 / 16;   // 16 k rows of a row-is-k tile
    constexpr uint32_t KB_MN = 8192 / 16;           // 64 k rows
    constexpr uint32_t KB_K = AT_TILE_BYTES / 16;   // next 64-wide k block of a two-tile operand
    auto second_products = [&](int j) {  // dQ = dS K and dK = dS^T Q of item j
      const uint32_t g = (uint32_t)j & 1;
      const uint32_t base = smem_u32(smem + (size_t)g * AB_STAGE_BYTES);
      const uint32_t ds = addr16(base + 4 * AT_TILE_BYTES);
      const uint32_t acc = tmem_base + g * AB_GROUP_COLS;
      mma_k128(acc, lbo_k | ds, KB_K, KS_K, lbo_mn1 | addr16(base + AT_TILE_BYTES), KB_MN, KS_MN, p.idesc_dq);
      mma_k128(acc + 64, lbo_mn2 | ds, KB_MN, KS_MN, lbo_mn1 | addr16(base), KB_MN, KS_MN, p.idesc_dk);
      tc_commit(smem_u32(&gfull_bar[g]));
      tc_commit(smem_u32(&empty_bar[g]));
    };
    for (int i = 0; i < n_my && ok; i++) {
      const uint32_t g = (uint32_t)i & 1, use = (uint32_t)i >> 1;
      if (!mbar_wait(smem_u32(&full_bar[g]), use & 1, abort_flag, p.status)) { ok = false; break; }
      if (!mbar_wait(smem_u32(&accfree_bar[g]), (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      const uint32_t base = smem_u32(smem + (size_t)g * AB_STAGE_BYTES);
      const uint32_t acc = tmem_base + g * AB_GROUP_COLS;
      const uint32_t dc = addr16(base + 3 * AT_TILE_BYTES);
      // dV = P^T dC: both operands with rows = query index = k
      mma_k128(acc + 128, lbo_mn2 | addr16(base + 4 * AT_TILE_BYTES), KB_MN, KS_MN, lbo_mn1 | dc, KB_MN, KS_MN,
               p.idesc_dv);
      // dP = dC V^T: both operands k-contiguous, contraction over the head width
#pragma unroll
      for (int k = 0; k < 4; k++) {
        const uint64_t ad = ((uint64_t)hi << 32) | ((lbo_k | dc) + k * KS_K);
        const uint64_t bd = ((uint64_t)hi << 32) | ((lbo_k | addr16(base + 2 * AT_TILE_BYTES)) + k * KS_K);
        tc_mma(acc, ad, bd, p.idesc_dp, k > 0 ? 1u : 0u);
      }
      tc_commit(smem_u32(&dpfull_bar[g]));
      if (i > 0) {
        const uint32_t g1 = (uint32_t)(i - 1) & 1, use1 = (uint32_t)(i - 1) >> 1;
        if (!mbar_wait(smem_u32(&dsready_bar[g1]), use1 & 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        second_products(i - 1);
      }
    }
    if (ok && n_my > 0) {
      const uint32_t g1 = (uint32_t)(n_my - 1) & 1, use1 = (uint32_t)(n_my - 1) >> 1;
      if (mbar_wait(smem_u32(&dsready_bar[g1]), use1 & 1, abort_flag, p.status)) {
        tc_fence_after();
        second_products(n_my - 1);
      } else {
        ok = false;
      }
    }
    if (!ok || *abort_flag) {
      tc_commit(smem_u32(&dpfull_bar[0]));
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < 2000000ll) {}
    }
  } else if (warp >= 2) {
    // ------------------------------- softmax-backward groups -------------------------------
    const int q = warp & 3;
    const int g = (warp - 2) >> 2;
    uint8_t* stg = staging + (size_t)(warp - 2) * AT_STAGING;
    const int r = q * 32 + lane;
    bool ok = true;
    for (int i = g; i < n_my && ok; i += 2) {
      const int w = (int)blockIdx.x + i * (int)gridDim.x;
      const int zo = w / p.heads, zi = w - zo * p.heads;
      const uint32_t use = (uint32_t)i >> 1;
      if (!mbar_wait(smem_u32(&dpfull_bar[g]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      float2 v[4][16];  // row r of dP
      const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)g * AB_GROUP_COLS;
#pragma unroll
      for (int c = 0; c < 4; c++) tc_ld32(trow + c * 32, v[c]);
      // row r of P (and then of dS): two 128-byte halves, 16-byte pieces permuted by r mod 8
      uint8_t* prow = smem + (size_t)g * AB_STAGE_BYTES + 4 * AT_TILE_BYTES + r * 128;
      float2 dl[4];
#pragma unroll
      for (int c = 0; c < 4; c++) {
        dl[c] = make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 4; j++) {
          const uint4 pk = *reinterpret_cast<const uint4*>(prow + (c >> 1) * AT_TILE_BYTES +
                                                           ((((c & 1) * 4 + j) ^ (r & 7)) << 4));
          dl[c] = __ffma2_rn(v[c][4 * j], bf162_to_f2(pk.x), dl[c]);
          dl[c] = __ffma2_rn(v[c][4 * j + 1], bf162_to_f2(pk.y), dl[c]);
          dl[c] = __ffma2_rn(v[c][4 * j + 2], bf162_to_f2(pk.z), dl[c]);
          dl[c] = __ffma2_rn(v[c][4 * j + 3], bf162_to_f2(pk.w), dl[c]);
        }
      }
      const float delta = ((dl[0].x + dl[0].y) + (dl[1].x + dl[1].y)) + ((dl[2].x + dl[2].y) + (dl[3].x + dl[3].y));
      const float2 nd = splat2(-delta), sc2 = splat2(p.scale);
#pragma unroll
      for (int c = 0; c < 4; c++) {
#pragma unroll
        for (int j = 0; j < 4; j++) {
          uint8_t* piece = prow + (c >> 1) * AT_TILE_BYTES + ((((c & 1) * 4 + j) ^ (r & 7)) << 4);
          const uint4 pk = *reinterpret_cast<const uint4*>(piece);
          const uint32_t pw[4] = {pk.x, pk.y, pk.z, pk.w};
          uint4 out;
          __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
          for (int e = 0; e < 4; e++) {
            const float2 t = __fmul2_rn(__fadd2_rn(v[c][4 * j + e], nd), sc2);
            h[e] = __float22bfloat162_rn(__fmul2_rn(t, bf162_to_f2(pw[e])));
          }
          *reinterpret_cast<uint4*>(piece) = out;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&dsready_bar[g]));
      bf16* gq = p.dQKV + zo * p.g_bo + zi * 64;
      // dV (complete since dP was): key r, 64 columns
      tc_ld32(trow + 128, v[0]);
      tc_ld32(trow + 160, v[1]);
      if (p.fast) {
        if (r < p.S) {
          store_row32_bf16(gq + 2 * p.H + (long long)r * p.g_ld, v[0]);
          store_row32_bf16(gq + 2 * p.H + (long long)r * p.g_ld + 32, v[1]);
        }
      } else {
        stage_store_bf16(stg, lane, v[0], gq + 2 * p.H, p.g_ld, q * 32, 0, p.S, 64, p.vec_ok);
        stage_store_bf16(stg, lane, v[1], gq + 2 * p.H, p.g_ld, q * 32, 32, p.S, 64, p.vec_ok);
      }
      if (!mbar_wait(smem_u32(&gfull_bar[g]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; c++) tc_ld32(trow + c * 32, v[c]);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&accfree_bar[g]));
      if (p.fast) {
        if (r < p.S) {
          bf16* row = gq + (long long)r * p.g_ld;
          store_row32_bf16(row, v[0]);
          store_row32_bf16(row + 32, v[1]);
          store_row32_bf16(row + p.H, v[2]);
          store_row32_bf16(row + p.H + 32, v[3]);
        }
      } else {
        stage_store_bf16(stg, lane, v[0], gq, p.g_ld, q * 32, 0, p.S, 64, p.vec_ok);
        stage_store_bf16(stg, lane, v[1], gq, p.g_ld, q * 32, 32, p.S, 64, p.vec_ok);
        stage_store_bf16(stg, lane, v[2], gq + p.H, p.g_ld, q * 32, 0, p.S, 64, p.vec_ok);
        stage_store_bf16(stg, lane, v[3], gq + p.H, p.g_ld, q * 32, 32, p.S, 64, p.vec_ok);
      }
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
static std::atomic<int> g_attn_starve{0};
void attn_starve_next(int on) { g_attn_starve.store(on ? 1 : 0); }
long long attn_launches() { return g_attn_launches.load(); }

namespace {
// per-device facts and one-time kernel attributes (a process may drive several GPUs)
struct AttnDevice {
  int num_sms = 0, smem_optin = 0;
  bool attr_fwd = false, attr_long = false, attr_bwd = false;
};
constexpr int kMaxDevices = 64;
AttnDevice g_adev[kMaxDevices];
std::mutex g_adev_mu;
AttnDevice* attn_device(char* err) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    snprintf(err, 256, "attention: no CUDA device");
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_adev_mu);
  AttnDevice& a = g_adev[dev];
  if (a.num_sms == 0) {
    cudaDeviceGetAttribute(&a.num_sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&a.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (a.num_sms <= 0) { snprintf(err, 256, "attention: no CUDA device"); return nullptr; }
  }
  return &a;
}
// opts a kernel in to the large dynamic shared memory size once per device
template <typename K>
int attn_opt_in(K kernel, bool* done, int smem_optin, char* err) {
  std::lock_guard<std::mutex> lock(g_adev_mu);
  if (*done) return 0;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
  if (e != cudaSuccess) { snprintf(err, 256, "attention: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
  *done = true;
  return 0;
}
}  // namespace

int attn_fwd_launch(const void* qkv, void* probs, void* ctx, const int* seq_lens, int B, int S, int A, int d,
                    float scale, int* status, cudaStream_t st, char* err) {
  // the test hook is used up by this call even if an argument check below rejects it
  const bool starve = g_attn_starve.exchange(0) != 0;
  AttnDevice* adev = attn_device(err);
  if (!adev) return MSLT_ERR_CUDA;
  const int num_sms = adev->num_sms, smem_optin = adev->smem_optin;
  if (d != 64 || S < 1 || S > 512 || B < 1 || A < 1 || !status) {
    snprintf(err, 256, "attention: the fused kernel needs head width 64 and 1 <= S <= 512");
    return MSLT_ERR_ARG;
  }
  const bool long_rows = S > 128;  // several key blocks per row: the two-pass kernel
  const long long H = (long long)A * d;
  AttnParams p;
  memset(&p, 0, sizeof(p));
  p.S = S; p.heads = A; p.items = B * A * (long_rows ? (S + 127) / 128 : 1); p.scale = scale; p.seq_lens = seq_lens;
  p.P = (bf16*)probs; p.p_bo = (long long)A * S * S; p.p_bi = (long long)S * S;
  p.C = (bf16*)ctx; p.c_ld = H; p.c_bo = (long long)S * H; p.c_bi = d;
  p.vec_ok_p = (S % 8 == 0 && ((uintptr_t)probs & 15) == 0) ? 1 : 0;
  p.vec_ok_c = (H % 8 == 0 && ((uintptr_t)ctx & 15) == 0) ? 1 : 0;
  p.fast_c = row_fast(ctx, H);
  p.fast_p = (probs != nullptr && S % 32 == 0) ? row_fast(probs, S) : 0;
  p.wait_limit = WAIT_LIMIT_CYCLES;
  p.status = status;
  if (starve) {  // armed by mslt_debug_starve_next_attention
    p.starve = 1;
    p.wait_limit = 40000000ll;  // about 20 ms
  }
  // fp32 accumulate, bf16 x bf16; scores: both operands k-contiguous, N = 128; context: V row-contiguous, N = 64
  p.idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  p.idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
  const bf16* base = (const bf16*)qkv;
  MapVal mq, mk, mv;
  int rc = get_map(base, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mq, err);
  if (rc) return rc;
  rc = get_map(base + H, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mk, err);
  if (rc) return rc;
  // V: the short kernel reads it as two boxes of 64 keys with the head width contiguous; the long
  // one as one box of 128 key rows, which are the same bytes in shared memory
  if (long_rows) rc = get_map(base + 2 * H, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mv, err);
  else rc = get_map(base + 2 * H, d, S, 1, 3 * H, (long long)S * 3 * H, d, A, B, 64, &mv, err);
  if (rc) return rc;
  for (int i = 0; i < 3; i++) { p.q_perm[i] = mq.perm[i]; p.k_perm[i] = mk.perm[i]; p.v_perm[i] = mv.perm[i]; }
  if (long_rows) {
    const size_t smem_long = 2 * (size_t)AT_TILE_BYTES + 2 * (size_t)AL_RING * AT_TILE_BYTES + 2 * (size_t)AL_P_BYTES +
                             NUM_EPI_WARPS * AT_STAGING + 1024 + 512;
    if ((int)smem_long > smem_optin) { snprintf(err, 256, "attention: not enough shared memory"); return MSLT_ERR_CUDA; }
    rc = attn_opt_in(attn_fwd_long_kernel, &adev->attr_long, smem_optin, err);
    if (rc) return rc;
    const int grid_long = p.items < num_sms ? p.items : num_sms;
    attn_fwd_long_kernel<<<grid_long, AL_THREADS, smem_long, st>>>(mq.map, mk.map, mv.map, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { snprintf(err, 256, "attention: launch failed: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
    g_attn_launches++;
    return 0;
  }
  const size_t smem_bytes = (size_t)AT_STAGES * AT_STAGE_BYTES + NUM_EPI_WARPS * AT_STAGING + 1024 + 256;
  if ((int)smem_bytes > smem_optin) { snprintf(err, 256, "attention: not enough shared memory"); return MSLT_ERR_CUDA; }
  rc = attn_opt_in(attn_fwd_kernel, &adev->attr_fwd, smem_optin, err);
  if (rc) return rc;
  const int grid = p.items < num_sms ? p.items : num_sms;
  attn_fwd_kernel<<<grid, NUM_THREADS, smem_bytes, st>>>(mq.map, mk.map, mv.map, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { snprintf(err, 256, "attention: launch failed: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
  g_attn_launches++;
  return 0;
}

int attn_bwd_launch(const void* qkv, const void* probs, const void* dctx, void* dqkv, int B, int S, int A, int d,
                    float scale, int* status, cudaStream_t st, char* err) {
  // the test hook is used up by this call even if an argument check below rejects it
  const bool starve = g_attn_starve.exchange(0) != 0;
  AttnDevice* adev = attn_device(err);
  if (!adev) return MSLT_ERR_CUDA;
  const int num_sms = adev->num_sms, smem_optin = adev->smem_optin;
  if (d != 64 || S < 8 || S > 128 || S % 8 || B < 1 || A < 1 || !status || !qkv || !probs || !dctx || !dqkv) {
    snprintf(err, 256, "attention backward: the fused kernel needs head width 64 and S a multiple of 8 in [8, 128]");
    return MSLT_ERR_ARG;
  }
  const long long H = (long long)A * d;
  AttnBwdParams p;
  memset(&p, 0, sizeof(p));
  p.S = S; p.heads = A; p.items = B * A; p.scale = scale;
  p.dQKV = (bf16*)dqkv; p.g_ld = 3 * H; p.g_bo = (long long)S * 3 * H; p.H = H;
  p.vec_ok = ((uintptr_t)dqkv & 15) == 0 ? 1 : 0;
  p.fast = 0;  // direct 32-byte row stores measured slower here (58 vs 54 us): three 128-byte pieces per row
  p.wait_limit = WAIT_LIMIT_CYCLES;
  p.status = status;
  if (starve) {  // armed by mslt_debug_starve_next_attention
    p.starve = 1;
    p.wait_limit = 40000000ll;  // about 20 ms
  }
  // fp32 accumulate, bf16 x bf16, M = 128; bit 15 / 16: A / B operand with rows = k index
  const uint32_t common = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BM >> 4) << 24);
  p.idesc_dv = common | (1u << 15) | (1u << 16) | ((uint32_t)(64 >> 3) << 17);
  p.idesc_dp = common | ((uint32_t)(128 >> 3) << 17);
  p.idesc_dq = common | (1u << 16) | ((uint32_t)(64 >> 3) << 17);
  p.idesc_dk = common | (1u << 15) | (1u << 16) | ((uint32_t)(64 >> 3) << 17);
  const bf16* base = (const bf16*)qkv;
  MapVal mq, mk, mv, mc, mp;
  int rc = get_map(base, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mq, err);
  if (rc) return rc;
  rc = get_map(base + H, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mk, err);
  if (rc) return rc;
  rc = get_map(base + 2 * H, S, d, 3 * H, 1, (long long)S * 3 * H, d, A, B, BM, &mv, err);
  if (rc) return rc;
  rc = get_map(dctx, S, d, H, 1, (long long)S * H, d, A, B, BM, &mc, err);
  if (rc) return rc;
  rc = get_map(probs, S, S, S, 1, (long long)A * S * S, (long long)S * S, A, B, BM, &mp, err);
  if (rc) return rc;
  for (int i = 0; i < 3; i++) {
    p.q_perm[i] = mq.perm[i]; p.k_perm[i] = mk.perm[i]; p.v_perm[i] = mv.perm[i];
    p.c_perm[i] = mc.perm[i]; p.p_perm[i] = mp.perm[i];
  }
  const size_t smem_bytes = (size_t)2 * AB_STAGE_BYTES + NUM_EPI_WARPS * AT_STAGING + 1024 + 256;
  if ((int)smem_bytes > smem_optin) { snprintf(err, 256, "attention: not enough shared memory"); return MSLT_ERR_CUDA; }
  rc = attn_opt_in(attn_bwd_kernel, &adev->attr_bwd, smem_optin, err);
  if (rc) return rc;
  const int grid = p.items < num_sms ? p.items : num_sms;
  attn_bwd_kernel<<<grid, NUM_THREADS, smem_bytes, st>>>(mq.map, mk.map, mv.map, mc.map, mp.map, p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) { snprintf(err, 256, "attention: launch failed: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
  g_attn_launches++;
  return 0;
}

}  // namespace mslt
