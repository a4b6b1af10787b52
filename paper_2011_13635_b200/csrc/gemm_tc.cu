// bf16 dense contraction on the 5th-generation tensor cores (sm_100a):
//   D[z][m][n] = epilogue(alpha * sum_k A[z](m,k) * B[z](n,k)),  fp32 accumulation in TMEM.
//
// One persistent CTA per SM walks a list of (split, batch, m-tile, n-tile) work items.
//   warps 0, 2, 3: TMA producers (one thread each).  128-byte-swizzled operand tiles go global ->
//              shared through a ring of stages, each guarded by a full/empty mbarrier pair.  The
//              k blocks are dealt out round robin: measured on B200, one thread needs about 560
//              cycles for {wait, expect_tx, two tile copies} however small the tiles are, more than
//              the 512 cycles the tensor core takes for a 128 x 256 x 64 block, while several
//              threads in different warps issue side by side at the same per-thread cost.
//   warp 1   : allocates tensor memory and issues tcgen05.mma (one thread) for 128 x BN x 16
//              steps; tcgen05.commit hands shared-memory stages back to the producers and
//              accumulators over to the epilogue.
//   warps 4-11: epilogue.  Two warps per 32-lane quarter of TMEM read the accumulator with
//              tcgen05.ld, apply scale, bias, GELU / GELU', residual, and store bf16 or fp32
//              (plain, or as vector reductions for split-k) through a swizzled staging buffer so
//              that global stores are whole row segments.  Two accumulators of up to 256 columns
//              let the epilogue of one tile overlap the main loop of the next.
// Operands may be k-contiguous ("K-major") or row-contiguous ("MN-major"); the second form is
// what input-gradient and weight-gradient products need, and is fed to the tensor cores through
// the MN-major shared-memory descriptor, so no transposed copies exist anywhere.
// Every wait is bounded: when one runs out the CTA raises a status bit, drains and returns.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <string>
#include <unordered_map>

#include "gemm.h"
#include "tc_common.cuh"

namespace mslt {

namespace {

constexpr int NUM_PRODUCERS = 3;                              // warps 0, 2, 3
constexpr int FIRST_EPI_WARP = 4;                             // warps 4..11 (warp & 3 = TMEM lane quarter)
constexpr int GEMM_THREADS = 32 * (FIRST_EPI_WARP + NUM_EPI_WARPS);

struct TcParams {
  int M, N, K, batch, hdiv;
  int bn, stages, a_mn, b_mn;
  int m_tiles, n_tiles, splits, kb_total, kb_per_split, total_work;
  int a_perm[3], b_perm[3];  // slot (1..3) of the (outer, inner-batch, outer-batch) coordinates
  char* D;
  long long ldd, d_bo, d_bi;
  int d_fp32, accumulate, vec_ok;
  int direct;           // rows of D (and aux) may be stored straight from registers, 32 bytes at a time
  int tma_store;        // bf16 D leaves through shared memory and tile stores of 32 rows x 64 columns
  int d_perm[3];        // slots of D's (row, inner-batch, outer-batch) coordinates in its tensor map
  float alpha;
  const float* bias;
  int act;
  bf16* aux;
  const bf16* residual;
  const int* seq_lens;  // act 3: valid keys per outer batch index, or null
  long long wait_limit; // SM cycles a wait may take before the CTA gives up
  int starve;           // test hook: the producer issues no copies, so the first wait runs out
  int* status;
  uint32_t idesc;
};

// GELU on the FMA pipe only: the epilogue of a GELU tile is bound by the special-function unit when
// erf costs a reciprocal and an exponential per element, and by instruction issue after that, so
// the polynomials below run on the packed two-wide fp32 instructions (fma.rn.f32x2), two columns
// per instruction.  gelu(u) = u * Phi(u) with Phi(u) - 1/2 = u * Q(u^2), Q a degree-8
// least-maximum-error fit on |u| <= 4 (gelu is off by less than 3e-5 in fp32 there, far inside bf16
// resolution).  Outside, u^2 is clamped to 16 and Phi saturates to [0, 1], which gives gelu(u) = u
// above and 0 below (the exact values differ from those by less than 2e-4).
__device__ __forceinline__ float2 gelu_fast2(float2 u) {
  float2 t = __fmul2_rn(u, u);
  t.x = fminf(t.x, 16.0f);
  t.y = fminf(t.y, 16.0f);
  float2 q = splat2(8.093845117e-11f);
  q = __ffma2_rn(q, t, splat2(-7.032516570e-09f));
  q = __ffma2_rn(q, t, splat2(2.727248615e-07f));
  q = __ffma2_rn(q, t, splat2(-6.317188128e-06f));
  q = __ffma2_rn(q, t, splat2(9.916073864e-05f));
  q = __ffma2_rn(q, t, splat2(-1.135572678e-03f));
  q = __ffma2_rn(q, t, splat2(9.883344319e-03f));
  q = __ffma2_rn(q, t, splat2(-6.642043264e-02f));
  q = __ffma2_rn(q, t, splat2(3.989280708e-01f));
  float2 phi;
  phi.x = __saturatef(fmaf(q.x, u.x, 0.5f));
  phi.y = __saturatef(fmaf(q.y, u.y, 0.5f));
  return __fmul2_rn(u, phi);
}
// GELU'(u) = Phi(u) + u phi(u), also on the FMA pipe: 0.5 + u * P(u^2) with a degree-17 odd
// least-maximum-error fit on |u| <= 4 (absolute error below 1e-4); beyond that the derivative is
// 0 or 1 to within 5e-4.  The result multiplies a gradient that is then rounded to bf16.
__device__ __forceinline__ float2 gelu_grad_fast2(float2 u) {
  const float2 t = __fmul2_rn(u, u);
  float2 p = splat2(9.837601957e-10f);
  p = __ffma2_rn(p, t, splat2(-8.257008028e-08f));
  p = __ffma2_rn(p, t, splat2(3.042579986e-06f));
  p = __ffma2_rn(p, t, splat2(-6.523749948e-05f));
  p = __ffma2_rn(p, t, splat2(9.104776309e-04f));
  p = __ffma2_rn(p, t, splat2(-8.736754371e-03f));
  p = __ffma2_rn(p, t, splat2(5.852845753e-02f));
  p = __ffma2_rn(p, t, splat2(-2.649477277e-01f));
  p = __ffma2_rn(p, t, splat2(7.976755055e-01f));
  p = __ffma2_rn(p, u, splat2(0.5f));
  // step(u) without a second comparison: u * 2^100 saturated to [0, 1]
  p.x = fabsf(u.x) >= 4.0f ? __saturatef(u.x * 1.2676506e30f) : p.x;
  p.y = fabsf(u.y) >= 4.0f ? __saturatef(u.y * 1.2676506e30f) : p.y;
  return p;
}
// Epilogue flavours.  Each is its own kernel instantiation: one kernel with every flavour behind
// run-time branches measured 2-3x slower per chunk (register pressure and jumps across large code
// blocks), which made shallow contractions wait for their epilogue.
enum : int {
  EPI_STORE = 0,   // bf16 out = alpha * acc + bias
  EPI_RESIDUAL,    // bf16 out = alpha * acc + bias + residual row
  EPI_GELU,        // bf16 out = gelu(alpha * acc + bias)
  EPI_GELU_AUX,    // the same, and the pre-activation goes to aux
  EPI_DGELU,       // bf16 out = (alpha * acc + bias) * gelu'(aux)
  EPI_F32,         // fp32 out (stored, or added to what is there) = alpha * acc + bias
  EPI_GENERIC,     // every other combination the descriptor allows, and unaligned buffers
  EPI_SOFTMAX,     // masked row softmax (its own epilogue)
  EPI_COUNT
};

// A lane that owns a row stores 32 of its columns without a trip through shared memory: two
// 32-byte stores for bf16 (every store fills a whole sector), four for fp32, or eight 16-byte
// vector reductions when partial sums are added.  dst must be 32-byte aligned.
__device__ __forceinline__ void row32_store_bf16(bf16* dst, const float2 (&w)[16]) {
  uint32_t h[16];
#pragma unroll
  for (int e = 0; e < 16; e++) {
    const __nv_bfloat162 t = __float22bfloat162_rn(w[e]);
    h[e] = *reinterpret_cast<const uint32_t*>(&t);
  }
#pragma unroll
  for (int c = 0; c < 2; c++)
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 16 * c), "r"(h[8 * c]),
                 "r"(h[8 * c + 1]), "r"(h[8 * c + 2]), "r"(h[8 * c + 3]), "r"(h[8 * c + 4]), "r"(h[8 * c + 5]),
                 "r"(h[8 * c + 6]), "r"(h[8 * c + 7])
                 : "memory");
}
// The same 32 columns into a 32-row x 128-byte staging tile in the 128-byte swizzle layout of the
// output's tensor map: row `lane`, 16-byte units 4 * half .. 4 * half + 3, unit u stored at
// position u ^ (row & 7).  Eight neighbouring lanes hit eight different bank groups.
__device__ __forceinline__ void row32_stage_bf16(uint32_t tile, int lane, int half, const float2 (&w)[16]) {
  uint32_t h[16];
#pragma unroll
  for (int e = 0; e < 16; e++) {
    const __nv_bfloat162 t = __float22bfloat162_rn(w[e]);
    h[e] = *reinterpret_cast<const uint32_t*>(&t);
  }
  const uint32_t row = tile + (uint32_t)lane * 128u;
#pragma unroll
  for (int c = 0; c < 4; c++) {
    const uint32_t u = (uint32_t)((4 * half + c) ^ (lane & 7));
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + u * 16u), "r"(h[4 * c]), "r"(h[4 * c + 1]),
                 "r"(h[4 * c + 2]), "r"(h[4 * c + 3])
                 : "memory");
  }
}
__device__ __forceinline__ void row32_store_f32(float* dst, const float2 (&w)[16], int accumulate) {
  if (accumulate) {
#pragma unroll
    for (int c = 0; c < 8; c++)
      asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4 * c), "f"(w[2 * c].x), "f"(w[2 * c].y),
                   "f"(w[2 * c + 1].x), "f"(w[2 * c + 1].y)
                   : "memory");
  } else {
#pragma unroll
    for (int c = 0; c < 4; c++)
      asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + 8 * c), "f"(w[4 * c].x),
                   "f"(w[4 * c].y), "f"(w[4 * c + 1].x), "f"(w[4 * c + 1].y), "f"(w[4 * c + 2].x), "f"(w[4 * c + 2].y),
                   "f"(w[4 * c + 3].x), "f"(w[4 * c + 3].y)
                   : "memory");
  }
}

// One 32 x 32 chunk of a specialised flavour: a = this lane's 32 accumulator columns, bias_c = the
// chunk's bias values in shared memory (zeros without a bias), x = this lane's 32 bf16 values of
// the row-shaped extra operand (EPI_RESIDUAL, EPI_DGELU).
// `direct`: this lane's row exists and the whole chunk lies inside the output, so the lane stores
// its 32 columns itself; otherwise the chunk goes through the staging buffer, which handles ragged
// edges element by element (every lane of the warp takes the same branch).
// `tile` != 0: the bf16 result goes into that staging tile (shared-memory address) as half `half`
// of its 64 columns instead, for a tile store by the caller.
template <int kMode>
__device__ __forceinline__ void epi_chunk(const TcParams& p, const uint32_t (&a)[32], const uint4 (&x)[4],
                                          const float* bias_c, uint8_t* stg, int lane, long long zoff,
                                          int m_warp, int n0, bool direct, uint32_t tile = 0, int half = 0) {
  float2 v[16];
  const float2 al = splat2(p.alpha);
  const float4* b4 = reinterpret_cast<const float4*>(bias_c);
#pragma unroll
  for (int j = 0; j < 8; j++) {
    const float4 t = b4[j];
    v[2 * j] = __ffma2_rn(make_float2(__uint_as_float(a[4 * j]), __uint_as_float(a[4 * j + 1])), al,
                          make_float2(t.x, t.y));
    v[2 * j + 1] = __ffma2_rn(make_float2(__uint_as_float(a[4 * j + 2]), __uint_as_float(a[4 * j + 3])), al,
                              make_float2(t.z, t.w));
  }
  const bool row_ok = m_warp + lane < p.M;
  const long long off = zoff + (long long)(m_warp + lane) * p.ldd + n0;
  if constexpr (kMode == EPI_GELU_AUX) {
    if (direct) { if (row_ok) row32_store_bf16(p.aux + off, v); }
    else stage_store_bf16(stg, lane, v, p.aux + zoff, p.ldd, m_warp, n0, p.M, p.N, p.vec_ok);
  }
  if constexpr (kMode == EPI_GELU || kMode == EPI_GELU_AUX) {
#pragma unroll
    for (int j = 0; j < 16; j++) v[j] = gelu_fast2(v[j]);
  }
  if constexpr (kMode == EPI_DGELU) {
#pragma unroll
    for (int j = 0; j < 4; j++) {
      v[4 * j] = __fmul2_rn(v[4 * j], gelu_grad_fast2(bf162_to_f2(x[j].x)));
      v[4 * j + 1] = __fmul2_rn(v[4 * j + 1], gelu_grad_fast2(bf162_to_f2(x[j].y)));
      v[4 * j + 2] = __fmul2_rn(v[4 * j + 2], gelu_grad_fast2(bf162_to_f2(x[j].z)));
      v[4 * j + 3] = __fmul2_rn(v[4 * j + 3], gelu_grad_fast2(bf162_to_f2(x[j].w)));
    }
  }
  if constexpr (kMode == EPI_RESIDUAL) {
#pragma unroll
    for (int j = 0; j < 4; j++) {
      v[4 * j] = __fadd2_rn(v[4 * j], bf162_to_f2(x[j].x));
      v[4 * j + 1] = __fadd2_rn(v[4 * j + 1], bf162_to_f2(x[j].y));
      v[4 * j + 2] = __fadd2_rn(v[4 * j + 2], bf162_to_f2(x[j].z));
      v[4 * j + 3] = __fadd2_rn(v[4 * j + 3], bf162_to_f2(x[j].w));
    }
  }
  if constexpr (kMode == EPI_F32) {
    if (direct) { if (row_ok) row32_store_f32(reinterpret_cast<float*>(p.D) + off, v, p.accumulate); }
    else stage_store_f32(stg, lane, v, reinterpret_cast<float*>(p.D) + zoff, p.ldd, m_warp, n0, p.M, p.N, p.vec_ok,
                         p.accumulate);
  } else {
    if (tile) row32_stage_bf16(tile, lane, half, v);
    else if (direct) { if (row_ok) row32_store_bf16(reinterpret_cast<bf16*>(p.D) + off, v); }
    else stage_store_bf16(stg, lane, v, reinterpret_cast<bf16*>(p.D) + zoff, p.ldd, m_warp, n0, p.M, p.N, p.vec_ok);
  }
}

// ---- the kernel ---------------------------------------------------------------------------------
// 12 warps: a thread may use up to 168 registers
template <int kMode, bool kPair>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmD, const TcParams p) {
  constexpr bool kSoftmax = kMode == EPI_SOFTMAX;
  constexpr bool kHasX = kMode == EPI_RESIDUAL || kMode == EPI_DGELU;
  extern __shared__ uint8_t smem_raw[];
  // tiles need 1024-byte alignment for the 128-byte swizzle pattern
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  // CTA-pair mode: the two CTAs of a cluster share one 256 x 256 tile.  Each loads its own 128
  // rows of A and its own 128 columns of B; the leader (rank 0) issues MMAs that read both CTAs'
  // shared memory and write both CTAs' tensor memory.
  const uint32_t cta_rank = kPair ? cluster_ctarank() : 0u;
  const bool leader = cta_rank == 0;
  const int bn_cta = kPair ? p.bn / 2 : p.bn;   // B columns held by this CTA
  const int mt_rows = kPair ? 2 * BM : BM;      // rows of a work item's output tile
  const int w_first = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int w_step = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  // A ring stage holds KSUB 64-deep k blocks of both operands ("a round").  The issuing thread
  // spends a fixed ~250-350 cycles per round on its barrier hand-shakes whatever the round holds;
  // with four MMAs (512 cycles of tensor-core work) per round that kept the tensor core waiting,
  // with eight it does not.  The pair form has the shared memory for three such stages.
  constexpr int KSUB = kPair ? 2 : 1;
  const int b_stage_bytes = bn_cta * BK * 2;
  const int sub_bytes = A_STAGE_BYTES + b_stage_bytes;
  const int stage_bytes = KSUB * sub_bytes;
  uint8_t* staging = smem + (size_t)p.stages * stage_bytes;
  uint64_t* bars = (uint64_t*)(staging + NUM_EPI_WARPS * STAGING_BYTES);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + MAX_STAGES;
  uint64_t* tfull_bar = bars + 2 * MAX_STAGES;
  uint64_t* tempty_bar = bars + 2 * MAX_STAGES + 2;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * MAX_STAGES + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  // softmax epilogue only: hand-over flags and per-row partial results of the two warps of a quarter
  volatile int* xflag = (volatile int*)((uint8_t*)bars + 256);
  float* xmax = (float*)((uint8_t*)bars + 256 + 64);
  float* xsum = xmax + NUM_EPI_WARPS * 32;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; s++) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int a = 0; a < 2; a++) {
      mbar_init(smem_u32(&tfull_bar[a]), 1);
      mbar_init(smem_u32(&tempty_bar[a]), kPair ? 2 * NUM_EPI_WARPS : NUM_EPI_WARPS);
    }
    *abort_flag = 0;
    *reinterpret_cast<volatile long long*>(abort_flag + 1) = p.wait_limit;  // read by every bounded wait
    if (kSoftmax)
      for (int i = 0; i < NUM_EPI_WARPS; i++) xflag[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();  // the peer's barriers must exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int tiles_per_z = p.m_tiles * p.n_tiles;
  const int per_split = tiles_per_z * p.batch;

  if ((warp == 0 || warp == 2 || warp == 3) && lane == 0 && !p.starve) {
    // ------------------------------- TMA producers -------------------------------
    // Producer j takes the k blocks whose running index is j modulo NUM_PRODUCERS.  Every producer
    // walks the whole work list (ring position as (stage, phase) counters, tile coordinates in
    // scalars) and issues only its own blocks.
    const uint32_t me = warp == 0 ? 0u : (uint32_t)warp - 1u;
    uint32_t it = 0, s = 0, ph = 0, turn = 0;
    uint32_t last_it = 0, mine = 0;
    bool ok = true;
    // which coordinate slot carries k: slot 0 for a k-contiguous operand, else the permuted one
    const int ak = p.a_mn ? p.a_perm[0] : 0, bk = p.b_mn ? p.b_perm[0] : 0;
    constexpr int RK = KSUB * BK;  // k extent of a round
    const int da0 = ak == 0 ? RK : 0, da1 = ak == 1 ? RK : 0, da2 = ak == 2 ? RK : 0, da3 = ak == 3 ? RK : 0;
    const int db0 = bk == 0 ? RK : 0, db1 = bk == 1 ? RK : 0, db2 = bk == 2 ? RK : 0, db3 = bk == 3 ? RK : 0;
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
    const uint32_t tx_bytes = kPair ? 2 * stage_bytes : stage_bytes;
    const int a_boxes = p.a_mn ? BM / 64 : 1, b_boxes = p.b_mn ? bn_cta / 64 : 1;
    for (int w = w_first; w < p.total_work && ok; w += w_step) {
      const int split = w / per_split;
      int r = w - split * per_split;
      const int z = r / tiles_per_z;
      r -= z * tiles_per_z;
      const int mt = r / p.n_tiles, nt = r - mt * p.n_tiles;
      const int zo = z / p.hdiv, zi = z - zo * p.hdiv;
      const int kb0 = split * p.kb_per_split;
      const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
      const int row0 = mt * mt_rows + (int)cta_rank * BM;
      const int col0 = nt * p.bn + (int)cta_rank * bn_cta;
      int ca[4], cb[4];
      if (!p.a_mn) { ca[0] = kb0 * RK; ca[p.a_perm[0]] = row0; }
      else         { ca[0] = row0; ca[p.a_perm[0]] = kb0 * RK; }
      ca[p.a_perm[1]] = zi; ca[p.a_perm[2]] = zo;
      if (!p.b_mn) { cb[0] = kb0 * RK; cb[p.b_perm[0]] = col0; }
      else         { cb[0] = col0; cb[p.b_perm[0]] = kb0 * RK; }
      cb[p.b_perm[1]] = zi; cb[p.b_perm[2]] = zo;
      int a0 = ca[0], a1 = ca[1], a2 = ca[2], a3 = ca[3];
      int b0 = cb[0], b1 = cb[1], b2 = cb[2], b3 = cb[3];
      for (int kb = kb0; kb < kb1; kb++, it++) {
        if (turn == me) {
          if (!mbar_wait(empty0 + s * 8, ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t fb_own = full0 + s * 8;
          // pair mode: both CTAs' copies are counted on the leader's barrier
          const uint32_t fb = kPair ? mapa_u32(fb_own, 0) : fb_own;
          if (leader) mbar_expect_tx(fb_own, tx_bytes);
          // k-contiguous operand: one box {64 k, rows} per k block; row-contiguous: boxes {64 rows,
          // 64 k}.  A k block that starts at or beyond K is filled with zeros by the copy engine.
#pragma unroll
          for (int sub = 0; sub < KSUB; sub++) {
            const uint32_t sa = smem0 + s * (uint32_t)stage_bytes + sub * (uint32_t)sub_bytes;
            const uint32_t sb = sa + A_STAGE_BYTES;
            const int ko = sub * BK;
            const int x0 = a0 + (ak == 0 ? ko : 0), x1 = a1 + (ak == 1 ? ko : 0), x2 = a2 + (ak == 2 ? ko : 0),
                      x3 = a3 + (ak == 3 ? ko : 0);
            const int y0 = b0 + (bk == 0 ? ko : 0), y1 = b1 + (bk == 1 ? ko : 0), y2 = b2 + (bk == 2 ? ko : 0),
                      y3 = b3 + (bk == 3 ? ko : 0);
            for (int h = 0; h < a_boxes; h++) {
              if (kPair) tma_load_4d_pair(sa + h * (64 * BK * 2), &tmA, fb, x0 + (p.a_mn ? h * 64 : 0), x1, x2, x3);
              else tma_load_4d(sa + h * (64 * BK * 2), &tmA, fb, x0 + (p.a_mn ? h * 64 : 0), x1, x2, x3);
            }
            for (int h = 0; h < b_boxes; h++) {
              if (kPair) tma_load_4d_pair(sb + h * (64 * BK * 2), &tmB, fb, y0 + (p.b_mn ? h * 64 : 0), y1, y2, y3);
              else tma_load_4d(sb + h * (64 * BK * 2), &tmB, fb, y0 + (p.b_mn ? h * 64 : 0), y1, y2, y3);
            }
          }
          last_it = it;
          mine++;
        }
        a0 += da0; a1 += da1; a2 += da2; a3 += da3;
        b0 += db0; b1 += db1; b2 += db2; b3 += db3;
        if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1; }
        if (++turn == (uint32_t)NUM_PRODUCERS) turn = 0;
      }
    }
    if (!ok || *abort_flag) {
      // give up: let this thread's copies that may still be in flight land before the CTA leaves
      if (!leader) {  // its copies are counted on the leader's barriers: give them time to land
        const long long t0 = now_cycles();
        while (now_cycles() - t0 < 2000000ll) {}
      } else {
        for (uint32_t back = 0; back < mine && back * NUM_PRODUCERS < (uint32_t)p.stages; back++) {
          const uint32_t j = last_it - back * NUM_PRODUCERS;
          const uint32_t fb = smem_u32(&full_bar[j % p.stages]);
          const long long t0 = now_cycles();
          while (!mbar_try_wait(fb, (j / p.stages) & 1) && now_cycles() - t0 < 200000000ll) {}
        }
      }
    }
  } else if (warp == 1 && lane == 0 && leader) {
    // ------------------------------- MMA issuer -------------------------------
    // One thread feeds the tensor core, so its loop is kept short: ring position as counters,
    // descriptors as a constant high word plus a low word that only gains the stage and k offsets.
    uint32_t tile = 0, s = 0, ph = 0;
    bool ok = true;
    const uint32_t a_lbo = p.a_mn ? 64 * BK * 2 : 16;
    const uint32_t b_lbo = p.b_mn ? 64 * BK * 2 : 16;
    const uint32_t a_kstep = (p.a_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;  // 16-byte units per 16-wide k step
    const uint32_t b_kstep = (p.b_mn ? UMMA_K * 128 : UMMA_K * 2) >> 4;
    const uint64_t a_desc0 = make_smem_desc(smem_u32(smem), a_lbo);
    const uint64_t b_desc0 = make_smem_desc(smem_u32(smem) + A_STAGE_BYTES, b_lbo);
    const uint32_t a_hi = (uint32_t)(a_desc0 >> 32), b_hi = (uint32_t)(b_desc0 >> 32);
    const uint32_t a_lo0 = (uint32_t)a_desc0, b_lo0 = (uint32_t)b_desc0;
    const uint32_t stage_units = (uint32_t)stage_bytes >> 4, sub_units = (uint32_t)sub_bytes >> 4;
    const uint32_t full0 = smem_u32(&full_bar[0]), empty0 = smem_u32(&empty_bar[0]);
    // A wait on a barrier that another thread completed costs this thread about 250 cycles even
    // when the phase is long over, which alone would keep it from issuing a k block's four MMAs
    // within the 512 cycles they run.  So every wait is issued one step early, before the MMAs
    // of the current block, and its answer is only read afterwards: `ready` for the next ring
    // slot, `acc_free` for the next work item's accumulator.
    uint32_t ready = 0, acc_free = 0;
    for (int w = w_first; w < p.total_work && ok; w += w_step, tile++) {
      const int split = w / per_split;
      const int kb0 = split * p.kb_per_split;
      const int kb1 = min(p.kb_total, kb0 + p.kb_per_split);
      const uint32_t acc = tile & 1, use = tile >> 1;
      if (!acc_free && !mbar_wait(smem_u32(&tempty_bar[acc]), (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
      acc_free = 0;
      tc_fence_after();
      const uint32_t d_tmem = tmem_base + acc * 256;
      uint32_t accum = 0;
      for (int kb = kb0; kb < kb1; kb++) {
        if (!ready && !mbar_wait(full0 + s * 8, ph, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        uint32_t s1 = s + 1, ph1 = ph;
        if (s1 == (uint32_t)p.stages) { s1 = 0; ph1 ^= 1; }
        ready = mbar_try_wait(full0 + s1 * 8, ph1) ? 1u : 0u;
        if (kb == kb1 - 1 && w + w_step < p.total_work) {
          const uint32_t nt = tile + 1;
          acc_free = mbar_try_wait(smem_u32(&tempty_bar[nt & 1]), ((nt >> 1) & 1) ^ 1) ? 1u : 0u;
        }
#pragma unroll
        for (int sub = 0; sub < KSUB; sub++) {
          const uint32_t a_lo = a_lo0 + s * stage_units + sub * sub_units;
          const uint32_t b_lo = b_lo0 + s * stage_units + sub * sub_units;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; k++) {
            const uint64_t ad = ((uint64_t)a_hi << 32) | (a_lo + k * a_kstep);
            const uint64_t bd = ((uint64_t)b_hi << 32) | (b_lo + k * b_kstep);
            if (kPair) tc_mma_pair(d_tmem, ad, bd, p.idesc, accum);
            else tc_mma(d_tmem, ad, bd, p.idesc, accum);
            accum = 1;
          }
        }
        // the stage is free (in both CTAs) once these MMAs have read it
        if (kPair) tc_commit_pair(empty0 + s * 8); else tc_commit(empty0 + s * 8);
        s = s1; ph = ph1;
      }
      if (ok) {  // accumulator complete
        if (kPair) tc_commit_pair(smem_u32(&tfull_bar[acc])); else tc_commit(smem_u32(&tfull_bar[acc]));
      }
    }
    if (!ok || *abort_flag) {
      // make sure no MMA is still writing tensor memory before it is freed
      if (kPair) tc_commit_pair(smem_u32(&tfull_bar[0])); else tc_commit(smem_u32(&tfull_bar[0]));
      const long long t0 = now_cycles();
      while (now_cycles() - t0 < 2000000ll) {}
    }
  } else if (warp >= FIRST_EPI_WARP) {
    // ------------------------------- epilogue -------------------------------
    // Two warps share each TMEM lane quarter and take alternate 32-column chunks.  A warp reads
    // its 32 x 32 chunk (one row per lane), applies the epilogue, then turns the chunk through a
    // swizzled staging buffer so that global stores cover whole row segments.
    const int q = warp & 3;              // TMEM lane quarter this warp may read
    const int hsel = (warp - FIRST_EPI_WARP) >> 2;    // which of the two warps of the quarter
    uint8_t* stg = staging + (size_t)(warp - FIRST_EPI_WARP) * STAGING_BYTES;
    float* bias_s = reinterpret_cast<float*>(stg + 2048);  // bias of this warp's columns, chunk by chunk
    float* bias_r = reinterpret_cast<float*>((uint8_t*)bars + 256) + (warp - FIRST_EPI_WARP) * 32;
    uint32_t tile = 0;
    bool ok = true;
    if constexpr (kMode != EPI_GENERIC && !kSoftmax) {
      // The specialised flavours.  What keeps a tile's epilogue short enough to hide behind the
      // next tile's main loop: the work-item coordinates advance by mixed-radix addition (no
      // division per tile); the bias of the NEXT tile is fetched while this tile is worked on; the
      // TMEM read of the next chunk is in flight while the current chunk is converted and stored;
      // and a lane stores its row segment straight from registers.
      const int nch = p.bn >> 6;
      constexpr bool kHasXf = kMode == EPI_RESIDUAL || kMode == EPI_DGELU;
      const bf16* xsrc = kMode == EPI_DGELU ? p.aux : kMode == EPI_RESIDUAL ? p.residual : nullptr;
      // digits of the work index (n tile fastest, then m tile, batch, split) and of the step
      int nt, mt, z, sp, d_nt, d_mt, d_z, d_sp;
      {
        int r = w_first;
        sp = r / per_split; r -= sp * per_split;
        z = r / tiles_per_z; r -= z * tiles_per_z;
        mt = r / p.n_tiles; nt = r - mt * p.n_tiles;
        r = w_step;
        d_sp = r / per_split; r -= d_sp * per_split;
        d_z = r / tiles_per_z; r -= d_z * tiles_per_z;
        d_mt = r / p.n_tiles; d_nt = r - d_mt * p.n_tiles;
      }
      auto advance = [&](int& nt_, int& mt_, int& z_, int& sp_) {
        nt_ += d_nt;
        int c = nt_ >= p.n_tiles ? 1 : 0;
        nt_ -= c ? p.n_tiles : 0;
        mt_ += d_mt + c;
        c = mt_ >= p.m_tiles ? 1 : 0;
        mt_ -= c ? p.m_tiles : 0;
        z_ += d_z + c;
        c = z_ >= p.batch ? 1 : 0;
        z_ -= c ? p.batch : 0;
        sp_ += d_sp + c;
      };
      // This warp's i-th chunk, in units of 32 columns.  The two warps of a quarter interleave
      // their chunks; with tile stores they interleave pairs of chunks, so that a warp owns whole
      // 64-column (128-byte) groups.
      const bool tma_out = p.tma_store != 0;
      auto ccol = [&](int i) { return tma_out ? 2 * (hsel + 2 * (i >> 1)) + (i & 1) : hsel + 2 * i; };
      const uint32_t stg_tile = smem_u32(stg);
      // bias values of this warp's columns of tile `nt_`, one value per lane and chunk
      auto fetch_bias = [&](int nt_, float (&b)[4]) {
#pragma unroll
        for (int i = 0; i < 4; i++) {
          const int n = nt_ * p.bn + ccol(i) * 32 + lane;
          b[i] = (i < nch && p.bias && n < p.N) ? p.bias[n] : 0.f;
        }
      };
      float bnext[4];
      if (w_first < p.total_work && !tma_out) {
        fetch_bias(nt, bnext);
#pragma unroll
        for (int i = 0; i < 4; i++) bias_s[i * 32 + lane] = bnext[i];
        __syncwarp();
      }
      for (int w = w_first; w < p.total_work && ok; w += w_step, tile++) {
        const int zo = p.hdiv == 1 ? z : z / p.hdiv, zi = p.hdiv == 1 ? 0 : z - zo * p.hdiv;
        const uint32_t acc = tile & 1, use = tile >> 1;
        const int m_warp = mt * mt_rows + (int)cta_rank * BM + q * 32;  // first row of this warp
        const int m = m_warp + lane;
        const bool row_ok = m < p.M;
        const long long zoff = zo * p.d_bo + zi * p.d_bi;
        const long long off0 = zoff + (long long)m * p.ldd;
        const int n_base = nt * p.bn;
        const float* bias_t = bias_s + (tile & 1) * 128;
        const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
        auto chunk_n0 = [&](int i) { return n_base + ccol(i) * 32; };
        auto chunk_ok = [&](int i) { return i < nch && chunk_n0(i) < p.N; };
        auto prefetch_x = [&](int i, uint4 (&x)[4]) {
          if (kHasXf && row_ok) {
            const uint4* src = reinterpret_cast<const uint4*>(xsrc + off0 + chunk_n0(i));
#pragma unroll
            for (int j = 0; j < 4; j++) x[j] = src[j];
          }
        };
        // the next work item and its bias (the loads travel while this tile is worked on)
        int nt2 = nt, mt2 = mt, z2 = z, sp2 = sp;
        advance(nt2, mt2, z2, sp2);
        const bool more = w + w_step < p.total_work && !tma_out;  // (of interest to the bias hand-over only)
        if (more) fetch_bias(nt2, bnext);
        uint4 x[4];
        const bool c0ok = chunk_ok(0);
        if (c0ok) prefetch_x(0, x);
        if (!mbar_wait(smem_u32(&tfull_bar[acc]), use & 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        auto release_acc = [&]() {  // every TMEM read of this tile has returned
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (kPair && !leader) mbar_arrive_cluster(mapa_u32(smem_u32(&tempty_bar[acc]), 0));
            else mbar_arrive(smem_u32(&tempty_bar[acc]));
          }
        };
        auto work = [&](const uint32_t (&a)[32], int i, bool has_next) {
          uint4 xc[4];
          if constexpr (kHasXf) {
#pragma unroll
            for (int j = 0; j < 4; j++) xc[j] = x[j];
            if (has_next) prefetch_x(i + 1, x);
          }
          const int n0 = chunk_n0(i);
          if (tma_out) {
            // an even chunk opens a 64-column group: the tile store of the previous group must
            // have read the staging tile; an odd chunk, or the last one, closes it
            if (!(i & 1)) {
              if (lane == 0) tma_store_wait_read();
              __syncwarp();
            }
            // The staging buffer holds the output tile, so the chunk's bias comes straight from
            // global memory (32 floats that every lane reads alike: one L1 line), or, for a
            // ragged chunk or no bias at all, from 32 floats of scratch.
            const float* bias_c = p.bias + n0;
            if (!p.bias || n0 + 32 > p.N) {
              __syncwarp();
              bias_r[lane] = (p.bias && n0 + lane < p.N) ? p.bias[n0 + lane] : 0.f;
              __syncwarp();
              bias_c = bias_r;
            }
            epi_chunk<kMode>(p, a, xc, bias_c, stg, lane, zoff, m_warp, n0, p.direct != 0, stg_tile, i & 1);
            if ((i & 1) || !has_next) {
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0 && m_warp < p.M) {
                auto slot = [&](int sl) { return p.d_perm[0] == sl ? m_warp : (p.d_perm[1] == sl ? zi : zo); };
                tma_store_4d(&tmD, stg_tile, n0 - (i & 1) * 32, slot(1), slot(2), slot(3));
              }
            }
          } else {
            epi_chunk<kMode>(p, a, xc, bias_t + i * 32, stg, lane, zoff, m_warp, n0, p.direct && n0 + 32 <= p.N);  // warp-uniform
          }
        };
        if (c0ok && kHasXf) {
          // the flavours with a row-shaped extra operand have no registers to spare for a second
          // chunk in flight
          uint32_t ra[32];
          for (int i = 0;; i++) {
            const bool v1 = chunk_ok(i + 1);
            tc_ld32_issue(trow + ccol(i) * 32, ra);
            tc_ld32_wait(ra);
            if (!v1) release_acc();
            work(ra, i, v1);
            if (!v1) break;
          }
        } else if (c0ok) {
          uint32_t ra[32], rb[32];
          tc_ld32_issue(trow + ccol(0) * 32, ra);
          for (int i = 0;; i += 2) {
            const bool v1 = chunk_ok(i + 1);
            tc_ld32_wait(ra);
            if (v1) tc_ld32_issue(trow + ccol(i + 1) * 32, rb); else release_acc();
            work(ra, i, v1);
            if (!v1) break;
            const bool v2 = chunk_ok(i + 2);
            tc_ld32_wait(rb);
            if (v2) tc_ld32_issue(trow + ccol(i + 2) * 32, ra); else release_acc();
            work(rb, i + 1, v2);
            if (!v2) break;
          }
        } else {
          release_acc();
        }
        if (more) {
          float* bias_n = bias_s + ((tile + 1) & 1) * 128;
#pragma unroll
          for (int i = 0; i < 4; i++) bias_n[i * 32 + lane] = bnext[i];
          __syncwarp();
        }
        nt = nt2; mt = mt2; z = z2; sp = sp2;
      }
    } else
    for (int w = w_first; w < p.total_work && ok; w += w_step, tile++) {
      const int split = w / per_split;
      int r = w - split * per_split;
      const int z = r / tiles_per_z;
      r -= z * tiles_per_z;
      const int mt = r / p.n_tiles, nt = r - mt * p.n_tiles;
      const int zo = z / p.hdiv, zi = z - zo * p.hdiv;
      const uint32_t acc = tile & 1, use = tile >> 1;
      const int m_warp = mt * mt_rows + (int)cta_rank * BM + q * 32;  // first row of this warp
      const int m = m_warp + lane;
      const long long zoff = zo * p.d_bo + zi * p.d_bi;
      const long long off0 = zoff + (long long)m * p.ldd;
      const int n_base = nt * p.bn;
      if constexpr (kSoftmax) {
        if (!mbar_wait(smem_u32(&tfull_bar[acc]), use & 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        // Scaled masked softmax over whole rows (one n-tile of at most 128 columns holds a row).
        // Each warp keeps its (up to) two 32-column chunks in registers; the two warps of a
        // quarter exchange row maxima and row sums through shared memory.
        int len = p.seq_lens ? p.seq_lens[zo] : p.N;
        len = min(max(len, 1), p.N);
        const int c0 = hsel, c1 = hsel + 2;
        const bool h0 = c0 * 32 < p.N && c0 < p.bn / 32, h1 = c1 * 32 < p.N && c1 < p.bn / 32;
        float2 v0[16], v1[16];
        float mx = -INFINITY;
        const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
        if (h0) {
          tc_ld32(trow + c0 * 32, v0);
#pragma unroll
          for (int j = 0; j < 16; j++) {
            v0[j].x = (c0 * 32 + 2 * j < len) ? v0[j].x * p.alpha : -INFINITY;
            v0[j].y = (c0 * 32 + 2 * j + 1 < len) ? v0[j].y * p.alpha : -INFINITY;
            mx = fmaxf(mx, fmaxf(v0[j].x, v0[j].y));
          }
        }
        if (h1) {
          tc_ld32(trow + c1 * 32, v1);
#pragma unroll
          for (int j = 0; j < 16; j++) {
            v1[j].x = (c1 * 32 + 2 * j < len) ? v1[j].x * p.alpha : -INFINITY;
            v1[j].y = (c1 * 32 + 2 * j + 1 < len) ? v1[j].y * p.alpha : -INFINITY;
            mx = fmaxf(mx, fmaxf(v1[j].x, v1[j].y));
          }
        }
        // the accumulator is in registers now: hand it back before the slow part
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
        if (kPair && !leader) mbar_arrive_cluster(mapa_u32(smem_u32(&tempty_bar[acc]), 0));
        else mbar_arrive(smem_u32(&tempty_bar[acc]));
      }
        const int seq = (int)tile * 2 + 1;
        const int me = q * 2 + hsel, other = q * 2 + (hsel ^ 1);
        xmax[me * 32 + lane] = mx;
        if (!pair_sync(xflag, me, other, seq, lane, abort_flag, p.status)) { ok = false; break; }
        mx = fmaxf(mx, xmax[other * 32 + lane]);
        float sum = 0.f;
        if (h0) {
#pragma unroll
          for (int j = 0; j < 16; j++) {
            v0[j].x = __expf(v0[j].x - mx);
            v0[j].y = __expf(v0[j].y - mx);
            sum += v0[j].x + v0[j].y;
          }
        }
        if (h1) {
#pragma unroll
          for (int j = 0; j < 16; j++) {
            v1[j].x = __expf(v1[j].x - mx);
            v1[j].y = __expf(v1[j].y - mx);
            sum += v1[j].x + v1[j].y;
          }
        }
        xsum[me * 32 + lane] = sum;
        if (!pair_sync(xflag, me, other, seq + 1, lane, abort_flag, p.status)) { ok = false; break; }
        sum += xsum[other * 32 + lane];
        const float inv = 1.0f / sum;
        if (h0) {
#pragma unroll
          for (int j = 0; j < 16; j++) v0[j] = __fmul2_rn(v0[j], splat2(inv));
          stage_store_bf16(stg, lane, v0, reinterpret_cast<bf16*>(p.D) + zoff, p.ldd, m_warp, c0 * 32, p.M, p.N,
                           p.vec_ok);
        }
        if (h1) {
#pragma unroll
          for (int j = 0; j < 16; j++) v1[j] = __fmul2_rn(v1[j], splat2(inv));
          stage_store_bf16(stg, lane, v1, reinterpret_cast<bf16*>(p.D) + zoff, p.ldd, m_warp, c1 * 32, p.M, p.N,
                           p.vec_ok);
        }
        continue;
      } else {
      // Software pipeline over this warp's 32-column chunks (cidx = hsel, hsel + 2, ...): the
      // TMEM read of the next chunk and the global loads it needs (GELU' argument or residual
      // row) are issued before the current chunk is worked on.
      const int nch = p.bn >> 6;
      const bool row_ok = m < p.M;
      const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + acc * 256;
      // the row-shaped extra operand, if any
      const bf16* xsrc = kMode == EPI_GENERIC ? (p.act == 2 ? p.aux : p.residual)
                       : kMode == EPI_DGELU ? p.aux : kMode == EPI_RESIDUAL ? p.residual : nullptr;
      auto chunk_n0 = [&](int i) { return n_base + (hsel + 2 * i) * 32; };
      auto chunk_ok = [&](int i) { return i < nch && chunk_n0(i) < p.N; };
      auto prefetch_x = [&](int i, uint4 (&x)[4]) {
        const int n0 = chunk_n0(i);
        if ((kHasX && row_ok) || (kMode == EPI_GENERIC && xsrc && row_ok && p.vec_ok && n0 + 32 <= p.N)) {
          const uint4* src = reinterpret_cast<const uint4*>(xsrc + off0 + n0);
#pragma unroll
          for (int j = 0; j < 4; j++) x[j] = src[j];
        }
      };
      auto release_acc = [&]() {  // every TMEM read of this tile has returned
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kPair && !leader) mbar_arrive_cluster(mapa_u32(smem_u32(&tempty_bar[acc]), 0));
          else mbar_arrive(smem_u32(&tempty_bar[acc]));
        }
      };
      auto process = [&](uint32_t (&a)[32], uint4 (&x)[4], int i, bool has_next) {
        const int n0 = chunk_n0(i);
        if constexpr (kMode != EPI_GENERIC) {
          uint4 xc[4];
          if constexpr (kHasX) {
#pragma unroll
            for (int j = 0; j < 4; j++) xc[j] = x[j];
            // the extra operand of the next chunk travels while this chunk is worked on
            if (has_next) prefetch_x(i + 1, x);
          }
          epi_chunk<kMode>(p, a, xc, bias_s + i * 32, stg, lane, zoff, m_warp, n0, false);
          return;
        }
        const long long off = off0 + n0;
        const bool fullv = p.vec_ok && (n0 + 32 <= p.N);
        float2 v[16];
#pragma unroll
        for (int j = 0; j < 16; j++) v[j] = make_float2(__uint_as_float(a[2 * j]), __uint_as_float(a[2 * j + 1]));
        if (p.alpha != 1.0f) {
          const float2 a2 = splat2(p.alpha);
#pragma unroll
          for (int j = 0; j < 16; j++) v[j] = __fmul2_rn(v[j], a2);
        }
        if (p.bias) {  // this warp's bias values were put in shared memory at the start of the tile
          const float4* b4 = reinterpret_cast<const float4*>(bias_s + i * 32);
#pragma unroll
          for (int j = 0; j < 8; j++) {
            const float4 t = b4[j];
            v[2 * j] = __fadd2_rn(v[2 * j], make_float2(t.x, t.y));
            v[2 * j + 1] = __fadd2_rn(v[2 * j + 1], make_float2(t.z, t.w));
          }
        }
        if (p.act == 1) {
          if (p.aux) stage_store_bf16(stg, lane, v, p.aux + zoff, p.ldd, m_warp, n0, p.M, p.N, p.vec_ok);
#pragma unroll
          for (int j = 0; j < 16; j++) v[j] = gelu_fast2(v[j]);
        } else if (p.act == 2 && row_ok) {
          if (fullv) {
#pragma unroll
            for (int j = 0; j < 4; j++) {
              v[4 * j] = __fmul2_rn(v[4 * j], gelu_grad_fast2(bf162_to_f2(x[j].x)));
              v[4 * j + 1] = __fmul2_rn(v[4 * j + 1], gelu_grad_fast2(bf162_to_f2(x[j].y)));
              v[4 * j + 2] = __fmul2_rn(v[4 * j + 2], gelu_grad_fast2(bf162_to_f2(x[j].z)));
              v[4 * j + 3] = __fmul2_rn(v[4 * j + 3], gelu_grad_fast2(bf162_to_f2(x[j].w)));
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; j++) {
              float2 u = make_float2(0.f, 0.f);
              if (n0 + 2 * j < p.N) u.x = __bfloat162float(p.aux[off + 2 * j]);
              if (n0 + 2 * j + 1 < p.N) u.y = __bfloat162float(p.aux[off + 2 * j + 1]);
              v[j] = __fmul2_rn(v[j], gelu_grad_fast2(u));
            }
          }
        }
        if (p.residual && row_ok) {
          if (fullv && p.act != 2) {
#pragma unroll
            for (int j = 0; j < 4; j++) {
              v[4 * j] = __fadd2_rn(v[4 * j], bf162_to_f2(x[j].x));
              v[4 * j + 1] = __fadd2_rn(v[4 * j + 1], bf162_to_f2(x[j].y));
              v[4 * j + 2] = __fadd2_rn(v[4 * j + 2], bf162_to_f2(x[j].z));
              v[4 * j + 3] = __fadd2_rn(v[4 * j + 3], bf162_to_f2(x[j].w));
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; j++) {
              if (n0 + 2 * j < p.N) v[j].x += __bfloat162float(p.residual[off + 2 * j]);
              if (n0 + 2 * j + 1 < p.N) v[j].y += __bfloat162float(p.residual[off + 2 * j + 1]);
            }
          }
        }
        // the extra operand of the next chunk travels while this chunk is stored
        if (has_next) prefetch_x(i + 1, x);
        if (p.d_fp32)
          stage_store_f32(stg, lane, v, reinterpret_cast<float*>(p.D) + zoff, p.ldd, m_warp, n0, p.M, p.N,
                          p.vec_ok, p.accumulate);
        else
          stage_store_bf16(stg, lane, v, reinterpret_cast<bf16*>(p.D) + zoff, p.ldd, m_warp, n0, p.M, p.N,
                           p.vec_ok);
      };
      // before the accumulator is ready: bias values of this warp's columns to shared memory,
      // first chunk's extra operand on its way
      uint32_t a0[32];
      uint4 x[4];
      const bool c0ok = chunk_ok(0);
      if (kMode != EPI_GENERIC || p.bias) {
        for (int i = 0; i < nch; i++) {
          const int n = chunk_n0(i) + lane;
          bias_s[i * 32 + lane] = (p.bias && n < p.N) ? p.bias[n] : 0.f;
        }
        __syncwarp();
      }
      if (c0ok) prefetch_x(0, x);
      if (!mbar_wait(smem_u32(&tfull_bar[acc]), use & 1, abort_flag, p.status)) { ok = false; break; }
      tc_fence_after();
      if (c0ok) {
        for (int i = 0;; i++) {
          const bool v1 = chunk_ok(i + 1);
          tc_ld32_issue(trow + (hsel + 2 * i) * 32, a0);
          tc_ld32_wait(a0);
          if (!v1) release_acc();
          process(a0, x, i, v1);
          if (!v1) break;
        }
      } else {
        release_acc();
      }
      }
    }
    // tile stores read this CTA's shared memory: they end before the CTA does
    if (p.tma_store && lane == 0) tma_store_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (kPair) cluster_sync_all();  // neither CTA frees tensor memory while the other may still use it
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    if (kPair)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS)
                   : "memory");
  }
}

}  // namespace

static std::atomic<int> g_starve_next{0};
void gemm_tc_starve_next(int on) { g_starve_next.store(on ? 1 : 0); }

// Measurement hook (mslt_debug_set_gemm_variant): 0 = automatic choice, 1 = one CTA per tile,
// 2 = a CTA pair per 256 x 256 tile wherever the shape allows it.
static std::atomic<int> g_tile_variant{0};
static std::atomic<int> g_store_variant{0};  // 1 = no tile stores (bit 2 of the hook's argument)
void gemm_tc_set_variant(int v) { g_tile_variant.store(v & 3); g_store_variant.store((v >> 2) & 1); }

namespace {
// Per-device facts and one-time set-up, indexed by device ordinal (a process may drive several GPUs).
struct DeviceInfo {
  int num_sms = 0, smem_optin = 0;
  bool attr_set = false;
};
constexpr int kMaxDevices = 64;
DeviceInfo g_dev[kMaxDevices];
std::mutex g_dev_mu;
}  // namespace

int gemm_tc_launch(const mslt_gemm_desc& d, int* status, cudaStream_t st, char* err) {
  // the test hook is used up by this call even if an argument check below rejects it
  const bool starve = g_starve_next.exchange(0) != 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    snprintf(err, 256, "gemm: no CUDA device");
    return MSLT_ERR_CUDA;
  }
  DeviceInfo& di = g_dev[dev];
  {
    std::lock_guard<std::mutex> lock(g_dev_mu);
    if (di.num_sms == 0) {
      cudaDeviceGetAttribute(&di.num_sms, cudaDevAttrMultiProcessorCount, dev);
      cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
      if (di.num_sms <= 0) { snprintf(err, 256, "gemm: no CUDA device"); return MSLT_ERR_CUDA; }
    }
  }
  const int num_sms = di.num_sms, smem_optin = di.smem_optin;
  if (!status) { snprintf(err, 256, "gemm: the tensor-core kernel needs a device status word"); return MSLT_ERR_ARG; }
  TcParams p;
  memset(&p, 0, sizeof(p));
  p.M = d.M; p.N = d.N; p.K = d.K; p.batch = d.batch; p.hdiv = d.hdiv;
  p.a_mn = (d.a_rs == 1 && d.a_ks != 1) ? 1 : 0;
  p.b_mn = (d.b_rs == 1 && d.b_ks != 1) ? 1 : 0;
  p.bn = d.N <= 64 ? 64 : (d.N <= 128 ? 128 : 256);
  // Two CTAs per 256 x 256 tile: each SM then streams 64 instead of 96 bytes of operands per clock
  // from L2 (about 117 is what an SM was measured to take) and has six instead of four stages in
  // flight.
  const int variant = g_tile_variant.load();
  // Small products (under ~30 GFLOP, e.g. 16384 x 768 x 768) measured 5-10 % faster on single CTAs.
  const double flops = 2.0 * d.M * d.N * (double)d.K * d.batch;
  bool pair = variant != 1 && p.bn == 256 && d.M > BM && d.act != 3 && num_sms % 2 == 0 &&
              (variant == 2 || flops >= 30e9);
  // share of the SMs that the last wave of tiles keeps busy
  auto wave_eff = [](long long work, int units_) {
    const long long waves = (work + units_ - 1) / units_;
    return (double)work / (double)(waves * units_);
  };
  const bool can_split = d.split_k != 1 && d.d_fp32 && d.accumulate;
  if (p.bn == 256 && !can_split) {
    // few large tiles leave SMs idle: 128-wide tiles on single CTAs may fill the machine better
    const long long t256 = (long long)((d.M + (pair ? 2 * BM : BM) - 1) / (pair ? 2 * BM : BM)) *
                           ((d.N + 255) / 256) * d.batch;
    const long long t128 = (long long)((d.M + BM - 1) / BM) * ((d.N + 127) / 128) * d.batch;
    if (wave_eff(t128, num_sms) > 1.25 * wave_eff(t256, pair ? num_sms / 2 : num_sms)) {
      p.bn = 128;
      pair = false;
    }
  }
  const int tile_m = pair ? 2 * BM : BM;
  p.m_tiles = (d.M + tile_m - 1) / tile_m;
  p.n_tiles = (d.N + p.bn - 1) / p.bn;
  const int round_k = pair ? 2 * BK : BK;  // k extent of a ring stage (see KSUB in the kernel)
  p.kb_total = (d.K + round_k - 1) / round_k;
  const long long tiles = (long long)p.m_tiles * p.n_tiles * d.batch;
  const int units = pair ? num_sms / 2 : num_sms;  // CTAs or CTA pairs that run concurrently
  int splits = 1;
  if (d.split_k > 1) {
    splits = d.split_k;
  } else if (d.split_k == 0 && can_split && tiles < 2 * units && p.kb_total * round_k >= 8 * BK) {
    // the split count that fills the last wave best, with at least 256 k per split
    const int max_by_k = p.kb_total * round_k / (4 * BK);
    double best = wave_eff(tiles, units);
    for (int sp = 2; sp <= 16 && sp <= max_by_k; sp++) {
      const double e = wave_eff(tiles * sp, units);
      if (e > best + 0.04) { best = e; splits = sp; }
    }
  }
  if (splits > 1 && !(d.d_fp32 && d.accumulate)) {
    snprintf(err, 256, "gemm: split_k needs an fp32 accumulating output");
    return MSLT_ERR_ARG;
  }
  if (splits > p.kb_total) splits = p.kb_total;
  p.kb_per_split = (p.kb_total + splits - 1) / splits;
  p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
  const long long total = tiles * p.splits;
  if (total > 0x7fffffffll) { snprintf(err, 256, "gemm: too many tiles"); return MSLT_ERR_SIZE; }
  p.total_work = (int)total;
  if (d.act == 3 && (d.N > 128 || d.d_fp32 || splits != 1)) {
    snprintf(err, 256, "gemm: the softmax epilogue needs bf16 output rows of at most 128 columns");
    return MSLT_ERR_ARG;
  }
  const int stage_bytes = (pair ? 2 : 1) * (A_STAGE_BYTES + (pair ? p.bn / 2 : p.bn) * BK * 2);  // per CTA
  // barriers, then the softmax epilogue's exchange area or the 32 floats per epilogue warp that
  // hold the bias of a ragged chunk when the staging buffers carry output tiles
  const int book_bytes = 256 + (d.act == 3 ? 64 + 2 * NUM_EPI_WARPS * 32 * 4 : NUM_EPI_WARPS * 32 * 4);
  int stages = (smem_optin - NUM_EPI_WARPS * STAGING_BYTES - 1024 - book_bytes) / stage_bytes;
  if (stages > MAX_STAGES) stages = MAX_STAGES;
  if (stages < 2) { snprintf(err, 256, "gemm: not enough shared memory"); return MSLT_ERR_CUDA; }
  p.stages = stages;
  const size_t smem_bytes = (size_t)stages * stage_bytes + NUM_EPI_WARPS * STAGING_BYTES + 1024 + book_bytes;
  if ((int)smem_bytes > smem_optin) { snprintf(err, 256, "gemm: not enough shared memory"); return MSLT_ERR_CUDA; }

  MapVal ma, mb;
  const int nb = d.batch / d.hdiv;
  if (d.batch % d.hdiv) { snprintf(err, 256, "gemm: batch must be a multiple of hdiv"); return MSLT_ERR_ARG; }
  int rc = get_map(d.A, d.M, d.K, d.a_rs, d.a_ks, d.a_bo, d.a_bi, d.hdiv, nb, BM, &ma, err);
  if (rc) return rc;
  rc = get_map(d.B, d.N, d.K, d.b_rs, d.b_ks, d.b_bo, d.b_bi, d.hdiv, nb, pair ? p.bn / 2 : p.bn, &mb, err);
  if (rc) return rc;
  for (int i = 0; i < 3; i++) { p.a_perm[i] = ma.perm[i]; p.b_perm[i] = mb.perm[i]; }

  p.D = (char*)d.D; p.ldd = d.ldd; p.d_bo = d.d_bo; p.d_bi = d.d_bi;
  p.d_fp32 = d.d_fp32; p.accumulate = d.accumulate; p.alpha = d.alpha; p.bias = d.bias; p.act = d.act;
  p.aux = (bf16*)d.aux; p.residual = (const bf16*)d.residual; p.status = status;
  p.seq_lens = d.seq_lens;
  p.wait_limit = WAIT_LIMIT_CYCLES;
  if (starve) {  // armed by mslt_debug_starve_next_gemm
    p.starve = 1;
    p.wait_limit = 40000000ll;  // about 20 ms
  }
  // 16-byte vector access in the epilogue needs every row segment to start on a 16-byte boundary
  // in each of the buffers it touches (bf16 ones are the stricter case: 8 elements)
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  p.vec_ok = (d.ldd % 8 == 0 && d.d_bo % 8 == 0 && d.d_bi % 8 == 0 && al16(d.D) && al16(d.aux) &&
              al16(d.residual) && al16(d.bias)) ? 1 : 0;
  // straight-from-register row stores write 32 bytes at a time
  auto al32 = [](const void* q) { return ((uintptr_t)q & 31) == 0; };
  const long long esz = d.d_fp32 ? 4 : 2;
  p.direct = (p.vec_ok && al32(d.D) && (d.ldd * esz) % 32 == 0 && (d.d_bo * esz) % 32 == 0 && (d.d_bi * esz) % 32 == 0 &&
              !(d.d_fp32 && d.accumulate) &&  // vector reductions do better as whole row segments
              (!d.aux || d.act != 1 || (al32(d.aux) && (d.ldd * 2) % 32 == 0 && (d.d_bo * 2) % 32 == 0 && (d.d_bi * 2) % 32 == 0)))
                 ? 1 : 0;
  // instruction descriptor: fp32 accumulate, bf16 x bf16, operand majors, N and M of the tile
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.a_mn << 15) | ((uint32_t)p.b_mn << 16) |
            ((uint32_t)(p.bn >> 3) << 17) | ((uint32_t)(tile_m >> 4) << 24);

  // epilogue flavour: a specialised kernel where one fits, the general one otherwise
  int mode = EPI_GENERIC;
  const bool x_ok = p.vec_ok && d.N % 32 == 0;  // row-shaped extra operands are read 16 bytes at a time
  if (d.act == 3) mode = EPI_SOFTMAX;
  else if (d.d_fp32) { if (d.act == 0 && !d.residual) mode = EPI_F32; }
  else if (d.act == 0 && !d.residual) mode = EPI_STORE;
  else if (d.act == 0 && d.residual && x_ok) mode = EPI_RESIDUAL;
  else if (d.act == 1 && !d.residual) mode = d.aux ? EPI_GELU_AUX : EPI_GELU;
  else if (d.act == 2 && d.aux && !d.residual && x_ok) mode = EPI_DGELU;

  // Tile stores for the bf16 flavours: the output leaves through the copy engine as whole
  // 128-byte lines.  Row stores from registers (2 x 32 bytes per lane and chunk) were measured to
  // hold up the operand loads that share the SM's path to L2: 16384 x 2304 x 768 took 51.7 us with
  // them, 41.3 us with the stores left out, and a load stream beside such stores fell from 68 to
  // 12 bytes per clock per SM while beside copy-engine stores it kept 68.
  MapVal md;
  md.map = ma.map;
  p.tma_store = 0;
  if ((mode == EPI_STORE || mode == EPI_RESIDUAL || mode == EPI_GELU || mode == EPI_DGELU ||
       (mode == EPI_GELU_AUX && p.direct && d.N % 32 == 0)) &&
      p.bn >= 128 && p.vec_ok && d.N % 8 == 0 &&  // a tile store was seen to write whole 16-byte pieces
      g_store_variant.load() != 1) {
    char ignored[256];
    if (get_map(d.D, d.M, d.N, d.ldd, 1, d.d_bo, d.d_bi, d.hdiv, nb, 32, &md, ignored) == 0) {
      p.tma_store = 1;
      for (int i = 0; i < 3; i++) p.d_perm[i] = md.perm[i];
    } else {
      md.map = ma.map;
    }
  }

  typedef void (*KernelFn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const TcParams);
  static const KernelFn kernels[EPI_COUNT][2] = {
      {gemm_tc_kernel<EPI_STORE, false>, gemm_tc_kernel<EPI_STORE, true>},
      {gemm_tc_kernel<EPI_RESIDUAL, false>, gemm_tc_kernel<EPI_RESIDUAL, true>},
      {gemm_tc_kernel<EPI_GELU, false>, gemm_tc_kernel<EPI_GELU, true>},
      {gemm_tc_kernel<EPI_GELU_AUX, false>, gemm_tc_kernel<EPI_GELU_AUX, true>},
      {gemm_tc_kernel<EPI_DGELU, false>, gemm_tc_kernel<EPI_DGELU, true>},
      {gemm_tc_kernel<EPI_F32, false>, gemm_tc_kernel<EPI_F32, true>},
      {gemm_tc_kernel<EPI_GENERIC, false>, gemm_tc_kernel<EPI_GENERIC, true>},
      {gemm_tc_kernel<EPI_SOFTMAX, false>, nullptr}};
  std::unique_lock<std::mutex> dev_lock(g_dev_mu);
  if (!di.attr_set) {
    for (int mo = 0; mo < EPI_COUNT; mo++)
      for (int pr = 0; pr < 2; pr++) {
        if (!kernels[mo][pr]) continue;
        cudaError_t e = cudaFuncSetAttribute((const void*)kernels[mo][pr], cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin);
        if (e != cudaSuccess) { snprintf(err, 256, "gemm: cudaFuncSetAttribute: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
      }
    di.attr_set = true;
  }
  dev_lock.unlock();
  const KernelFn fn = kernels[mode][pair ? 1 : 0];
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (pair) {
    const int clusters = p.total_work < units ? p.total_work : units;
    cfg.gridDim = dim3(2 * clusters);
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
  } else {
    cfg.gridDim = dim3(p.total_work < num_sms ? p.total_work : num_sms);
  }
  cudaError_t e = cudaLaunchKernelEx(&cfg, fn, ma.map, mb.map, md.map, p);
  if (e != cudaSuccess) { snprintf(err, 256, "gemm: launch failed: %s", cudaGetErrorString(e)); return MSLT_ERR_CUDA; }
  return 0;
}

}  // namespace mslt
